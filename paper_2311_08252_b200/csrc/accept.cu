// rest_accept: draft acceptance (Sec. 3.2 "Draft acceptance").  One warp per context walks
// from the root; at each step the lanes look for a child of the current node whose token is
// the verifier's token there (siblings have distinct tokens, so at most one lane hits).
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.cuh"
#include "rest.h"

namespace {

constexpr int kWarpsPerBlock = 4;

__global__ void __launch_bounds__(kWarpsPerBlock * 32)
rest_accept_kernel(const int32_t* __restrict__ tokens, const int32_t* __restrict__ parents,
                   const int32_t* __restrict__ n_nodes, const int32_t* __restrict__ verifier,
                   int B, int N, int max_depth, int32_t* __restrict__ accept_len,
                   int32_t* __restrict__ accept_nodes, int32_t* __restrict__ out_tokens) {
  const int lane = threadIdx.x & 31;
  const int b = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
  // launched with programmatic stream serialisation: wait for the kernel before it in the
  // stream to complete before touching global memory
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (b >= B) return;   // warp-uniform
  const int32_t* tok = tokens + (int64_t)b * N;
  const int32_t* par = parents + (int64_t)b * N;
  const int32_t* ver = verifier + (int64_t)b * (N + 1);
  int32_t* an = accept_nodes + (int64_t)b * max_depth;
  int32_t* ot = out_tokens + (int64_t)b * (max_depth + 1);
  int nn = n_nodes[b];
  nn = nn < 0 ? 0 : (nn > N ? N : nn);
  for (int d = lane; d < max_depth; d += 32) an[d] = -1;
  for (int d = lane; d <= max_depth; d += 32) ot[d] = -1;
  __syncwarp();
  int cur = -1, len = 0;
  while (len < max_depth) {
    const int want = ver[cur + 1];
    int child = -1;
    for (int base = 0; base < nn; base += 32) {   // warp-uniform trip count
      const int i = base + lane;
      bool hit = i < nn && par[i] == cur && tok[i] == want;
      unsigned bal = __ballot_sync(0xFFFFFFFFu, hit);
      if (bal) { child = base + __ffs(bal) - 1; break; }
    }
    if (child < 0) break;
    if (lane == 0) { an[len] = child; ot[len] = want; }
    ++len;
    cur = child;
  }
  if (lane == 0) { ot[len] = ver[cur + 1]; accept_len[b] = len; }
}

}  // namespace

extern "C" rest_status rest_accept(const int32_t* d_tokens, const int32_t* d_parents,
                                   const int32_t* d_n_nodes, const int32_t* d_verifier_tokens,
                                   int32_t B, int32_t N, int32_t max_depth,
                                   int32_t* d_accept_len, int32_t* d_accept_nodes,
                                   int32_t* d_out_tokens, void* stream) {
  if (B < 0 || N < 1 || max_depth < 0) return REST_INVALID_ARG;
  if (B == 0) return REST_OK;
  if (!d_tokens || !d_parents || !d_n_nodes || !d_verifier_tokens || !d_accept_len ||
      (!d_accept_nodes && max_depth > 0) || !d_out_tokens)
    return REST_INVALID_ARG;
  int blocks = (B + kWarpsPerBlock - 1) / kWarpsPerBlock;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)blocks, 1, 1);
  cfg.blockDim = dim3(kWarpsPerBlock * 32, 1, 1);
  cfg.stream = static_cast<cudaStream_t>(stream);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  REST_CUDA_TRY(cudaLaunchKernelEx(&cfg, rest_accept_kernel, d_tokens, d_parents, d_n_nodes,
                                   d_verifier_tokens, (int)B, (int)N, (int)max_depth, d_accept_len,
                                   d_accept_nodes, d_out_tokens));
  rest::count_launch();
  return REST_OK;
}
