// rest_kv_commit: after acceptance, move the K/V rows of the accepted draft nodes (tree slots
// L + node) to the contiguous slots L .. L + len - 1, so that the next decoding step sees an
// ordinary prefix.  Not in the paper (it never describes the cache); every implementation of
// the loop of Sec. 3.2 needs it.
//
// One thread block per context; its warps take the (kv head, K or V) units in turn.  A lane owns
// the same 8-byte column of every row, so reading all accepted rows into registers first and
// writing them afterwards is race-free even though source and destination slots overlap (a
// destination slot i may be the source of an earlier path position): all conflicts are inside
// one thread's program order.  The new length is written by the same block after a block
// barrier, when every warp that reads the old length has done so: d_new_kv_len may therefore
// be the very array the old lengths are read from, whatever the size of the grid.
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.cuh"
#include "rest.h"

namespace {

constexpr int kMaxDepth = REST_MAX_M;

constexpr int kCommitThreads = 512;

__global__ void __launch_bounds__(kCommitThreads)
rest_kv_commit_kernel(uint2* __restrict__ k, uint2* __restrict__ v, int64_t kv_b, int64_t kv_h, int64_t kv_l,
                      const int32_t* kv_len, const int32_t* __restrict__ accept_nodes,
                      const int32_t* __restrict__ accept_len, int B, int H_kv, int N, int max_depth,
                      int32_t* new_kv_len) {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int b = blockIdx.x;
  // kv_len and new_kv_len may be the same array: plain (coherent) loads, no restrict
  const int L = *reinterpret_cast<const volatile int32_t*>(kv_len + b);
  int len = accept_len[b];
  len = len < 0 ? 0 : (len > max_depth ? max_depth : len);
  int node[kMaxDepth];
#pragma unroll
  for (int i = 0; i < kMaxDepth; ++i) {
    node[i] = 0;
    if (i < len) {
      const int nd = accept_nodes[(int64_t)b * max_depth + i];
      node[i] = nd < 0 ? 0 : (nd >= N ? N - 1 : nd);
    }
  }
  for (int unit = warp; unit < 2 * H_kv; unit += kCommitThreads / 32) {   // warp-uniform
    const int which = unit & 1, h = unit >> 1;
    // strides are in bf16 elements; a uint2 is four of them
    uint2* base = (which ? v : k) + (b * kv_b + h * kv_h) / 4;
    uint2 rows[kMaxDepth];
#pragma unroll
    for (int i = 0; i < kMaxDepth; ++i)
      if (i < len) rows[i] = base[((int64_t)(L + node[i]) * kv_l) / 4 + lane];
#pragma unroll
    for (int i = 0; i < kMaxDepth; ++i)
      if (i < len) base[((int64_t)(L + i) * kv_l) / 4 + lane] = rows[i];
  }
  __syncthreads();                      // every warp of this context has read the old length
  if (new_kv_len && threadIdx.x == 0) new_kv_len[b] = L + len;
}

}  // namespace

extern "C" rest_status rest_kv_commit(void* d_k, void* d_v, const int64_t* kv_strides,
                                      const int32_t* d_kv_len, const int32_t* d_accept_nodes,
                                      const int32_t* d_accept_len, int32_t B, int32_t H_kv, int32_t N,
                                      int32_t D, int32_t max_depth, int32_t* d_new_kv_len, void* stream) {
  if (B < 0 || H_kv < 1 || N < 1 || max_depth < 0 || !kv_strides) return REST_INVALID_ARG;
  if (B == 0 || max_depth == 0) {
    // nothing can have been accepted; the new length equals the old one, which the caller has
    if (B > 0 && d_new_kv_len && d_kv_len)
      REST_CUDA_TRY(cudaMemcpyAsync(d_new_kv_len, d_kv_len, sizeof(int32_t) * (size_t)B,
                                    cudaMemcpyDeviceToDevice, static_cast<cudaStream_t>(stream)));
    return REST_OK;
  }
  if (!d_k || !d_v || !d_kv_len || !d_accept_nodes || !d_accept_len) return REST_INVALID_ARG;
  if (D != REST_HEAD_DIM || max_depth > kMaxDepth) return REST_UNSUPPORTED;
  for (int i = 0; i < 3; ++i)
    if (kv_strides[i] < 0 || (kv_strides[i] % 8) != 0) return REST_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(d_k) | reinterpret_cast<uintptr_t>(d_v)) & 15) return REST_INVALID_ARG;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)B, 1, 1);
  cfg.blockDim = dim3(kCommitThreads, 1, 1);
  cfg.stream = static_cast<cudaStream_t>(stream);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  REST_CUDA_TRY(cudaLaunchKernelEx(&cfg, rest_kv_commit_kernel, static_cast<uint2*>(d_k),
                                   static_cast<uint2*>(d_v), kv_strides[0], kv_strides[1], kv_strides[2],
                                   d_kv_len, d_accept_nodes, d_accept_len, (int)B, (int)H_kv, (int)N,
                                   (int)max_depth, d_new_kv_len));
  rest::count_launch();
  return REST_OK;
}
