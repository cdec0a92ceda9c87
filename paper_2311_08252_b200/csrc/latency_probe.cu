// rest_probe_dependent_reads: a measurement aid, not a step of the method.  One thread follows a
// chain of dependent global loads (idx = next[idx]) through a table much larger than L2 and
// reports the elapsed device time.  The suffix-array searches of Algorithm 1 are chains of
// exactly such loads (suffix-array entry, then the tokens it points to), so this number times
// the length of the chain is the latency floor of a single draft, whatever the bandwidth.
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.cuh"
#include "rest.h"

namespace {

__global__ void dependent_read_kernel(const uint32_t* __restrict__ next, uint64_t n, uint32_t start,
                                      uint32_t steps, uint64_t* __restrict__ out) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  uint32_t idx = start;
  uint64_t t0, t1;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
  for (uint32_t s = 0; s < steps; ++s) {
    if (idx >= n) idx = 0;                    // whatever the table holds, stay inside it
    idx = next[idx];
  }
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
  out[0] = t1 - t0;
  out[1] = idx;                               // keeps the chain alive
}

}  // namespace

extern "C" rest_status rest_probe_dependent_reads(const uint32_t* d_next, uint64_t n, uint32_t start,
                                                  uint32_t steps, uint64_t* d_out, void* stream) {
  if (!d_next || !d_out || n == 0 || n > 0xFFFFFFFFull) return REST_INVALID_ARG;
  dependent_read_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(d_next, n, start, steps, d_out);
  rest::count_launch();
  REST_CUDA_TRY(cudaGetLastError());
  return REST_OK;
}
