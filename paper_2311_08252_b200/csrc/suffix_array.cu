// rest_suffix_array_build: the datastore's suffix array, built on the device (Sec. 3.2
// "Datastore construction" / "Retrieving from the datastore": exact matching through a suffix
// array).  Set-up work, outside the decoding step.
//
// Order: suffixes compare on their first 32 tokens (tokens as unsigned integers, a suffix that
// ends early is smaller); suffixes equal on those 32 tokens are ordered by position.  A draft only
// ever looks at n_max + m <= 32 tokens of a suffix, so this order serves it exactly like the full
// lexicographic one, and it bounds the work on highly repetitive streams.
//
// Method: prefix doubling.  rank_1[i] = T[i] + 1; for h = 1, 2, 4, 8, 16 the pairs
// (rank_h[i], rank_h[i + h]) (0 past the end) are sorted as 64-bit keys together with i, and
// rank_2h[i] = 1 + the index of the first pair equal to i's pair.  The sort is stable and its input
// is in position order every time, so equal keys stay in position order; the values of the last
// sort are the suffix array.  The sort and the scan are CUB's device-wide primitives (a library
// routine for a set-up step); everything else is the few kernels below.
#include <cub/cub.cuh>
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.cuh"
#include "rest.h"

namespace {

constexpr int kBlock = 256;
constexpr size_t kAlign = 256;
constexpr size_t kCubTempBytes = 64ull << 20;     // fixed slice of the workspace for CUB's own scratch

__host__ __device__ inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct SaLayout {
  size_t keys_a, keys_b, vals_a, vals_b, rank, head, temp, total;
};
SaLayout sa_layout(uint64_t n) {
  SaLayout l;
  size_t o = 0;
  l.keys_a = o; o += align_up(n * 8);
  l.keys_b = o; o += align_up(n * 8);
  l.vals_a = o; o += align_up(n * 4);
  l.vals_b = o; o += align_up(n * 4);
  l.rank = o; o += align_up(n * 4);
  l.head = o; o += align_up(n * 4);
  l.temp = o; o += kCubTempBytes + align_up(n / 16);
  l.total = o;
  return l;
}

__global__ void sa_init_rank(const int32_t* __restrict__ T, uint32_t* __restrict__ rank, int64_t n) {
  const int64_t i = (int64_t)blockIdx.x * kBlock + threadIdx.x;
  if (i < n) rank[i] = (uint32_t)T[i] + 1u;
}
__global__ void sa_make_keys(const uint32_t* __restrict__ rank, uint64_t* __restrict__ keys,
                             uint32_t* __restrict__ vals, int64_t n, int64_t h) {
  const int64_t i = (int64_t)blockIdx.x * kBlock + threadIdx.x;
  if (i >= n) return;
  const uint32_t second = i + h < n ? rank[i + h] : 0u;
  keys[i] = ((uint64_t)rank[i] << 32) | second;
  vals[i] = (uint32_t)i;
}
__global__ void sa_mark_heads(const uint64_t* __restrict__ keys, uint32_t* __restrict__ head, int64_t n) {
  const int64_t j = (int64_t)blockIdx.x * kBlock + threadIdx.x;
  if (j < n) head[j] = (j == 0 || keys[j] != keys[j - 1]) ? (uint32_t)(j + 1) : 0u;
}
__global__ void sa_scatter_rank(const uint32_t* __restrict__ vals, const uint32_t* __restrict__ head,
                                uint32_t* __restrict__ rank, int64_t n) {
  const int64_t j = (int64_t)blockIdx.x * kBlock + threadIdx.x;
  if (j < n) rank[vals[j]] = head[j];
}
template <typename OutT>
__global__ void sa_write(const uint32_t* __restrict__ vals, OutT* __restrict__ sa, int64_t n) {
  const int64_t j = (int64_t)blockIdx.x * kBlock + threadIdx.x;
  if (j < n) sa[j] = (OutT)vals[j];
}

}  // namespace

extern "C" size_t rest_suffix_array_workspace_bytes(uint64_t n_tokens) {
  if (n_tokens == 0 || n_tokens > 0x7FFFFFFFull) return 0;
  return sa_layout(n_tokens).total;
}

extern "C" rest_status rest_suffix_array_build(const int32_t* d_tokens, uint64_t n_tokens,
                                               int32_t sa_bytes, void* d_sa, void* d_ws,
                                               size_t ws_bytes, void* stream) {
  if (!d_tokens || !d_sa || !d_ws || n_tokens == 0) return REST_INVALID_ARG;
  if (sa_bytes != 4 && sa_bytes != 8) return REST_INVALID_ARG;
  if (n_tokens > 0x7FFFFFFFull) return REST_UNSUPPORTED;
  if (reinterpret_cast<uintptr_t>(d_ws) & (kAlign - 1)) return REST_INVALID_ARG;
  const SaLayout l = sa_layout(n_tokens);
  if (ws_bytes < l.total) return REST_WORKSPACE_TOO_SMALL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  unsigned char* ws = static_cast<unsigned char*>(d_ws);
  uint64_t* keys[2] = {reinterpret_cast<uint64_t*>(ws + l.keys_a), reinterpret_cast<uint64_t*>(ws + l.keys_b)};
  uint32_t* vals[2] = {reinterpret_cast<uint32_t*>(ws + l.vals_a), reinterpret_cast<uint32_t*>(ws + l.vals_b)};
  uint32_t* rank = reinterpret_cast<uint32_t*>(ws + l.rank);
  uint32_t* head = reinterpret_cast<uint32_t*>(ws + l.head);
  void* temp = ws + l.temp;
  const size_t temp_bytes = l.total - l.temp;
  const int64_t n = (int64_t)n_tokens;
  const unsigned blocks = (unsigned)((n + kBlock - 1) / kBlock);

  // CUB's scratch needs, checked against the slice set aside for them
  {
    cub::DoubleBuffer<uint64_t> dk(keys[0], keys[1]);
    cub::DoubleBuffer<uint32_t> dv(vals[0], vals[1]);
    size_t need_sort = 0, need_scan = 0;
    REST_CUDA_TRY(cub::DeviceRadixSort::SortPairs(nullptr, need_sort, dk, dv, n, 0, 64, st));
    REST_CUDA_TRY(cub::DeviceScan::InclusiveScan(nullptr, need_scan, head, head, cub::Max(), n, st));
    if (need_sort > temp_bytes || need_scan > temp_bytes) return REST_WORKSPACE_TOO_SMALL;
  }

  sa_init_rank<<<blocks, kBlock, 0, st>>>(d_tokens, rank, n);
  rest::count_launch();
  const uint32_t* result = nullptr;
  for (int64_t h = 1; h <= 16; h *= 2) {
    sa_make_keys<<<blocks, kBlock, 0, st>>>(rank, keys[0], vals[0], n, h);
    cub::DoubleBuffer<uint64_t> dk(keys[0], keys[1]);
    cub::DoubleBuffer<uint32_t> dv(vals[0], vals[1]);
    size_t tb = temp_bytes;
    // ranks never exceed n <= 2^31 - 1 and tokens stay below 2^31: bit 63 and bit 31 are unused
    REST_CUDA_TRY(cub::DeviceRadixSort::SortPairs(temp, tb, dk, dv, n, 0, 64, st));
    result = dv.Current();
    rest::count_launch(2);
    if (h < 16) {
      sa_mark_heads<<<blocks, kBlock, 0, st>>>(dk.Current(), head, n);
      tb = temp_bytes;
      REST_CUDA_TRY(cub::DeviceScan::InclusiveScan(temp, tb, head, head, cub::Max(), n, st));
      sa_scatter_rank<<<blocks, kBlock, 0, st>>>(dv.Current(), head, rank, n);
      rest::count_launch(3);
    }
  }
  if (sa_bytes == 4)
    sa_write<int32_t><<<blocks, kBlock, 0, st>>>(result, static_cast<int32_t*>(d_sa), n);
  else
    sa_write<int64_t><<<blocks, kBlock, 0, st>>>(result, static_cast<int64_t*>(d_sa), n);
  rest::count_launch();
  REST_CUDA_TRY(cudaGetLastError());
  return REST_OK;
}
