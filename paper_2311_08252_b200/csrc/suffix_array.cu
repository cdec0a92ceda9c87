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

static rest_status build_by_doubling(const int32_t* d_tokens, uint64_t n_tokens, int32_t sa_bytes, void* d_sa,
                                     void* d_ws, size_t ws_bytes, void* stream) {
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

// ---------------------------------------------------------------------------------------
// Second method, for streams the doubling above has no room for (more than 2^31 - 1 tokens,
// or a workspace smaller than its 32 bytes per token): positions are first thrown into
// buckets by their first token (a histogram, then a scatter with one cursor per bucket), so
// that the buckets follow each other in suffix order; consecutive buckets are then taken in
// groups of at most `cap` positions, and a group is sorted by itself: once by position, then,
// stably, by the packed 32-token key from its last 64-bit word to its first (least significant
// word first).  The result is the same order: first 32 tokens, ties by position.
// Needs one read-back of the histogram (the call synchronises the stream), 32 bytes of scratch
// per position of a group, and no first token that starts more than `cap` suffixes.
// ---------------------------------------------------------------------------------------
namespace {

constexpr int kKeyTokens = 32;
constexpr uint32_t kMaxBuckets = 1u << 22;

__global__ void sa_max_token(const int32_t* __restrict__ T, int64_t n, unsigned int* __restrict__ out) {
  unsigned int m = 0;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    const unsigned int t = (unsigned int)T[i];
    m = t > m ? t : m;
  }
  for (int o = 16; o > 0; o >>= 1) {
    const unsigned int u = __shfl_xor_sync(0xFFFFFFFFu, m, o);
    m = u > m ? u : m;
  }
  if ((threadIdx.x & 31) == 0) atomicMax(out, m);
}

// counts[bucket of T[i]] += 1, one atomic per distinct bucket of a warp
__global__ void sa_bucket_count(const int32_t* __restrict__ T, int64_t n, int shift,
                                unsigned long long* __restrict__ counts) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i0 = (int64_t)blockIdx.x * blockDim.x; i0 < n; i0 += stride) {
    const int64_t i = i0 + threadIdx.x;
    const bool in = i < n;
    const unsigned int bkt = in ? ((unsigned int)T[i] >> shift) : 0xFFFFFFFFu;
    const unsigned int peers = __match_any_sync(0xFFFFFFFFu, bkt);
    if (in && (int)(threadIdx.x & 31) == __ffs(peers) - 1) atomicAdd(counts + bkt, (unsigned long long)__popc(peers));
  }
}

// sa[cursor[bucket]++] = i (the order inside a bucket is settled by the sorts that follow)
template <typename OutT>
__global__ void sa_bucket_scatter(const int32_t* __restrict__ T, int64_t n, int shift,
                                  unsigned long long* __restrict__ cursor, OutT* __restrict__ sa) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i0 = (int64_t)blockIdx.x * blockDim.x; i0 < n; i0 += stride) {
    const int64_t i = i0 + threadIdx.x;
    const bool in = i < n;
    const unsigned int bkt = in ? ((unsigned int)T[i] >> shift) : 0xFFFFFFFFu;
    const unsigned int peers = __match_any_sync(0xFFFFFFFFu, bkt);
    const int lane = threadIdx.x & 31, leader = __ffs(peers) - 1;
    unsigned long long base = 0;
    if (in && lane == leader) base = atomicAdd(cursor + bkt, (unsigned long long)__popc(peers));
    base = __shfl_sync(0xFFFFFFFFu, base, leader);
    if (in) sa[base + __popc(peers & ((1u << lane) - 1u))] = (OutT)i;
  }
}

template <typename OutT>
__global__ void sa_group_load(const OutT* __restrict__ sa, int64_t first, int64_t count,
                              uint64_t* __restrict__ pos) {
  const int64_t j = (int64_t)blockIdx.x * kBlock + threadIdx.x;
  if (j < count) pos[j] = (uint64_t)sa[first + j];
}
template <typename OutT>
__global__ void sa_group_store(const uint64_t* __restrict__ pos, int64_t first, int64_t count,
                               OutT* __restrict__ sa) {
  const int64_t j = (int64_t)blockIdx.x * kBlock + threadIdx.x;
  if (j < count) sa[first + j] = (OutT)pos[j];
}
// key word `word` of the suffix at pos[j]: tokens word * per_word ... + per_word - 1 of the
// suffix, each as token + 1 in `bits` bits (0 past the end of the stream), first token highest
__global__ void sa_group_keys(const int32_t* __restrict__ T, int64_t n, const uint64_t* __restrict__ pos,
                              int64_t count, int word, int per_word, int bits, uint64_t* __restrict__ keys) {
  const int64_t j = (int64_t)blockIdx.x * kBlock + threadIdx.x;
  if (j >= count) return;
  const int64_t p = (int64_t)pos[j] + (int64_t)word * per_word;
  uint64_t key = 0;
  for (int t = 0; t < per_word; ++t) {
    const bool real = word * per_word + t < kKeyTokens && p + t < n;
    key = (key << bits) | (real ? (uint64_t)(uint32_t)T[p + t] + 1u : 0u);
  }
  keys[j] = key;
}

struct ChunkLayout { size_t keys_a, keys_b, pos_a, pos_b, counts, temp, total; };
ChunkLayout chunk_layout(uint64_t cap) {
  ChunkLayout l;
  size_t o = 0;
  l.keys_a = o; o += align_up(cap * 8);
  l.keys_b = o; o += align_up(cap * 8);
  l.pos_a = o; o += align_up(cap * 8);
  l.pos_b = o; o += align_up(cap * 8);
  l.counts = o; o += align_up(((size_t)kMaxBuckets + 1) * 8 * 2 + 256);
  l.temp = o; o += kCubTempBytes;
  l.total = o;
  return l;
}
constexpr uint64_t kChunkCapDefault = 1ull << 30;

template <typename OutT>
rest_status build_by_buckets(const int32_t* d_tokens, uint64_t n_tokens, OutT* d_sa, uint64_t max_group,
                             void* d_ws, size_t ws_bytes, cudaStream_t st) {
  // the largest group capacity the workspace allows (and the caller wants)
  const ChunkLayout fixed = chunk_layout(0);
  if (ws_bytes <= fixed.total + 4096) return REST_WORKSPACE_TOO_SMALL;
  uint64_t cap = (ws_bytes - fixed.total - 4 * kAlign) / 32;
  if (max_group > 0 && cap > max_group) cap = max_group;
  if (cap > n_tokens) cap = n_tokens;
  if (cap < 1024 && cap < n_tokens) return REST_WORKSPACE_TOO_SMALL;
  const ChunkLayout l = chunk_layout(cap);
  unsigned char* ws = static_cast<unsigned char*>(d_ws);
  uint64_t* keys[2] = {reinterpret_cast<uint64_t*>(ws + l.keys_a), reinterpret_cast<uint64_t*>(ws + l.keys_b)};
  uint64_t* pos[2] = {reinterpret_cast<uint64_t*>(ws + l.pos_a), reinterpret_cast<uint64_t*>(ws + l.pos_b)};
  unsigned long long* counts = reinterpret_cast<unsigned long long*>(ws + l.counts);
  unsigned int* d_max = reinterpret_cast<unsigned int*>(counts + 2 * ((size_t)kMaxBuckets + 1));
  void* temp = ws + l.temp;
  const int64_t n = (int64_t)n_tokens;
  const int sms = rest::sm_count() > 0 ? rest::sm_count() : 148;
  const unsigned wide = (unsigned)std::min<int64_t>((n + kBlock - 1) / kBlock, (int64_t)sms * 32);

  // token range -> bits per token, tokens per key word, bucket shift
  REST_CUDA_TRY(cudaMemsetAsync(d_max, 0, sizeof(unsigned int), st));
  sa_max_token<<<wide, kBlock, 0, st>>>(d_tokens, n, d_max);
  unsigned int max_token = 0;
  REST_CUDA_TRY(cudaMemcpyAsync(&max_token, d_max, sizeof(max_token), cudaMemcpyDeviceToHost, st));
  REST_CUDA_TRY(cudaStreamSynchronize(st));
  rest::count_launch();
  if (max_token >= 0x7FFFFFFFu) return REST_INVALID_ARG;
  int bits = 1;
  while ((1ull << bits) < (unsigned long long)max_token + 2) ++bits;      // symbols 0 ... max_token + 1
  const int per_word = 64 / bits, words = (kKeyTokens + per_word - 1) / per_word;
  int shift = 0;
  while (((unsigned long long)max_token >> shift) + 1 > kMaxBuckets) ++shift;
  const size_t nb = (size_t)(max_token >> shift) + 1;

  // histogram of first tokens, read back; bucket starts; groups of whole buckets
  REST_CUDA_TRY(cudaMemsetAsync(counts, 0, (2 * nb + 2) * sizeof(unsigned long long), st));
  sa_bucket_count<<<wide, kBlock, 0, st>>>(d_tokens, n, shift, counts);
  rest::count_launch();
  unsigned long long* h_counts = static_cast<unsigned long long*>(malloc((nb + 1) * sizeof(unsigned long long)));
  if (!h_counts) return REST_INVALID_ARG;
  cudaError_t e = cudaMemcpyAsync(h_counts, counts, nb * sizeof(unsigned long long), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) { free(h_counts); return rest::note_cuda_error(e, "read back of the bucket histogram"); }
  unsigned long long run = 0;
  bool too_big = false;
  for (size_t b = 0; b < nb; ++b) {
    const unsigned long long c = h_counts[b];
    too_big = too_big || c > cap;
    h_counts[b] = run;                      // start of bucket b
    run += c;
  }
  h_counts[nb] = run;
  if (too_big || run != n_tokens) { free(h_counts); return too_big ? REST_UNSUPPORTED : REST_INVALID_ARG; }
  unsigned long long* cursor = counts + nb + 1;
  e = cudaMemcpyAsync(cursor, h_counts, nb * sizeof(unsigned long long), cudaMemcpyHostToDevice, st);
  if (e != cudaSuccess) { free(h_counts); return rest::note_cuda_error(e, "bucket starts"); }
  sa_bucket_scatter<OutT><<<wide, kBlock, 0, st>>>(d_tokens, n, shift, cursor, d_sa);
  rest::count_launch();

  int pos_bits = 1;
  while ((1ull << pos_bits) < n_tokens) ++pos_bits;
  rest_status rc = REST_OK;
  size_t b0 = 0;
  while (b0 < nb && rc == REST_OK) {
    size_t b1 = b0 + 1;
    while (b1 < nb && h_counts[b1 + 1] - h_counts[b0] <= cap) ++b1;
    const int64_t first = (int64_t)h_counts[b0], count = (int64_t)(h_counts[b1] - h_counts[b0]);
    b0 = b1;
    if (count == 0) continue;
    const unsigned blocks = (unsigned)((count + kBlock - 1) / kBlock);
    sa_group_load<OutT><<<blocks, kBlock, 0, st>>>(d_sa, first, count, pos[0]);
    rest::count_launch();
    cub::DoubleBuffer<uint64_t> dp(pos[0], pos[1]);
    size_t tb = kCubTempBytes;
    if (count > 1) {
      e = cub::DeviceRadixSort::SortKeys(temp, tb, dp, count, 0, pos_bits, st);
      if (e != cudaSuccess) { rc = rest::note_cuda_error(e, "sort by position"); break; }
      rest::count_launch();
      for (int w = words - 1; w >= 0; --w) {
        sa_group_keys<<<blocks, kBlock, 0, st>>>(d_tokens, n, dp.Current(), count, w, per_word, bits, keys[0]);
        cub::DoubleBuffer<uint64_t> dk(keys[0], keys[1]);
        tb = kCubTempBytes;
        e = cub::DeviceRadixSort::SortPairs(temp, tb, dk, dp, count, 0, per_word * bits, st);
        if (e != cudaSuccess) { rc = rest::note_cuda_error(e, "sort by key word"); break; }
        rest::count_launch(2);
      }
      if (rc != REST_OK) break;
    }
    sa_group_store<OutT><<<blocks, kBlock, 0, st>>>(dp.Current(), first, count, d_sa);
    rest::count_launch();
  }
  free(h_counts);
  if (rc == REST_OK) REST_CUDA_TRY(cudaGetLastError());
  return rc;
}

}  // namespace

extern "C" size_t rest_suffix_array_workspace_bytes(uint64_t n_tokens) {
  if (n_tokens == 0 || n_tokens > (1ull << 40)) return 0;
  if (n_tokens <= 0x7FFFFFFFull) return sa_layout(n_tokens).total;
  return chunk_layout(n_tokens < kChunkCapDefault ? n_tokens : kChunkCapDefault).total + 4 * kAlign;
}

extern "C" size_t rest_suffix_array_min_workspace_bytes(uint64_t n_tokens, uint64_t largest_bucket) {
  if (n_tokens == 0 || n_tokens > (1ull << 40)) return 0;
  uint64_t cap = largest_bucket < 1024 ? 1024 : largest_bucket;
  if (cap > n_tokens) cap = n_tokens;
  return chunk_layout(cap).total + 4 * kAlign;
}

extern "C" rest_status rest_suffix_array_build(const int32_t* d_tokens, uint64_t n_tokens,
                                               int32_t sa_bytes, void* d_sa, void* d_ws,
                                               size_t ws_bytes, void* stream) {
  if (!d_tokens || !d_sa || !d_ws || n_tokens == 0) return REST_INVALID_ARG;
  if (sa_bytes != 4 && sa_bytes != 8) return REST_INVALID_ARG;
  if (n_tokens > (1ull << 40)) return REST_UNSUPPORTED;
  if (sa_bytes == 4 && n_tokens > 0x7FFFFFFFull) return REST_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(d_ws) & (kAlign - 1)) return REST_INVALID_ARG;
  // prefix doubling when the stream is short enough for 32-bit ranks and the workspace holds
  // its 32 bytes per token; else buckets by first token, each group sorted by itself
  if (n_tokens <= 0x7FFFFFFFull && ws_bytes >= sa_layout(n_tokens).total)
    return build_by_doubling(d_tokens, n_tokens, sa_bytes, d_sa, d_ws, ws_bytes, stream);
  return rest_suffix_array_build_in_groups(d_tokens, n_tokens, sa_bytes, d_sa, 0, d_ws, ws_bytes, stream);
}

extern "C" rest_status rest_suffix_array_build_in_groups(const int32_t* d_tokens, uint64_t n_tokens,
                                                         int32_t sa_bytes, void* d_sa, uint64_t max_group,
                                                         void* d_ws, size_t ws_bytes, void* stream) {
  if (!d_tokens || !d_sa || !d_ws || n_tokens == 0) return REST_INVALID_ARG;
  if (sa_bytes != 4 && sa_bytes != 8) return REST_INVALID_ARG;
  if (n_tokens > (1ull << 40)) return REST_UNSUPPORTED;
  if (sa_bytes == 4 && n_tokens > 0x7FFFFFFFull) return REST_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(d_ws) & (kAlign - 1)) return REST_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (sa_bytes == 4)
    return build_by_buckets<int32_t>(d_tokens, n_tokens, static_cast<int32_t*>(d_sa), max_group, d_ws, ws_bytes, st);
  return build_by_buckets<int64_t>(d_tokens, n_tokens, static_cast<int64_t*>(d_sa), max_group, d_ws, ws_bytes, st);
}
