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

__global__ void sa_any_tie(const uint64_t* __restrict__ keys, int64_t n, unsigned int* __restrict__ flag) {
  const int64_t j = (int64_t)blockIdx.x * kBlock + threadIdx.x;
  if (j > 0 && j < n && keys[j] == keys[j - 1]) *flag = 1u;
}

// full = false: the order on the first 32 tokens (five rounds).  full = true: rounds go on, the
// compared length doubling each time, until no two suffixes are tied: the true suffix array.
static rest_status build_by_doubling(const int32_t* d_tokens, uint64_t n_tokens, int32_t sa_bytes, void* d_sa,
                                     void* d_ws, size_t ws_bytes, void* stream, bool full = false) {
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
    if (need_sort > temp_bytes - kAlign || need_scan > temp_bytes - kAlign) return REST_WORKSPACE_TOO_SMALL;
  }

  sa_init_rank<<<blocks, kBlock, 0, st>>>(d_tokens, rank, n);
  rest::count_launch();
  const uint32_t* result = nullptr;
  unsigned int* d_tie = reinterpret_cast<unsigned int*>(static_cast<unsigned char*>(temp) + temp_bytes - kAlign);
  for (int64_t h = 1; h < ((int64_t)1 << 31); h *= 2) {
    sa_make_keys<<<blocks, kBlock, 0, st>>>(rank, keys[0], vals[0], n, h);
    cub::DoubleBuffer<uint64_t> dk(keys[0], keys[1]);
    cub::DoubleBuffer<uint32_t> dv(vals[0], vals[1]);
    size_t tb = temp_bytes - kAlign;
    // ranks never exceed n <= 2^31 - 1 and tokens stay below 2^31: bit 63 and bit 31 are unused
    REST_CUDA_TRY(cub::DeviceRadixSort::SortPairs(temp, tb, dk, dv, n, 0, 64, st));
    result = dv.Current();
    rest::count_launch(2);
    bool last = !full && h == 16;
    if (full && h >= 16) {
      // the true suffix array is reached when no two suffixes compare equal any more (at the
      // latest when the compared length exceeds the stream); one flag read back per round
      unsigned int tie = 0;
      REST_CUDA_TRY(cudaMemsetAsync(d_tie, 0, sizeof(unsigned int), st));
      sa_any_tie<<<blocks, kBlock, 0, st>>>(dk.Current(), n, d_tie);
      rest::count_launch();
      REST_CUDA_TRY(cudaMemcpyAsync(&tie, d_tie, sizeof(tie), cudaMemcpyDeviceToHost, st));
      REST_CUDA_TRY(cudaStreamSynchronize(st));
      last = tie == 0 || 2 * h > n;
    }
    if (last) break;
    sa_mark_heads<<<blocks, kBlock, 0, st>>>(dk.Current(), head, n);
    tb = temp_bytes - kAlign;
    REST_CUDA_TRY(cub::DeviceScan::InclusiveScan(temp, tb, head, head, cub::Max(), n, st));
    sa_scatter_rank<<<blocks, kBlock, 0, st>>>(dv.Current(), head, rank, n);
    rest::count_launch(3);
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

extern "C" rest_status rest_suffix_array_build_full(const int32_t* d_tokens, uint64_t n_tokens,
                                                    int32_t sa_bytes, void* d_sa, void* d_ws,
                                                    size_t ws_bytes, void* stream) {
  if (!d_tokens || !d_sa || !d_ws || n_tokens == 0) return REST_INVALID_ARG;
  if (sa_bytes != 4 && sa_bytes != 8) return REST_INVALID_ARG;
  if (n_tokens > 0x7FFFFFFFull) return REST_UNSUPPORTED;
  if (reinterpret_cast<uintptr_t>(d_ws) & (kAlign - 1)) return REST_INVALID_ARG;
  return build_by_doubling(d_tokens, n_tokens, sa_bytes, d_sa, d_ws, ws_bytes, stream, true);
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

// ---------------------------------------------------------------------------------------
// Appending tokens to a datastore.  The order compares 32 tokens, so only the suffixes that
// start in the last 31 old positions (their windows now reach into the new tokens) and the
// suffixes of the new tokens can change place; all other old entries keep their relative
// order.  The "dirty" positions are sorted by themselves (the tail of the stream is a stream
// of its own), each is located among the old entries by bisection, and one pass writes the
// merged array.
// ---------------------------------------------------------------------------------------
namespace {

// order of two suffixes on their first 32 tokens, ties by position: true when a sorts before b
__device__ __forceinline__ bool suffix_before(const int32_t* __restrict__ T, int64_t n, int64_t a, int64_t b) {
  for (int k = 0; k < kKeyTokens; ++k) {
    const bool ea = a + k >= n, eb = b + k >= n;
    if (ea || eb) {
      if (ea != eb) return ea;
      break;
    }
    const uint32_t x = (uint32_t)T[a + k], y = (uint32_t)T[b + k];
    if (x != y) return x < y;
  }
  return a < b;
}

// slots of the old array that hold dirty positions (at most 31), in ascending slot order
template <typename SaT>
__global__ void sa_find_dirty_slots(const SaT* __restrict__ sa_old, int64_t n_old, int64_t t0,
                                    long long* __restrict__ slots, unsigned int* __restrict__ count) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_old; i += stride)
    if ((int64_t)sa_old[i] >= t0) {
      const unsigned int at = atomicAdd(count, 1u);
      if (at < 32) slots[at] = i;
    }
}
__global__ void sa_sort_dirty_slots(long long* __restrict__ slots, const unsigned int* __restrict__ count) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  const int c = (int)min(*count, 32u);
  for (int i = 1; i < c; ++i) {              // insertion sort of at most 31 numbers
    const long long v = slots[i];
    int j = i - 1;
    while (j >= 0 && slots[j] > v) { slots[j + 1] = slots[j]; --j; }
    slots[j + 1] = v;
  }
  for (int i = c; i < 32; ++i) slots[i] = 0x7FFFFFFFFFFFFFFFll;
}

// where[k] = first old slot whose (clean) entry sorts after dirty suffix k; old slots that hold
// dirty positions are stepped over
template <typename SaT, typename SegT>
__global__ void sa_locate_dirty(const int32_t* __restrict__ T, int64_t n, const SaT* __restrict__ sa_old,
                                int64_t n_old, int64_t t0, const SegT* __restrict__ seg, int64_t d,
                                long long* __restrict__ where) {
  const int64_t k = (int64_t)blockIdx.x * kBlock + threadIdx.x;
  if (k >= d) return;
  const int64_t q = t0 + (int64_t)seg[k];
  int64_t lo = 0, hi = n_old;                // answer in [lo, hi]
  while (lo < hi) {
    int64_t mid = lo + ((hi - lo) >> 1), probe = mid;
    while (probe < hi && (int64_t)sa_old[probe] >= t0) ++probe;     // skip dirty slots to the right
    if (probe == hi) {                       // nothing clean in [mid, hi): the answer is at most mid
      hi = mid;
      continue;
    }
    if (suffix_before(T, n, (int64_t)sa_old[probe], q)) lo = probe + 1; else hi = mid;
  }
  where[k] = lo;
}

template <typename SaT, typename SegT>
__global__ void sa_merge_append(const SaT* __restrict__ sa_old, int64_t n_old, int64_t t0,
                                const SegT* __restrict__ seg, int64_t d, const long long* __restrict__ where,
                                const long long* __restrict__ dirty_slots, SaT* __restrict__ sa_new) {
  __shared__ long long ds[32];
  if (threadIdx.x < 32) ds[threadIdx.x] = dirty_slots[threadIdx.x];
  __syncthreads();
  auto dirty_before = [&](int64_t slot) {    // old dirty slots below `slot`
    int c = 0;
    for (int i = 0; i < 32; ++i) c += ds[i] < slot;
    return (int64_t)c;
  };
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_old + d; i += stride) {
    if (i < n_old) {
      const int64_t p = (int64_t)sa_old[i];
      if (p >= t0) continue;                 // its new place comes from the sorted tail
      int64_t lo = 0, hi = d;                // dirty suffixes placed at or before slot i: where[k] <= i
      while (lo < hi) {
        const int64_t mid = (lo + hi) >> 1;
        if (where[mid] <= i) lo = mid + 1; else hi = mid;
      }
      sa_new[i - dirty_before(i) + lo] = (SaT)p;
    } else {
      const int64_t k = i - n_old, w = where[k];
      sa_new[w - dirty_before(w) + k] = (SaT)(t0 + (int64_t)seg[k]);
    }
  }
}

template <typename SaT>
rest_status append_impl(const int32_t* d_tokens, int64_t n_old, int64_t n_new, const SaT* sa_old, SaT* sa_new,
                        void* d_ws, size_t ws_bytes, cudaStream_t st) {
  const int64_t n = n_old + n_new;
  const int64_t t0 = n_old > (kKeyTokens - 1) ? n_old - (kKeyTokens - 1) : 0;
  const int64_t d = n - t0;                  // dirty positions t0 ... n - 1
  if (d > 0x7FFFFFFFll) return REST_UNSUPPORTED;
  // workspace: [where: d x 8][dirty slots: 32 x 8 + counter][tail array: d x 4][tail build scratch]
  unsigned char* ws = static_cast<unsigned char*>(d_ws);
  size_t o = 0;
  long long* where = reinterpret_cast<long long*>(ws + o); o += align_up((size_t)d * 8);
  long long* slots = reinterpret_cast<long long*>(ws + o); o += align_up(32 * 8);
  unsigned int* count = reinterpret_cast<unsigned int*>(ws + o); o += kAlign;
  int32_t* seg = reinterpret_cast<int32_t*>(ws + o); o += align_up((size_t)d * 4);
  const size_t seg_ws = sa_layout((uint64_t)d).total;
  if (ws_bytes < o + seg_ws) return REST_WORKSPACE_TOO_SMALL;
  rest_status rc = build_by_doubling(d_tokens + t0, (uint64_t)d, 4, seg, ws + o, seg_ws, st);
  if (rc != REST_OK) return rc;
  REST_CUDA_TRY(cudaMemsetAsync(count, 0, sizeof(unsigned int), st));
  const int sms = rest::sm_count() > 0 ? rest::sm_count() : 148;
  const unsigned wide = (unsigned)std::min<int64_t>((n + kBlock - 1) / kBlock, (int64_t)sms * 32);
  if (n_old > 0) sa_find_dirty_slots<SaT><<<wide, kBlock, 0, st>>>(sa_old, n_old, t0, slots, count);
  sa_sort_dirty_slots<<<1, 32, 0, st>>>(slots, count);
  sa_locate_dirty<SaT, int32_t><<<(unsigned)((d + kBlock - 1) / kBlock), kBlock, 0, st>>>(
      d_tokens, n, sa_old, n_old, t0, seg, d, where);
  sa_merge_append<SaT, int32_t><<<wide, kBlock, 0, st>>>(sa_old, n_old, t0, seg, d, where, slots, sa_new);
  rest::count_launch(4);
  REST_CUDA_TRY(cudaGetLastError());
  return REST_OK;
}

}  // namespace

extern "C" size_t rest_suffix_array_append_workspace_bytes(uint64_t n_new) {
  if (n_new == 0 || n_new > 0x7FFFFF00ull) return 0;
  const uint64_t d = n_new + kKeyTokens - 1;
  return align_up(d * 8) + align_up(32 * 8) + kAlign + align_up(d * 4) + sa_layout(d).total;
}

extern "C" rest_status rest_suffix_array_append(const int32_t* d_tokens, uint64_t n_old, uint64_t n_new,
                                                const void* d_sa_old, int32_t sa_bytes, void* d_sa_new,
                                                void* d_ws, size_t ws_bytes, void* stream) {
  if (!d_tokens || !d_sa_new || !d_ws || n_new == 0 || (n_old > 0 && !d_sa_old)) return REST_INVALID_ARG;
  if (sa_bytes != 4 && sa_bytes != 8) return REST_INVALID_ARG;
  if (n_old + n_new > (1ull << 40) || n_new > 0x7FFFFF00ull) return REST_UNSUPPORTED;
  if (sa_bytes == 4 && n_old + n_new > 0x7FFFFFFFull) return REST_INVALID_ARG;
  if (d_sa_old == d_sa_new) return REST_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(d_ws) & (kAlign - 1)) return REST_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (sa_bytes == 4)
    return append_impl<int32_t>(d_tokens, (int64_t)n_old, (int64_t)n_new, static_cast<const int32_t*>(d_sa_old),
                                static_cast<int32_t*>(d_sa_new), d_ws, ws_bytes, st);
  return append_impl<int64_t>(d_tokens, (int64_t)n_old, (int64_t)n_new, static_cast<const int64_t*>(d_sa_old),
                              static_cast<int64_t*>(d_sa_new), d_ws, ws_bytes, st);
}
