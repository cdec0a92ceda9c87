// Datastore handle (Sec. 3.2 "Datastore construction": a token stream indexed by a suffix
// array) and its optional on-device validation, plus the library-wide status helpers.
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>

#include "common.cuh"
#include "rest.h"

namespace rest {

static thread_local char g_err[256] = "";
static std::atomic<uint64_t> g_launches{0};

rest_status note_cuda_error(cudaError_t e, const char* where) {
  snprintf(g_err, sizeof(g_err), "%s: %s", where, cudaGetErrorString(e));
  return REST_CUDA_ERROR;
}
void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

cudaError_t ensure_dynamic_smem(const void* kernel, int kernel_slot, size_t bytes) {
  constexpr int kMaxDev = 64, kSlots = kSmemSlots;
  static std::atomic<size_t> set_bytes[kMaxDev][kSlots];
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const bool cached = dev >= 0 && dev < kMaxDev && kernel_slot >= 0 && kernel_slot < kSlots;
  if (cached && set_bytes[dev][kernel_slot].load(std::memory_order_relaxed) >= bytes)
    return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e == cudaSuccess && cached) set_bytes[dev][kernel_slot].store(bytes, std::memory_order_relaxed);
  return e;
}

int sm_count() {
  constexpr int kMaxDev = 64;
  static std::atomic<int> cache[kMaxDev];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return 0; }
  const bool cached = dev >= 0 && dev < kMaxDev;
  if (cached) {
    const int have = cache[dev].load(std::memory_order_relaxed);
    if (have > 0) return have;
  }
  int n = 0;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
    (void)cudaGetLastError();
    return 0;
  }
  if (cached) cache[dev].store(n, std::memory_order_relaxed);
  return n;
}

}  // namespace rest

namespace {

constexpr int kOrderWindow = 32;   // tokens of each suffix that the order check compares

// flags[0] |= 1 token out of range, 2 entry out of range, 4 duplicate entry, 8 order violated
template <typename SaT>
__global__ void validate_kernel(const int32_t* __restrict__ T, const SaT* __restrict__ sa,
                                int64_t n, int64_t n_sa, uint32_t vocab, uint32_t* __restrict__ seen,
                                uint32_t* __restrict__ flags) {
  int64_t stride = (int64_t)gridDim.x * blockDim.x;
  uint32_t bad = 0;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    int32_t t = T[i];
    if (t < 0 || (uint32_t)t >= vocab) bad |= 1u;
    if (i >= n_sa) continue;             // the array may list fewer positions than there are tokens
    int64_t p = (int64_t)sa[i];
    if (p < 0 || p >= n) { bad |= 2u; continue; }
    uint32_t bit = 1u << (p & 31);
    if (atomicOr(&seen[p >> 5], bit) & bit) bad |= 4u;
    if (i > 0) {
      int64_t a = (int64_t)sa[i - 1];
      if (a < 0 || a >= n) continue;
      int cmp = 0;
      for (int k = 0; k < kOrderWindow; ++k) {
        bool ea = a + k >= n, eb = p + k >= n;
        if (ea || eb) { cmp = (ea && eb) ? 0 : (ea ? -1 : 1); break; }
        uint32_t x = (uint32_t)T[a + k], y = (uint32_t)T[p + k];
        if (x != y) { cmp = x < y ? -1 : 1; break; }
      }
      if (cmp > 0) bad |= 8u;
    }
  }
  if (bad) atomicOr(flags, bad);
}

// ---- bucket index ------------------------------------------------------------------------
constexpr uint32_t kIndexMaxVocab = 1u << 22;       // the first-token table has vocab + 1 entries
constexpr uint64_t kIndexMinEntries = 1ull << 12, kIndexMaxEntries = 1ull << 24;

constexpr size_t kIndexHeaderBytes = 256;           // word 0: "the datastore has an entry or token out of range"
struct IndexLayout {
  uint64_t entries;      // hash-table entries (a power of two; 0 = no index for this datastore)
  int64_t min_run;       // n-grams with fewer occurrences are not stored
  int levels, token_bits;
  size_t first_bytes, table_bytes, total;
};
IndexLayout index_layout(uint64_t n, uint32_t vocab) {
  IndexLayout l = {};
  if (vocab > kIndexMaxVocab || n < 2) return l;
  uint64_t e = kIndexMinEntries;
  while (e < 2 * n && e < kIndexMaxEntries) e <<= 1;
  l.entries = e;
  l.token_bits = 1;
  while ((1ull << l.token_bits) < (uint64_t)vocab) ++l.token_bits;
  l.levels = 60 / l.token_bits < rest::kIndexMaxLevel ? 60 / l.token_bits : rest::kIndexMaxLevel;
  if (l.levels < 2) { l.entries = 0; return l; }
  // at most n / min_run n-grams of each length are stored: the table stays at most one eighth
  // full, so a group of four overflows practically never (and an n-gram that finds its group
  // full is just left out)
  l.min_run = (int64_t)((8 * (uint64_t)(l.levels - 1) * n + e - 1) / e);
  if (l.min_run < 1) l.min_run = 1;
  l.first_bytes = (((size_t)vocab + 1) * 8 + 255) / 256 * 256;
  l.table_bytes = (size_t)e * 32;
  l.total = kIndexHeaderBytes + l.first_bytes + l.table_bytes;
  return l;
}
size_t validation_bytes(uint64_t n) {
  // one "seen" bit per position, rounded up to 32-bit words, plus one 256-byte block of flags
  return ((n + 31) / 32) * 4 + 256;
}

// The first tokens of the suffix in slot `slot`: tok[0 .. have), have <= kIndexMaxLevel (fewer
// when the suffix is shorter).  false when the entry or a token is out of range (such a
// datastore gets no usable index).
template <typename SaT>
__device__ __forceinline__ bool head_at(const int32_t* __restrict__ T, const SaT* __restrict__ sa, int64_t n,
                                        uint32_t vocab, int64_t slot, int32_t (&tok)[rest::kIndexMaxLevel], int& have) {
  const int64_t p = (int64_t)sa[slot];
  have = 0;
  if (p < 0 || p >= n) return false;
  for (int k = 0; k < rest::kIndexMaxLevel; ++k) {
    tok[k] = -1;
    if (p + k < n) {
      tok[k] = T[p + k];
      if (tok[k] < 0 || (uint32_t)tok[k] >= vocab) return false;
      have = k + 1;
    }
  }
  return true;
}
__device__ __forceinline__ bool same_head(const int32_t (&a)[rest::kIndexMaxLevel], int ha,
                                          const int32_t (&b)[rest::kIndexMaxLevel], int hb, int len) {
  if (ha < len || hb < len) return false;
  for (int k = 0; k < len; ++k)
    if (a[k] != b[k]) return false;
  return true;
}

// One thread per suffix-array slot.  The slot where a first token begins writes first[t]; for
// every n-gram length 2 ... levels the slots where a run of one n-gram begins and ends write
// that n-gram's lo and hi, provided the run has at least min_run members (seen by looking
// min_run - 1 slots ahead or back).
template <typename SaT>
__global__ void index_build_kernel(const int32_t* __restrict__ T, const SaT* __restrict__ sa, int64_t n,
                                   int64_t n_sa, uint32_t vocab, int64_t min_run, int levels, int token_bits,
                                   long long* __restrict__ first, unsigned long long* __restrict__ table,
                                   uint32_t group_mask, uint32_t* __restrict__ unusable) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_sa; i += stride) {
    int32_t me[rest::kIndexMaxLevel], up[rest::kIndexMaxLevel], dn[rest::kIndexMaxLevel], far[rest::kIndexMaxLevel];
    int hme = 0, hup = 0, hdn = 0, hfar = 0;
    // a datastore with an entry or a token out of range gets no index: searches then run over
    // the whole array, where such an entry is reported when it is met
    if (!head_at(T, sa, n, vocab, i, me, hme)) { *unusable = 1u; continue; }
    if (i > 0 && !head_at(T, sa, n, vocab, i - 1, up, hup)) hup = 0;
    if (i + 1 < n_sa && !head_at(T, sa, n, vocab, i + 1, dn, hdn)) hdn = 0;
    if (i == 0 || hup < 1 || up[0] != me[0]) first[me[0]] = i;
    for (int len = 2; len <= levels && len <= hme; ++len) {
      const bool starts = i == 0 || !same_head(me, hme, up, hup, len);
      const bool ends = i + 1 == n_sa || !same_head(me, hme, dn, hdn, len);
      if (!starts && !ends) continue;
      bool long_enough = true;
      if (min_run > 1) {
        long_enough = false;                     // a run of one is shorter than any minimum above one
        if (!(starts && ends)) {
          const int64_t f = starts ? i + min_run - 1 : i - min_run + 1;
          long_enough = f >= 0 && f < n_sa && head_at(T, sa, n, vocab, f, far, hfar) &&
                        same_head(me, hme, far, hfar, len);
        }
      }
      if (!long_enough) continue;
      const unsigned long long key = rest::index_key(me, len, token_bits);
      unsigned long long* grp = table + (size_t)rest::index_group_of(key, group_mask) * 16;
      for (int e = 0; e < 4; ++e) {
        const unsigned long long cur = atomicCAS(grp + e * 4, rest::kIndexEmptyKey, key);
        if (cur == rest::kIndexEmptyKey || cur == key) {
          if (starts) grp[e * 4 + 1] = (unsigned long long)i;
          if (ends) grp[e * 4 + 2] = (unsigned long long)(i + 1);
          break;
        }
      }
    }
  }
}

// first[t] of a token that never starts a suffix = first[] of the next token that does:
// a suffix minimum from the right, 1024 entries at a time (one block).
__global__ void __launch_bounds__(1024)
index_fill_kernel(long long* __restrict__ first, uint32_t vocab, int64_t n) {
  __shared__ long long buf[1024];
  __shared__ long long carry;
  if (threadIdx.x == 0) { carry = n; first[vocab] = n; }
  __syncthreads();
  for (int64_t top = (int64_t)vocab; top > 0; top -= 1024) {
    const int64_t t = top - 1 - threadIdx.x;          // thread 0 takes the rightmost entry
    long long v = t >= 0 ? first[t] : -1;
    buf[threadIdx.x] = v < 0 ? 0x7FFFFFFFFFFFFFFFll : v;
    __syncthreads();
    for (int o = 1; o < 1024; o <<= 1) {              // inclusive minimum over threads 0 .. x
      long long u = threadIdx.x >= o ? buf[threadIdx.x - o] : 0x7FFFFFFFFFFFFFFFll;
      __syncthreads();
      if (u < buf[threadIdx.x]) buf[threadIdx.x] = u;
      __syncthreads();
    }
    const long long c = carry;
    const long long r = buf[threadIdx.x] < c ? buf[threadIdx.x] : c;
    if (t >= 0) first[t] = r;
    __syncthreads();
    if (threadIdx.x == 1023) carry = r;
    __syncthreads();
  }
}

}  // namespace

extern "C" size_t rest_datastore_aux_bytes(uint64_t n_tokens, int32_t, uint32_t vocab) {
  return index_layout(n_tokens, vocab).total + validation_bytes(n_tokens);
}

extern "C" rest_status rest_datastore_create(const int32_t* d_tokens, uint64_t n_tokens,
                                             const void* d_sa, int32_t sa_bytes, uint32_t vocab,
                                             uint32_t flags, void* d_aux, size_t aux_bytes,
                                             void* stream, rest_datastore** out) {
  return rest_datastore_create_shard(d_tokens, n_tokens, d_sa, n_tokens, sa_bytes, vocab, flags, d_aux,
                                     aux_bytes, stream, out);
}

extern "C" rest_status rest_datastore_create_shard(const int32_t* d_tokens, uint64_t n_tokens,
                                                   const void* d_sa, uint64_t n_sa, int32_t sa_bytes,
                                                   uint32_t vocab, uint32_t flags, void* d_aux,
                                                   size_t aux_bytes, void* stream, rest_datastore** out) {
  if (!out) return REST_INVALID_ARG;
  *out = nullptr;
  if (!d_tokens || !d_sa || n_tokens == 0 || n_sa == 0 || n_sa > n_tokens || vocab == 0 ||
      vocab >= 0x80000000u)
    return REST_INVALID_ARG;
  if (sa_bytes != 4 && sa_bytes != 8) return REST_INVALID_ARG;
  if (sa_bytes == 4 && n_tokens > 0x7FFFFFFFull) return REST_INVALID_ARG;
  if (n_tokens > (1ull << 40)) return REST_UNSUPPORTED;
  if (flags & ~(REST_DS_VALIDATE | REST_DS_INDEX)) return REST_INVALID_ARG;
  const IndexLayout il = (flags & REST_DS_INDEX) ? index_layout(n_tokens, vocab) : IndexLayout{};
  const size_t aux_need = il.total + ((flags & REST_DS_VALIDATE) ? validation_bytes(n_tokens) : 0);
  if (aux_need > 0) {
    if (!d_aux || (reinterpret_cast<uintptr_t>(d_aux) & 255)) return REST_INVALID_ARG;
    if (aux_bytes < aux_need) return REST_WORKSPACE_TOO_SMALL;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (flags & REST_DS_VALIDATE) {
    const size_t need = validation_bytes(n_tokens);
    uint32_t* d_flags = reinterpret_cast<uint32_t*>(static_cast<unsigned char*>(d_aux) + il.total);
    uint32_t* d_seen = d_flags + 64;
    REST_CUDA_TRY(cudaMemsetAsync(d_flags, 0, need, st));
    const uint64_t wave = (uint64_t)(rest::sm_count() > 0 ? rest::sm_count() : 148) * 16;
    int blocks = (int)((n_tokens + 255) / 256 < wave ? (n_tokens + 255) / 256 : wave);
    if (sa_bytes == 4)
      validate_kernel<int32_t><<<blocks, 256, 0, st>>>(d_tokens, static_cast<const int32_t*>(d_sa),
                                                       (int64_t)n_tokens, (int64_t)n_sa, vocab, d_seen, d_flags);
    else
      validate_kernel<int64_t><<<blocks, 256, 0, st>>>(d_tokens, static_cast<const int64_t*>(d_sa),
                                                       (int64_t)n_tokens, (int64_t)n_sa, vocab, d_seen, d_flags);
    rest::count_launch();
    REST_CUDA_TRY(cudaGetLastError());
    uint32_t h_flags = 0;
    REST_CUDA_TRY(cudaMemcpyAsync(&h_flags, d_flags, sizeof(h_flags), cudaMemcpyDeviceToHost, st));
    REST_CUDA_TRY(cudaStreamSynchronize(st));
    if (h_flags != 0) return REST_BAD_DATASTORE;
  }
  rest::BucketIndex idx = {nullptr, nullptr, 0, nullptr, 0, 0};
  if (il.entries > 0) {
    // built after a successful validation (when asked for), on the same stream, without a sync:
    // calls that use the handle on this stream see the finished index
    unsigned char* base = static_cast<unsigned char*>(d_aux);
    uint32_t* unusable = reinterpret_cast<uint32_t*>(base);
    long long* first = reinterpret_cast<long long*>(base + kIndexHeaderBytes);
    unsigned long long* table = reinterpret_cast<unsigned long long*>(base + kIndexHeaderBytes + il.first_bytes);
    REST_CUDA_TRY(cudaMemsetAsync(base, 0xFF, il.total, st));      // first[] = -1, keys = empty, lo = hi = -1
    REST_CUDA_TRY(cudaMemsetAsync(base, 0, kIndexHeaderBytes, st));
    const uint32_t group_mask = (uint32_t)(il.entries / 4 - 1);
    const uint64_t wave = (uint64_t)(rest::sm_count() > 0 ? rest::sm_count() : 148) * 16;
    const int blocks = (int)((n_sa + 255) / 256 < wave ? (n_sa + 255) / 256 : wave);
    if (sa_bytes == 4)
      index_build_kernel<int32_t><<<blocks, 256, 0, st>>>(d_tokens, static_cast<const int32_t*>(d_sa),
                                                          (int64_t)n_tokens, (int64_t)n_sa, vocab, il.min_run, il.levels, il.token_bits, first, table, group_mask, unusable);
    else
      index_build_kernel<int64_t><<<blocks, 256, 0, st>>>(d_tokens, static_cast<const int64_t*>(d_sa),
                                                          (int64_t)n_tokens, (int64_t)n_sa, vocab, il.min_run, il.levels, il.token_bits, first, table, group_mask, unusable);
    index_fill_kernel<<<1, 1024, 0, st>>>(first, vocab, (int64_t)n_sa);
    rest::count_launch(2);
    REST_CUDA_TRY(cudaGetLastError());
    idx.first = first; idx.table = table; idx.group_mask = group_mask; idx.unusable = unusable;
    idx.levels = il.levels; idx.token_bits = il.token_bits;
  }
  rest_datastore* ds = static_cast<rest_datastore*>(malloc(sizeof(rest_datastore)));
  if (!ds) return REST_INVALID_ARG;
  ds->v.idx = idx;
  ds->v.tokens = d_tokens;
  ds->v.sa = d_sa;
  ds->v.n_tokens = (int64_t)n_tokens;
  ds->v.n_sa = (int64_t)n_sa;
  ds->v.sa_bytes = sa_bytes;
  ds->v.vocab = vocab;
  *out = ds;
  return REST_OK;
}

extern "C" void rest_datastore_destroy(rest_datastore* ds) { free(ds); }

extern "C" const char* rest_status_string(rest_status s) {
  switch (s) {
    case REST_OK: return "ok";
    case REST_INVALID_ARG: return "invalid argument";
    case REST_UNSUPPORTED: return "unsupported size or parameter";
    case REST_WORKSPACE_TOO_SMALL: return "workspace too small";
    case REST_CUDA_ERROR: return "CUDA runtime error";
    case REST_BAD_DATASTORE: return "datastore failed validation";
    default: return "unknown status";
  }
}

extern "C" const char* rest_last_cuda_error(void) { return rest::g_err; }
extern "C" uint64_t rest_launch_count(void) { return rest::g_launches.load(); }
