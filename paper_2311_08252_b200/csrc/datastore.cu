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
                                int64_t n, uint32_t vocab, uint32_t* __restrict__ seen,
                                uint32_t* __restrict__ flags) {
  int64_t stride = (int64_t)gridDim.x * blockDim.x;
  uint32_t bad = 0;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    int32_t t = T[i];
    if (t < 0 || (uint32_t)t >= vocab) bad |= 1u;
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

}  // namespace

extern "C" size_t rest_datastore_aux_bytes(uint64_t n_tokens, int32_t, uint32_t) {
  // one "seen" bit per position, rounded up to 32-bit words, plus one 256-byte block of flags
  return ((n_tokens + 31) / 32) * 4 + 256;
}

extern "C" rest_status rest_datastore_create(const int32_t* d_tokens, uint64_t n_tokens,
                                             const void* d_sa, int32_t sa_bytes, uint32_t vocab,
                                             uint32_t flags, void* d_aux, size_t aux_bytes,
                                             void* stream, rest_datastore** out) {
  if (!out) return REST_INVALID_ARG;
  *out = nullptr;
  if (!d_tokens || !d_sa || n_tokens == 0 || vocab == 0 || vocab >= 0x80000000u)
    return REST_INVALID_ARG;
  if (sa_bytes != 4 && sa_bytes != 8) return REST_INVALID_ARG;
  if (sa_bytes == 4 && n_tokens > 0x7FFFFFFFull) return REST_INVALID_ARG;
  if (n_tokens > (1ull << 40)) return REST_UNSUPPORTED;
  if (flags & REST_DS_VALIDATE) {
    size_t need = rest_datastore_aux_bytes(n_tokens, sa_bytes, vocab);
    if (!d_aux) return REST_INVALID_ARG;
    if (aux_bytes < need) return REST_WORKSPACE_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint32_t* d_flags = static_cast<uint32_t*>(d_aux);
    uint32_t* d_seen = d_flags + 64;
    REST_CUDA_TRY(cudaMemsetAsync(d_aux, 0, need, st));
    const uint64_t wave = (uint64_t)(rest::sm_count() > 0 ? rest::sm_count() : 148) * 16;
    int blocks = (int)((n_tokens + 255) / 256 < wave ? (n_tokens + 255) / 256 : wave);
    if (sa_bytes == 4)
      validate_kernel<int32_t><<<blocks, 256, 0, st>>>(d_tokens, static_cast<const int32_t*>(d_sa),
                                                       (int64_t)n_tokens, vocab, d_seen, d_flags);
    else
      validate_kernel<int64_t><<<blocks, 256, 0, st>>>(d_tokens, static_cast<const int64_t*>(d_sa),
                                                       (int64_t)n_tokens, vocab, d_seen, d_flags);
    rest::count_launch();
    REST_CUDA_TRY(cudaGetLastError());
    uint32_t h_flags = 0;
    REST_CUDA_TRY(cudaMemcpyAsync(&h_flags, d_flags, sizeof(h_flags), cudaMemcpyDeviceToHost, st));
    REST_CUDA_TRY(cudaStreamSynchronize(st));
    if (h_flags != 0) return REST_BAD_DATASTORE;
  }
  rest_datastore* ds = static_cast<rest_datastore*>(malloc(sizeof(rest_datastore)));
  if (!ds) return REST_INVALID_ARG;
  ds->v.tokens = d_tokens;
  ds->v.sa = d_sa;
  ds->v.n_tokens = (int64_t)n_tokens;
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
