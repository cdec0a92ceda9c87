// Shared host-side helpers of the REST CUDA library (error bookkeeping, launch counter).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "rest.h"
#include "rest_aids.h"

namespace rest {

// Records the text of a failed CUDA call for rest_last_cuda_error(); returns REST_CUDA_ERROR.
rest_status note_cuda_error(cudaError_t e, const char* where);
void count_launch(int n = 1);
// Raises a kernel's dynamic shared-memory limit on the current device when `bytes` exceeds
// what was set before (kernel_slot: small per-kernel index used for the per-device cache).
cudaError_t ensure_dynamic_smem(const void* kernel, int kernel_slot, size_t bytes);
// Streaming multiprocessors of the current device (asked once per device); 0 when there is no
// usable device.
int sm_count();
// One slot per kernel instance, library-wide: two kernels on one slot would skip each other's
// attribute call.  The draft kernel's instances take kSmemSlotDraft + 0 ... 19.
constexpr int kSmemSlotDraft = 0, kSmemSlotAttn = 20, kSmemSlotAttnWide = 21, kSmemSlots = 22;

#define REST_CUDA_TRY(expr)                                              \
  do {                                                                   \
    cudaError_t e_ = (expr);                                             \
    if (e_ != cudaSuccess) return ::rest::note_cuda_error(e_, #expr);    \
  } while (0)

// Bucket index over the suffix array (an accelerator built by rest_datastore_create; results
// never depend on it).  `first[t]` is the first suffix-array slot whose suffix starts with token
// t (first[vocab] = n_sa), so suffixes starting with t occupy [first[t], first[t + 1]).
// `table` is a hash table over the frequent token n-grams, n = 2 ... levels: groups of four
// 32-byte entries {key, lo, hi, unused}; an entry says that the suffixes starting with that
// n-gram occupy slots [lo, hi).  n-grams that occur fewer times than a size-dependent minimum
// are not stored: a search for them starts from the range of a shorter prefix instead.
struct BucketIndex {
  const long long* first;               // null: no index
  const unsigned long long* table;      // 4 words per entry
  uint32_t group_mask;                  // number of groups - 1 (a group = 4 entries = 128 bytes)
  const uint32_t* unusable;             // non-zero: the build met an entry or token out of range
  int levels;                           // longest n-gram stored (2 ... 4)
  int token_bits;                       // bits per token in a key
};
constexpr unsigned long long kIndexEmptyKey = ~0ull;
constexpr int kIndexMaxLevel = 4;
// key of an n-gram: n - 1 in the top two bits, the tokens below, first token lowest (n *
// token_bits <= 60, so no key equals the empty marker)
__host__ __device__ inline unsigned long long index_key(const int32_t* tok, int n, int token_bits) {
  unsigned long long key = (unsigned long long)(n - 1) << 62;
  for (int k = 0; k < n; ++k) key |= (unsigned long long)(uint32_t)tok[k] << (k * token_bits);
  return key;
}
__host__ __device__ inline uint32_t index_group_of(unsigned long long key, uint32_t group_mask) {
  key ^= key >> 29;
  key *= 0xBF58476D1CE4E5B9ull;
  key ^= key >> 32;
  key *= 0x94D049BB133111EBull;
  return (uint32_t)(key >> 35) & group_mask;
}

struct DatastoreView {
  const int32_t* tokens;
  const void* sa;
  int64_t n_tokens;
  int64_t n_sa;          // suffix-array entries: n_tokens, or fewer when the array lists only some positions
  int32_t sa_bytes;
  uint32_t vocab;
  BucketIndex idx;
};

}  // namespace rest

struct rest_datastore {
  rest::DatastoreView v;
};
