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
// attribute call.  The draft kernel's instances take kSmemSlotDraft + 0 ... 13.
constexpr int kSmemSlotDraft = 0, kSmemSlotAttn = 14, kSmemSlotAttnWide = 15, kSmemSlots = 16;

#define REST_CUDA_TRY(expr)                                              \
  do {                                                                   \
    cudaError_t e_ = (expr);                                             \
    if (e_ != cudaSuccess) return ::rest::note_cuda_error(e_, #expr);    \
  } while (0)

struct DatastoreView {
  const int32_t* tokens;
  const void* sa;
  int64_t n_tokens;
  int32_t sa_bytes;
  uint32_t vocab;
};

}  // namespace rest

struct rest_datastore {
  rest::DatastoreView v;
};
