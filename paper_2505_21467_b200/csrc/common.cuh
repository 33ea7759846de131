// Shared host/device declarations of the DLM FreeCache library (internal; the public
// interface is include/dlm.h).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "dlm.h"

// Device words owned by a context.  `status` holds the first data-dependent error code
// (0 = none); the ticket words let the last block of a kernel run a serial tail.
constexpr int kDlmUnmaskTickets = 1024;  // batch elements whose selection can run in the tail of the reduce kernel
constexpr int kDlmMaxSplitUnits = 2048;  // attention units that may be split across blocks in one call
struct dlm_device_words {
  int status;
  unsigned int commit_ticket;
  unsigned int unmask_ticket;
  unsigned int pad[13];
  unsigned int unmask_tickets[kDlmUnmaskTickets];     // blocks of a batch element finished so far
  unsigned int attn_unit_tickets[kDlmMaxSplitUnits];  // pieces of a split unit finished so far
};

struct dlm_ctx {
  int device;
  int num_sms;
  int64_t launches;
  dlm_device_words* words;  // device
  void* encode_tiled;       // cuTensorMapEncodeTiled entry point (driver API), resolved lazily
};

#define DLM_CUDA_TRY(expr)                         \
  do {                                             \
    cudaError_t _e = (expr);                       \
    if (_e != cudaSuccess) return DLM_ERR_CUDA;    \
  } while (0)

// Records the first error seen by any thread of any kernel.
__device__ __forceinline__ void dlm_set_status(int* status, int code) { atomicCAS(status, 0, code); }

static inline int dlm_launch_ok(dlm_ctx* ctx, int n_kernels) {
  if (cudaGetLastError() != cudaSuccess) return DLM_ERR_CUDA;
  ctx->launches += n_kernels;
  return DLM_OK;
}
