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
  int max_smem_optin;       // largest dynamic shared memory a block may opt in to, bytes
  int64_t launches;
  dlm_device_words* words;  // device
  void* encode_tiled;       // cuTensorMapEncodeTiled entry point (driver API), resolved lazily
  int commit_blocks_per_sm[2];  // resident blocks per SM of the two commit kernels (0 = not asked yet)
  unsigned long long wait_limit_ns;   // limit of the kernels' device-side waits (2 s; a test may shorten it)
  bool proj_configured;         // shared-memory opt-in of the projection kernel done on this context's device
  int attn_team_max;            // most blocks the attention call's team schedule may give one unit (1 = schedule off)
  bool attn_team_force;         // tests: take the team schedule wherever it is possible, whatever the cost estimate says
  int attn_smem_limit[8];       // dynamic shared memory the two attention kernels may use on this device (0 = not set up yet)
};

#define DLM_CUDA_TRY(expr)                         \
  do {                                             \
    cudaError_t _e = (expr);                       \
    if (_e != cudaSuccess) return DLM_ERR_CUDA;    \
  } while (0)

// Records the first error seen by any thread of any kernel.
__device__ __forceinline__ void dlm_set_status(int* status, int code) { atomicCAS(status, 0, code); }

// Programmatic dependent launch.  Every kernel of the library is launched with the
// programmatic-stream-serialization attribute, calls dlm_grid_dependency_wait() before it touches
// anything a predecessor in the stream may have written, and lets its own dependents start
// launching early with dlm_trigger_dependents(): block scheduling and the dependents' data-free
// set-up then overlap the predecessor's tail instead of following it.  A dependent's wait still
// returns only when the predecessor grid has completed and its writes are visible, and the
// hardware starts dependents only once every block of the predecessor is running, so nothing is
// reordered.  Predecessors that know nothing of this (any other kernel) simply release their
// dependents when they finish.
__device__ __forceinline__ void dlm_grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void dlm_trigger_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
static inline cudaError_t dlm_launch(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                     Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// The context's device must be the calling thread's current device: launches go to the current
// device, the context's words and the caller's pointers live on the context's.
static inline int dlm_check_device(const dlm_ctx* ctx) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return DLM_ERR_CUDA;
  return dev == ctx->device ? DLM_OK : DLM_ERR_DEVICE;
}
#define DLM_DEVICE_TRY(ctx)                        \
  do {                                             \
    const int _d = dlm_check_device(ctx);          \
    if (_d != DLM_OK) return _d;                   \
  } while (0)

static inline int dlm_launch_ok(dlm_ctx* ctx, int n_kernels) {
  if (cudaGetLastError() != cudaSuccess) return DLM_ERR_CUDA;
  ctx->launches += n_kernels;
  return DLM_OK;
}
