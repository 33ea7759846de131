// Context management of the DLM FreeCache library: creation, status word, error text.
#include <new>

#include "common.cuh"
#include "sm100_ptx.cuh"

extern "C" int dlm_create(dlm_ctx** out, int device) {
  if (!out) return DLM_ERR_NULL;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return DLM_ERR_CUDA;
  cudaDeviceProp prop;
  DLM_CUDA_TRY(cudaGetDeviceProperties(&prop, device));
  if (prop.major != 10) return DLM_ERR_UNSUPPORTED;  // the kernels are sm_100a only
  int prev = 0;
  DLM_CUDA_TRY(cudaGetDevice(&prev));
  DLM_CUDA_TRY(cudaSetDevice(device));
  dlm_ctx* ctx = new (std::nothrow) dlm_ctx();
  if (!ctx) return DLM_ERR_CUDA;
  ctx->device = device;
  ctx->num_sms = prop.multiProcessorCount;
  ctx->max_smem_optin = (int)prop.sharedMemPerBlockOptin;
  ctx->launches = 0;
  ctx->encode_tiled = nullptr;
  ctx->commit_blocks_per_sm[0] = ctx->commit_blocks_per_sm[1] = 0;
  for (int i = 0; i < 8; ++i) ctx->attn_smem_limit[i] = 0;
  ctx->proj_configured = false;
  ctx->wait_limit_ns = sm100::kWaitLimitNs;
  ctx->attn_team_max = 1 << 20;   // no limit beyond the schedule's own
  ctx->attn_team_force = false;
  if (cudaMalloc(&ctx->words, sizeof(dlm_device_words)) != cudaSuccess ||
      cudaMemset(ctx->words, 0, sizeof(dlm_device_words)) != cudaSuccess) {
    delete ctx;
    cudaSetDevice(prev);
    return DLM_ERR_CUDA;
  }
  cudaSetDevice(prev);
  *out = ctx;
  return DLM_OK;
}

extern "C" int dlm_destroy(dlm_ctx* ctx) {
  if (!ctx) return DLM_ERR_NULL;
  cudaFree(ctx->words);
  delete ctx;
  return DLM_OK;
}

extern "C" int dlm_get_status(dlm_ctx* ctx, void* stream) {
  if (!ctx) return DLM_ERR_NULL;
  DLM_DEVICE_TRY(ctx);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int code = 0;
  DLM_CUDA_TRY(cudaMemcpyAsync(&code, &ctx->words->status, sizeof(int), cudaMemcpyDeviceToHost, s));
  DLM_CUDA_TRY(cudaMemsetAsync(&ctx->words->status, 0, sizeof(int), s));
  DLM_CUDA_TRY(cudaStreamSynchronize(s));
  if (code != 0) {
    // a kernel that gave up may have left its ticket words half counted
    DLM_CUDA_TRY(cudaMemsetAsync(ctx->words, 0, sizeof(dlm_device_words), s));
    DLM_CUDA_TRY(cudaStreamSynchronize(s));
  }
  return code;
}

extern "C" int64_t dlm_launch_count(const dlm_ctx* ctx) { return ctx ? ctx->launches : 0; }

extern "C" const char* dlm_strerror(int code) {
  switch (code) {
    case DLM_OK: return "ok";
    case DLM_ERR_NULL: return "a required pointer is NULL";
    case DLM_ERR_SHAPE: return "a size is non-positive or inconsistent";
    case DLM_ERR_UNSUPPORTED: return "configuration not supported";
    case DLM_ERR_CAPACITY: return "cache length or row count exceeds capacity";
    case DLM_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case DLM_ERR_CUDA: return "a CUDA call failed";
    case DLM_ERR_TIMEOUT: return "a bounded device-side wait expired";
    case DLM_ERR_INDEX: return "a row index is out of range";
    case DLM_ERR_DEVICE: return "the current CUDA device is not the context's device";
    default: return "unknown error code";
  }
}

namespace {

// Waits on an mbarrier that nobody will ever arrive at, with the same bounded wait the kernels use.
__global__ void wait_probe_kernel(unsigned long long limit_ns, int* status) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    sm100::mbar_init(sm100::smem_u32(&bar), 1);
    sm100::mbar_fence_init();
    if (!sm100::mbar_wait_limit(sm100::smem_u32(&bar), 0, &abort_flag, limit_ns)) dlm_set_status(status, DLM_ERR_TIMEOUT);
  }
}

}  // namespace

extern "C" int dlm_selftest_set_wait_limit(dlm_ctx* ctx, uint64_t limit_ns) {
  if (!ctx) return DLM_ERR_NULL;
  if (limit_ns > sm100::kWaitLimitNs) return DLM_ERR_SHAPE;
  if (limit_ns != 0 && limit_ns != sm100::kWaitLimitNs) return DLM_ERR_UNSUPPORTED;   // the two compiled-in limits
  ctx->wait_limit_ns = limit_ns;
  return DLM_OK;
}

extern "C" int dlm_selftest_set_attn_team_max(dlm_ctx* ctx, int max_blocks, int force) {
  if (!ctx) return DLM_ERR_NULL;
  if (max_blocks < 1 || (force != 0 && force != 1)) return DLM_ERR_SHAPE;
  ctx->attn_team_max = max_blocks;
  ctx->attn_team_force = force != 0;
  return DLM_OK;
}

extern "C" int dlm_selftest_wait_timeout(dlm_ctx* ctx, uint64_t limit_ns, void* stream) {
  if (!ctx) return DLM_ERR_NULL;
  if (limit_ns == 0 || limit_ns > 1000000000ull) return DLM_ERR_SHAPE;   // at most one second
  DLM_DEVICE_TRY(ctx);
  wait_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(limit_ns, &ctx->words->status);
  return dlm_launch_ok(ctx, 1);
}
