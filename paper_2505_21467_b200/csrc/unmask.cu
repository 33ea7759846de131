// dlm_unmask_select: confidence scoring over the vocabulary and top-k unmasking
// (Eq. 2: one logit row per masked position; Eq. 3: fill with the argmax;
//  M_{t-1} = M_t \ U_t).
//
// Kernel 1 (vocab_reduce) is bound by HBM: only the logit rows of masked positions are read,
// once, as 16-byte vectors.  A row is split into chunks of kChunk logits, one block per
// (chunk, row); the block reduces its chunk to the triple (max, lowest argmax, sum of
// exp(z - max)) with warp shuffles and writes it to the workspace.
// Kernel 2 (unmask_select) runs one block per batch element: it merges the triples of each
// row in chunk order (so the result does not depend on block scheduling and identical rows
// give identical bits), then ranks the masked positions by (confidence desc, position asc).
#include <math_constants.h>

#include "common.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kVecPerThread = 4;
constexpr int kChunk = kThreads * kVecPerThread * 4;  // 4096 logits = 16 KB per block
constexpr int kMaxBlockLen = 1024;

struct Triple {
  float m;      // chunk maximum
  int idx;      // lowest index attaining it
  float s;      // sum over the chunk of exp(z - m)
  int pad;
};

__device__ __forceinline__ void take_better(float& m, int& i, float m2, int i2) {
  if (m2 > m || (m2 == m && i2 < i)) { m = m2; i = i2; }
}

__global__ void __launch_bounds__(kThreads)
vocab_reduce_kernel(const float* __restrict__ logits, const uint8_t* __restrict__ masked, int vocab,
                    int n_chunks, Triple* __restrict__ partial) {
  const int row = blockIdx.y;
  if (!masked[row]) return;
  const int chunk = blockIdx.x;
  const float* z = logits + (size_t)row * vocab;
  const int begin = chunk * kChunk;
  const int end = min(begin + kChunk, vocab);
  const int tid = threadIdx.x;

  float x[kVecPerThread * 4];
  float m = -CUDART_INF_F;
  int mi = 0x7fffffff;
  const bool vec_ok = (((uintptr_t)(z + begin)) & 15) == 0;
  if (vec_ok) {
    // thread t owns vectors t, t + 256, ... of the chunk: ascending indices within a thread
#pragma unroll
    for (int u = 0; u < kVecPerThread; ++u) {
      const int e = begin + (u * kThreads + tid) * 4;
      if (e + 3 < end) {
        const float4 v = __ldcs(reinterpret_cast<const float4*>(z + e));
        x[4 * u + 0] = v.x; x[4 * u + 1] = v.y; x[4 * u + 2] = v.z; x[4 * u + 3] = v.w;
      } else {
#pragma unroll
        for (int c = 0; c < 4; ++c) x[4 * u + c] = (e + c < end) ? z[e + c] : -CUDART_INF_F;
      }
    }
#pragma unroll
    for (int u = 0; u < kVecPerThread; ++u)
#pragma unroll
      for (int c = 0; c < 4; ++c)
        if (x[4 * u + c] > m) { m = x[4 * u + c]; mi = begin + (u * kThreads + tid) * 4 + c; }
  } else {
    // rows whose chunk start is not 16-byte aligned (vocab not a multiple of 4): scalar loads
#pragma unroll
    for (int u = 0; u < kVecPerThread * 4; ++u) {
      const int e = begin + u * kThreads + tid;
      x[u] = (e < end) ? z[e] : -CUDART_INF_F;
      if (x[u] > m) { m = x[u]; mi = e; }
    }
  }
  // block maximum and its lowest index
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, m, o);
    const int i2 = __shfl_xor_sync(0xffffffffu, mi, o);
    take_better(m, mi, m2, i2);
  }
  __shared__ float sm_m[kThreads / 32];
  __shared__ int sm_i[kThreads / 32];
  __shared__ float sm_s[kThreads / 32];
  const int warp = tid >> 5, lane = tid & 31;
  if (lane == 0) { sm_m[warp] = m; sm_i[warp] = mi; }
  __syncthreads();
  float bm = sm_m[0];
  int bi = sm_i[0];
#pragma unroll
  for (int w = 1; w < kThreads / 32; ++w) take_better(bm, bi, sm_m[w], sm_i[w]);
  // sum of exp(z - block max); an all -inf chunk contributes nothing
  float s = 0.f;
  if (bm > -CUDART_INF_F) {
#pragma unroll
    for (int u = 0; u < kVecPerThread * 4; ++u) s += __expf(x[u] - bm);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if (lane == 0) sm_s[warp] = s;
  __syncthreads();
  if (tid == 0) {
    float total = 0.f;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) total += sm_s[w];
    Triple t;
    t.m = bm; t.idx = bi; t.s = total; t.pad = 0;
    partial[(size_t)row * n_chunks + chunk] = t;
  }
}

__global__ void __launch_bounds__(kMaxBlockLen)
unmask_select_kernel(const Triple* __restrict__ partial, int n_chunks, int block_len, int k,
                     uint8_t* __restrict__ masked, int32_t* __restrict__ tokens,
                     int32_t* __restrict__ tok, float* __restrict__ conf,
                     int32_t* __restrict__ sel_idx, int32_t* __restrict__ n_sel) {
  __shared__ float s_conf[kMaxBlockLen];
  __shared__ uint8_t s_sel[kMaxBlockLen];
  __shared__ int s_count;
  const int b = blockIdx.x;
  const int i = threadIdx.x;
  const size_t p = (size_t)b * block_len + i;
  bool is_masked = false;
  int my_tok = -1;
  float my_conf = -1.f;
  if (i < block_len) {
    is_masked = masked[p] != 0;
    if (is_masked) {
      const Triple* t = partial + p * n_chunks;
      float m = -CUDART_INF_F;
      int idx = 0;
      for (int c = 0; c < n_chunks; ++c)
        if (t[c].m > m) { m = t[c].m; idx = t[c].idx; }   // chunks ascend: strict > keeps the lowest index
      float s = 0.f;
      for (int c = 0; c < n_chunks; ++c)
        if (t[c].m > -CUDART_INF_F) s += t[c].s * __expf(t[c].m - m);
      my_tok = idx;
      my_conf = 1.0f / s;
    }
    tok[p] = my_tok;
    conf[p] = my_conf;
    s_conf[i] = my_conf;
    s_sel[i] = 0;
  }
  if (k <= 0) return;
  if (i == 0) s_count = 0;
  __syncthreads();
  // rank among the masked positions of this batch element: (confidence desc, position asc)
  if (is_masked) {
    int rank = 0;
    for (int j = 0; j < block_len; ++j) {
      const float cj = s_conf[j];  // unmasked positions hold -1 < every confidence
      rank += (cj > my_conf || (cj == my_conf && j < i)) ? 1 : 0;
    }
    if (rank < k) {
      s_sel[i] = 1;
      atomicAdd(&s_count, 1);
    }
  }
  __syncthreads();
  if (i < block_len && s_sel[i]) {
    int order = 0;
    for (int j = 0; j < i; ++j) order += s_sel[j];
    sel_idx[(size_t)b * k + order] = i;
    tokens[p] = my_tok;
    masked[p] = 0;
  }
  const int count = s_count;
  for (int j = count + i; j < k; j += blockDim.x) sel_idx[(size_t)b * k + j] = -1;
  if (i == 0) n_sel[b] = count;
}

}  // namespace

extern "C" size_t dlm_unmask_workspace_bytes(const dlm_ctx* ctx, int batch, int block_len, int vocab) {
  (void)ctx;
  if (batch <= 0 || block_len <= 0 || vocab <= 0) return 0;
  const size_t n_chunks = ((size_t)vocab + kChunk - 1) / kChunk;
  return (size_t)batch * block_len * n_chunks * sizeof(Triple);
}

extern "C" int dlm_unmask_select(dlm_ctx* ctx, const float* logits, int batch, int block_len, int vocab,
                                 uint8_t* masked, int32_t* tokens, int k, int32_t* tok, float* conf,
                                 int32_t* sel_idx, int32_t* n_sel, void* workspace,
                                 size_t workspace_bytes, void* stream) {
  if (!ctx || !logits || !masked || !tok || !conf) return DLM_ERR_NULL;
  if (k > 0 && (!tokens || !sel_idx || !n_sel)) return DLM_ERR_NULL;
  if (batch <= 0 || block_len <= 0 || vocab <= 0 || k < 0) return DLM_ERR_SHAPE;
  if (block_len > kMaxBlockLen || (long long)batch * block_len > 65535) return DLM_ERR_UNSUPPORTED;
  if (((uintptr_t)logits & 3) != 0) return DLM_ERR_UNSUPPORTED;
  const size_t need = dlm_unmask_workspace_bytes(ctx, batch, block_len, vocab);
  if (!workspace || workspace_bytes < need || ((uintptr_t)workspace & 15)) return DLM_ERR_WORKSPACE;
  const int n_chunks = (vocab + kChunk - 1) / kChunk;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  Triple* partial = static_cast<Triple*>(workspace);
  vocab_reduce_kernel<<<dim3(n_chunks, batch * block_len), kThreads, 0, s>>>(logits, masked, vocab, n_chunks, partial);
  const int threads = ((block_len + 31) / 32) * 32;
  unmask_select_kernel<<<batch, threads, 0, s>>>(partial, n_chunks, block_len, k, masked, tokens, tok, conf,
                                                 sel_idx, n_sel);
  return dlm_launch_ok(ctx, 2);
}

// ---------------------------------------------------------------------------------------
// dlm_unmask_select_static: the same two kernels with the per-row partial reductions kept in
// a fixed device array that is part of the library image, for callers that cannot allocate
// device memory at all.
namespace {

constexpr int kStaticTriples = 65536;  // 1 MiB: rows x chunks of one call may not exceed this
static __device__ __align__(256) Triple g_static_partial[kStaticTriples];

constexpr int kMaxDevices = 64;
Triple* g_static_partial_addr[kMaxDevices];  // device address of the array, per device (0 = not looked up yet)

}  // namespace

extern "C" int dlm_unmask_select_static(const float* logits, int batch, int block_len, int vocab,
                                        uint8_t* masked, int32_t* tokens, int k, int32_t* tok, float* conf,
                                        int32_t* sel_idx, int32_t* n_sel, void* stream) {
  if (!logits || !masked || !tok || !conf) return DLM_ERR_NULL;
  if (k > 0 && (!tokens || !sel_idx || !n_sel)) return DLM_ERR_NULL;
  if (batch <= 0 || block_len <= 0 || vocab <= 0 || k < 0) return DLM_ERR_SHAPE;
  if (block_len > kMaxBlockLen || (long long)batch * block_len > 65535) return DLM_ERR_UNSUPPORTED;
  if (((uintptr_t)logits & 3) != 0) return DLM_ERR_UNSUPPORTED;
  const int n_chunks = (vocab + kChunk - 1) / kChunk;
  if ((long long)batch * block_len * n_chunks > kStaticTriples) return DLM_ERR_WORKSPACE;
  int device = -1;
  DLM_CUDA_TRY(cudaGetDevice(&device));
  if (device < 0 || device >= kMaxDevices) return DLM_ERR_UNSUPPORTED;
  if (!g_static_partial_addr[device]) {
    // In host code the array's name is only a handle; its address on the current device has to be
    // asked for, once per device.
    Triple* addr = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&addr), g_static_partial) != cudaSuccess || !addr)
      return DLM_ERR_CUDA;
    g_static_partial_addr[device] = addr;
  }
  Triple* partial = g_static_partial_addr[device];
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  vocab_reduce_kernel<<<dim3(n_chunks, batch * block_len), kThreads, 0, s>>>(logits, masked, vocab, n_chunks, partial);
  const int threads = ((block_len + 31) / 32) * 32;
  unmask_select_kernel<<<batch, threads, 0, s>>>(partial, n_chunks, block_len, k, masked, tokens, tok, conf,
                                                 sel_idx, n_sel);
  return cudaGetLastError() == cudaSuccess ? DLM_OK : DLM_ERR_CUDA;
}
