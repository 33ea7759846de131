// dlm_freecache_attn_step: attention of the active window over [cache rows ; fresh rows]
// (Sec. 3.2.1 "Windowed Re-computation"; Table 1 rows QK^T and Attention Score x Value).
//
// First correct version: one warp per query row, lanes split head_dim, keys visited one by
// one with an online softmax in fp32.  No tensor cores yet.
#include <cuda_bf16.h>
#include <math_constants.h>

#include "common.cuh"

namespace {

template <int D>
__global__ void __launch_bounds__(128)
attn_step_rowwarp_kernel(const __nv_bfloat16* __restrict__ cache_k, const __nv_bfloat16* __restrict__ cache_v,
                         const int32_t* __restrict__ cache_len, const int32_t* __restrict__ q_len,
                         const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k_new,
                         const __nv_bfloat16* __restrict__ v_new, __nv_bfloat16* __restrict__ out,
                         float* __restrict__ lse, int layer_begin, int batch, int n_q_heads, int n_kv_heads,
                         int capacity, int q_cap, float scale, int* status) {
  constexpr int E = D / 32;  // elements per lane
  const int lane = threadIdx.x & 31;
  const int i = blockIdx.y * 4 + (threadIdx.x >> 5);
  if (i >= q_cap) return;
  const int h = blockIdx.x % n_q_heads;
  const int b = (blockIdx.x / n_q_heads) % batch;
  const int lc = blockIdx.x / (n_q_heads * batch);
  const int kvh = h / (n_q_heads / n_kv_heads);
  int Lc = cache_len[b];
  int Lq = q_len ? q_len[b] : q_cap;
  if (Lc < 0 || Lc > capacity || Lq < 0 || Lq > q_cap) {
    if (lane == 0) dlm_set_status(status, DLM_ERR_CAPACITY);
    Lc = max(0, min(Lc, capacity));
    Lq = max(0, min(Lq, q_cap));
  }
  const size_t qrow = (((size_t)lc * batch + b) * n_q_heads + h) * q_cap + i;
  __nv_bfloat16* o = out + qrow * D + lane * E;
  if (i >= Lq) {
#pragma unroll
    for (int e = 0; e < E; ++e) o[e] = __float2bfloat16(0.f);
    if (lse && lane == 0) lse[qrow] = -CUDART_INF_F;
    return;
  }
  float qv[E], acc[E];
#pragma unroll
  for (int e = 0; e < E; ++e) {
    qv[e] = __bfloat162float(q[qrow * D + lane * E + e]) * scale;
    acc[e] = 0.f;
  }
  const __nv_bfloat16* Kc = cache_k + ((((size_t)(lc + layer_begin) * batch + b) * n_kv_heads + kvh) * capacity) * D;
  const __nv_bfloat16* Vc = cache_v + ((((size_t)(lc + layer_begin) * batch + b) * n_kv_heads + kvh) * capacity) * D;
  const __nv_bfloat16* Kn = k_new + ((((size_t)lc * batch + b) * n_kv_heads + kvh) * q_cap) * D;
  const __nv_bfloat16* Vn = v_new + ((((size_t)lc * batch + b) * n_kv_heads + kvh) * q_cap) * D;
  float m = -CUDART_INF_F, l = 0.f;
  for (int j = 0; j < Lc + Lq; ++j) {
    const __nv_bfloat16* kj = (j < Lc ? Kc + (size_t)j * D : Kn + (size_t)(j - Lc) * D) + lane * E;
    const __nv_bfloat16* vj = (j < Lc ? Vc + (size_t)j * D : Vn + (size_t)(j - Lc) * D) + lane * E;
    float s = 0.f;
#pragma unroll
    for (int e = 0; e < E; ++e) s += qv[e] * __bfloat162float(kj[e]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
    const float m_new = fmaxf(m, s);
    const float corr = __expf(m - m_new);
    const float p = __expf(s - m_new);
    l = l * corr + p;
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = acc[e] * corr + p * __bfloat162float(vj[e]);
    m = m_new;
  }
  const float inv = 1.f / l;
#pragma unroll
  for (int e = 0; e < E; ++e) o[e] = __float2bfloat16(acc[e] * inv);
  if (lse && lane == 0) lse[qrow] = m + __logf(l);
}

}  // namespace

extern "C" size_t dlm_attn_workspace_bytes(const dlm_ctx* ctx, const dlm_kv_cache* cache, int n_layers_in_call,
                                           int n_q_heads, int q_cap) {
  if (!ctx || !cache || n_layers_in_call <= 0 || n_q_heads <= 0 || q_cap <= 0 || cache->n_kv_heads <= 0) return 0;
  return 256;
}

extern "C" int dlm_freecache_attn_step(dlm_ctx* ctx, const dlm_kv_cache* cache, int layer_begin, int layer_end,
                                       const void* q, const void* k_new, const void* v_new, int n_q_heads,
                                       int q_cap, const int32_t* q_len, float softmax_scale, int cache_len_hint,
                                       void* out, float* lse, void* workspace, size_t workspace_bytes,
                                       void* stream) {
  (void)cache_len_hint;
  if (!ctx || !cache || !cache->k || !cache->v || !cache->cache_len || !q || !k_new || !v_new || !out)
    return DLM_ERR_NULL;
  if (cache->n_layers <= 0 || cache->batch <= 0 || cache->n_kv_heads <= 0 || cache->capacity <= 0 ||
      n_q_heads <= 0 || q_cap <= 0)
    return DLM_ERR_SHAPE;
  if (layer_begin < 0 || layer_end > cache->n_layers || layer_begin >= layer_end) return DLM_ERR_SHAPE;
  if (cache->head_dim != 64 && cache->head_dim != 128) return DLM_ERR_UNSUPPORTED;
  if (n_q_heads % cache->n_kv_heads != 0) return DLM_ERR_UNSUPPORTED;
  if ((n_q_heads / cache->n_kv_heads) * (long long)q_cap > 256) return DLM_ERR_UNSUPPORTED;
  const size_t need = dlm_attn_workspace_bytes(ctx, cache, layer_end - layer_begin, n_q_heads, q_cap);
  if (!workspace || workspace_bytes < need || ((uintptr_t)workspace & 255)) return DLM_ERR_WORKSPACE;
  const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)cache->head_dim);
  const int nl = layer_end - layer_begin;
  dim3 grid((unsigned)(nl * cache->batch * n_q_heads), (unsigned)((q_cap + 3) / 4));
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  auto k = cache->head_dim == 128 ? attn_step_rowwarp_kernel<128> : attn_step_rowwarp_kernel<64>;
  k<<<grid, 128, 0, s>>>(static_cast<const __nv_bfloat16*>(cache->k), static_cast<const __nv_bfloat16*>(cache->v),
                         cache->cache_len, q_len, static_cast<const __nv_bfloat16*>(q),
                         static_cast<const __nv_bfloat16*>(k_new), static_cast<const __nv_bfloat16*>(v_new),
                         static_cast<__nv_bfloat16*>(out), lse, layer_begin, cache->batch, n_q_heads,
                         cache->n_kv_heads, cache->capacity, q_cap, scale, &ctx->words->status);
  return dlm_launch_ok(ctx, 1);
}
