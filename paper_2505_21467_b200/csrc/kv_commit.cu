// dlm_kv_cache_commit: row gather/scatter of fresh K/V into the device-resident cache
// (Sec. 3.2.1: saving K/V at initialisation, freezing a finished block).
//
// Pure data movement, bound by HBM.  One work item is one 16-byte vector of one K row and
// the matching vector of the V row; items are ordered [layer][batch][head][row][vector] so
// that consecutive threads touch consecutive addresses whenever the row indices are
// consecutive (refresh / append).  The item list is cut into equal contiguous ranges, one per
// block, and the grid is one resident wave, so every SM moves the same number of bytes; a
// thread keeps kUnroll independent 16-byte loads of K and of V in flight.  Item numbers are
// decoded with 32-bit arithmetic whenever the call has fewer than 2^31 items (64-bit divisions
// by run-time divisors cost more than the copy).  The last block to finish advances cache_len.
#include "common.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kUnroll = 4;

struct CommitParams {
  uint4* cache_k;
  uint4* cache_v;
  int32_t* cache_len;
  const uint4* k_new;
  const uint4* v_new;
  const int32_t* src_idx;
  const int32_t* dst_pos;
  const int32_t* n_rows;
  int n_max, src_len, advance_len, layer_begin, n_layers_call, dst_mode;
  int batch, n_kv_heads, capacity;
  int vec_per_row;       // head_dim * 2 / 16
  int vec_shift;         // log2(vec_per_row) or -1
  long long n_items;     // n_layers_call * batch * heads * n_max * vec_per_row
  long long per_block;   // items per block (a multiple of 32)
  int* status;
  unsigned int* ticket;
};

// n(b), validated; -1 if this batch element must be skipped entirely.
__device__ __forceinline__ int valid_rows(const CommitParams& p, int b, int len0) {
  const int n = p.n_rows ? p.n_rows[b] : p.n_max;
  if (n < 0 || n > p.n_max) return -1;
  const bool append = p.dst_pos == nullptr && p.dst_mode == DLM_DST_APPEND;
  if ((append || p.advance_len) && (len0 < 0 || (long long)len0 + n > p.capacity)) return -1;
  return n;
}

template <typename Idx>
__global__ void __launch_bounds__(kThreads, 4) kv_commit_kernel(const CommitParams p) {
  dlm_grid_dependency_wait();
  dlm_trigger_dependents();
  const Idx begin = (Idx)blockIdx.x * (Idx)p.per_block;
  const Idx end = (Idx)min((long long)begin + p.per_block, p.n_items);
  const Idx n_max = (Idx)p.n_max, heads = (Idx)p.n_kv_heads, batch = (Idx)p.batch;
  for (Idx base = begin + threadIdx.x; base < end; base += kThreads * kUnroll) {
    uint4 kk[kUnroll], vv[kUnroll];
    long long to[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      to[u] = -1;
      const Idx item = base + (Idx)(u * kThreads);
      if (item >= end) continue;
      int vec;
      Idx rest;
      if (p.vec_shift >= 0) {
        vec = (int)(item & (Idx)(p.vec_per_row - 1));
        rest = item >> p.vec_shift;
      } else {
        vec = (int)(item % (Idx)p.vec_per_row);
        rest = item / (Idx)p.vec_per_row;
      }
      const int r = (int)(rest % n_max);
      rest /= n_max;
      const int h = (int)(rest % heads);
      rest /= heads;
      const int b = (int)(rest % batch);
      const int lc = (int)(rest / batch);  // layer within the call
      // the index words are read before the row count is checked (their slots always exist), so the
      // three small loads are in flight together instead of one after the other
      const int len0 = p.cache_len[b];
      const long long src = p.src_idx ? p.src_idx[(long long)b * p.n_max + r] : r;
      const long long dst_given = p.dst_pos ? p.dst_pos[(long long)b * p.n_max + r] : 0;
      const int n = valid_rows(p, b, len0);
      if (n < 0) {
        if (r == 0 && vec == 0 && h == 0 && lc == 0) dlm_set_status(p.status, DLM_ERR_CAPACITY);
        continue;
      }
      if (r >= n) continue;
      const long long dst = p.dst_pos ? dst_given : (long long)len0 + (p.dst_mode == DLM_DST_WINDOW ? src : r);
      if (src < 0 || src >= p.src_len || dst < 0 || dst >= p.capacity) {
        if (vec == 0 && h == 0 && lc == 0) dlm_set_status(p.status, DLM_ERR_INDEX);
        continue;
      }
      const long long from =
          ((((long long)lc * p.batch + b) * p.n_kv_heads + h) * p.src_len + src) * p.vec_per_row + vec;
      to[u] = ((((long long)(lc + p.layer_begin) * p.batch + b) * p.n_kv_heads + h) * p.capacity + dst) *
                  p.vec_per_row + vec;
      kk[u] = __ldcs(p.k_new + from);
      vv[u] = __ldcs(p.v_new + from);
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      if (to[u] >= 0) {
        p.cache_k[to[u]] = kk[u];
        p.cache_v[to[u]] = vv[u];
      }
    }
  }
  if (!p.advance_len) return;
  // Serial tail: the last block to arrive bumps cache_len once every row has been written.
  __shared__ bool is_last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned int t = atomicAdd(p.ticket, 1u);
    is_last = (t == gridDim.x - 1);
  }
  __syncthreads();
  if (!is_last) return;
  for (int b = threadIdx.x; b < p.batch; b += kThreads) {
    const int len0 = p.cache_len[b];
    const int n = valid_rows(p, b, len0);
    if (n > 0) p.cache_len[b] = len0 + n;
  }
  if (threadIdx.x == 0) *p.ticket = 0;
}

}  // namespace

extern "C" int dlm_kv_cache_commit(dlm_ctx* ctx, const dlm_kv_cache* cache, const void* k_new,
                                   const void* v_new, int src_len, const int32_t* src_idx,
                                   const int32_t* dst_pos, int dst_mode, const int32_t* n_rows, int n_max,
                                   int advance_len, int layer_begin, int layer_end, void* stream) {
  if (!ctx || !cache || !cache->k || !cache->v || !cache->cache_len || !k_new || !v_new) return DLM_ERR_NULL;
  if (cache->n_layers <= 0 || cache->batch <= 0 || cache->n_kv_heads <= 0 || cache->capacity <= 0 ||
      cache->head_dim <= 0 || src_len <= 0 || n_max <= 0 || (dst_mode != DLM_DST_APPEND && dst_mode != DLM_DST_WINDOW))
    return DLM_ERR_SHAPE;
  if (layer_begin < 0 || layer_end > cache->n_layers || layer_begin >= layer_end) return DLM_ERR_SHAPE;
  if ((cache->head_dim * 2) % 16 != 0) return DLM_ERR_UNSUPPORTED;
  if (((uintptr_t)cache->k | (uintptr_t)cache->v | (uintptr_t)k_new | (uintptr_t)v_new) & 15) return DLM_ERR_UNSUPPORTED;
  DLM_DEVICE_TRY(ctx);

  CommitParams p;
  p.cache_k = static_cast<uint4*>(cache->k);
  p.cache_v = static_cast<uint4*>(cache->v);
  p.cache_len = cache->cache_len;
  p.k_new = static_cast<const uint4*>(k_new);
  p.v_new = static_cast<const uint4*>(v_new);
  p.src_idx = src_idx;
  p.dst_pos = dst_pos;
  p.n_rows = n_rows;
  p.n_max = n_max;
  p.src_len = src_len;
  p.advance_len = advance_len ? 1 : 0;
  p.dst_mode = dst_mode;
  p.layer_begin = layer_begin;
  p.n_layers_call = layer_end - layer_begin;
  p.batch = cache->batch;
  p.n_kv_heads = cache->n_kv_heads;
  p.capacity = cache->capacity;
  p.vec_per_row = cache->head_dim * 2 / 16;
  p.vec_shift = -1;
  for (int s = 0; s < 16; ++s)
    if ((1 << s) == p.vec_per_row) p.vec_shift = s;
  p.n_items = (long long)p.n_layers_call * p.batch * p.n_kv_heads * n_max * p.vec_per_row;
  p.status = &ctx->words->status;
  p.ticket = &ctx->words->commit_ticket;

  // one resident wave of equal contiguous ranges; small calls get one block per kThreads * kUnroll items
  const bool narrow = p.n_items < (1LL << 31) - (long long)kThreads * kUnroll;
  int& per_sm = ctx->commit_blocks_per_sm[narrow ? 0 : 1];
  if (per_sm <= 0) {
    int n = 0;
    const cudaError_t e = narrow ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kv_commit_kernel<unsigned int>, kThreads, 0)
                                 : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kv_commit_kernel<unsigned long long>, kThreads, 0);
    if (e != cudaSuccess || n <= 0) return DLM_ERR_CUDA;
    per_sm = n;
  }
  const long long per_pass = (long long)kThreads * kUnroll;
  long long blocks = (p.n_items + per_pass - 1) / per_pass;
  const long long max_blocks = (long long)ctx->num_sms * per_sm;
  if (blocks > max_blocks) blocks = max_blocks;
  if (blocks < 1) blocks = 1;
  p.per_block = ((p.n_items + blocks - 1) / blocks + 31) & ~31LL;
  blocks = (p.n_items + p.per_block - 1) / p.per_block;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (narrow)
    DLM_CUDA_TRY(dlm_launch(kv_commit_kernel<unsigned int>, dim3((unsigned)blocks), dim3(kThreads), 0, st, p));
  else
    DLM_CUDA_TRY(dlm_launch(kv_commit_kernel<unsigned long long>, dim3((unsigned)blocks), dim3(kThreads), 0, st, p));
  return dlm_launch_ok(ctx, 1);
}
