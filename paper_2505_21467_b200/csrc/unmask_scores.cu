// dlm_unmask_select_scored: top-k unmasking ranked by one of several per-position scores computed
// in the same pass over the vocabulary (Sec. 3.1 names a MaskGIT-style, an entropy-based and a Top-K
// margin sampler beside plain confidence; the formulas are the readings given in include/dlm.h).
//
// Same shape as the confidence kernel: only the logit rows of masked positions are read, once, as
// 16-byte vectors; a row is cut into chunks, one block per (chunk, row); every thread keeps running
// statistics of its share
//     m   maximum            idx  lowest index attaining it       m2  second largest entry
//     s   sum exp(z - m)     t    sum (z - m) exp(z - m)
// which the block, and then one warp per row over the row's chunks, combine with fixed trees (so the
// result does not depend on block scheduling).  From them: conf = 1/s, negative entropy = t/s - ln s,
// margin = (1 - exp(m2 - m)) / s.  The last block of a batch element ranks its positions.
#include <math_constants.h>

#include "common.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kU = 4;                          // 16-byte vectors in flight per thread
constexpr int kStep = kThreads * 4 * kU;       // logits per block iteration
constexpr int kMaxBlockLen = 1024;

struct Stats {
  float m;
  int idx;
  float s, t, m2;
  int pad[3];
};

struct ScoredArgs {
  int block_len, k, kind;
  const float* noise;
  uint8_t* masked;
  int32_t* tokens;
  int32_t* tok;
  float* conf;
  float* score;
  float* zmax;
  int32_t* sel_idx;
  int32_t* n_sel;
};

__device__ __forceinline__ Stats empty_stats() {
  Stats e;
  e.m = -CUDART_INF_F; e.idx = 0x7fffffff; e.s = 0.f; e.t = 0.f; e.m2 = -CUDART_INF_F;
  e.pad[0] = e.pad[1] = e.pad[2] = 0;
  return e;
}

// Statistics of the union of two disjoint sets of entries.
__device__ __forceinline__ Stats combine(const Stats& a, const Stats& b) {
  Stats r;
  const bool a_first = a.m > b.m || (a.m == b.m && a.idx < b.idx);
  r.m = a_first ? a.m : b.m;
  r.idx = a_first ? a.idx : b.idx;
  r.m2 = a.m >= b.m ? fmaxf(a.m2, b.m) : fmaxf(b.m2, a.m);
  // re-base both sides on the common maximum; a side that saw nothing finite contributes nothing
  const float da = a.m - r.m, db = b.m - r.m;
  const float fa = a.m > -CUDART_INF_F ? __expf(da) : 0.f, fb = b.m > -CUDART_INF_F ? __expf(db) : 0.f;
  r.s = fa * a.s + fb * b.s;
  r.t = (fa > 0.f ? fa * fmaf(da, a.s, a.t) : 0.f) + (fb > 0.f ? fb * fmaf(db, b.s, b.t) : 0.f);
  r.pad[0] = r.pad[1] = r.pad[2] = 0;
  return r;
}

__device__ __forceinline__ Stats shuffle_xor(const Stats& v, int o) {
  Stats r;
  r.m = __shfl_xor_sync(0xffffffffu, v.m, o);
  r.idx = __shfl_xor_sync(0xffffffffu, v.idx, o);
  r.s = __shfl_xor_sync(0xffffffffu, v.s, o);
  r.t = __shfl_xor_sync(0xffffffffu, v.t, o);
  r.m2 = __shfl_xor_sync(0xffffffffu, v.m2, o);
  r.pad[0] = r.pad[1] = r.pad[2] = 0;
  return r;
}

// The tree keeps the lower lane's operand on the left, so ties on the maximum resolve by index as
// combine() prescribes and every lane ends with the same result.
__device__ __forceinline__ Stats warp_combine(Stats v, int lane) {
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const Stats w = shuffle_xor(v, o);
    v = (lane & o) ? combine(w, v) : combine(v, w);
  }
  return v;
}

__device__ __forceinline__ void reduce_chunk(const float* __restrict__ logits, int vocab, int chunk_len, int n_chunks,
                                             Stats* partial, int row) {
  const int chunk = blockIdx.x, tid = threadIdx.x;
  const float* z = logits + (size_t)row * vocab;
  const int begin = chunk * chunk_len;
  const int end = min(begin + chunk_len, vocab);
  Stats st = empty_stats();
  const bool vec_ok = (((uintptr_t)(z + begin)) & 15) == 0;
  for (int base = begin; base < end; base += kStep) {
    float x[kU * 4];
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      const int e = base + (u * kThreads + tid) * 4;
      if (vec_ok && e + 3 < end) {
        const float4 v = __ldcs(reinterpret_cast<const float4*>(z + e));
        x[4 * u + 0] = v.x; x[4 * u + 1] = v.y; x[4 * u + 2] = v.z; x[4 * u + 3] = v.w;
      } else {
#pragma unroll
        for (int c = 0; c < 4; ++c) x[4 * u + c] = (e + c < end) ? z[e + c] : -CUDART_INF_F;
      }
    }
    // the two largest entries seen so far and the lowest index of the largest (indices ascend within a thread)
    float m_new = st.m;
#pragma unroll
    for (int u = 0; u < kU; ++u)
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const float v = x[4 * u + c];
        const int e = base + (u * kThreads + tid) * 4 + c;
        if (v > m_new) { st.m2 = m_new; m_new = v; st.idx = e; }
        else if (e < end && v > st.m2) st.m2 = v;
      }
    if (m_new > st.m) {   // the running sums follow the running maximum
      const float d = st.m - m_new;
      const float f = st.m > -CUDART_INF_F ? __expf(d) : 0.f;
      st.t = f > 0.f ? f * fmaf(d, st.s, st.t) : 0.f;
      st.s *= f;
      st.m = m_new;
    }
    if (st.m > -CUDART_INF_F) {
#pragma unroll
      for (int j = 0; j < kU * 4; ++j) {
        const float d = x[j] - st.m;
        const float e = __expf(d);
        st.s += e;
        if (e > 0.f) st.t = fmaf(d, e, st.t);
      }
    }
  }
  const int warp = tid >> 5, lane = tid & 31;
  st = warp_combine(st, lane);
  __shared__ Stats sm[kThreads / 32];
  if (lane == 0) sm[warp] = st;
  __syncthreads();
  if (tid == 0) {
    Stats tot = sm[0];
#pragma unroll
    for (int w = 1; w < kThreads / 32; ++w) tot = combine(tot, sm[w]);
    int4* dst = reinterpret_cast<int4*>(partial + (size_t)row * n_chunks + chunk);
    __stcg(dst, make_int4(__float_as_int(tot.m), tot.idx, __float_as_int(tot.s), __float_as_int(tot.t)));
    __stcg(dst + 1, make_int4(__float_as_int(tot.m2), 0, 0, 0));
  }
}

__device__ __forceinline__ Stats load_stats(const Stats* p) {
  const int4 a = __ldcg(reinterpret_cast<const int4*>(p)), b = __ldcg(reinterpret_cast<const int4*>(p) + 1);
  Stats r;
  r.m = __int_as_float(a.x); r.idx = a.y; r.s = __int_as_float(a.z); r.t = __int_as_float(a.w); r.m2 = __int_as_float(b.x);
  r.pad[0] = r.pad[1] = r.pad[2] = 0;
  return r;
}

// Scores and selection for batch element b by the whole block.
__device__ void select_batch(const Stats* partial, int n_chunks, int b, const ScoredArgs& a) {
  __shared__ float s_score[kMaxBlockLen];
  __shared__ int32_t s_tok[kMaxBlockLen];
  __shared__ uint8_t s_on[kMaxBlockLen];
  __shared__ uint8_t s_sel[kMaxBlockLen];
  __shared__ int s_count;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, n_warps = blockDim.x >> 5;
  const int L = a.block_len, k = a.k;
  const size_t p0 = (size_t)b * L;
  if (tid == 0) s_count = 0;
  for (int i = warp; i < L; i += n_warps) {
    const bool on = a.masked[p0 + i] != 0;   // uniform across the warp
    int tok = -1;
    float conf = -1.f, score = 0.f, zmax = 0.f;
    if (on) {
      Stats st = empty_stats();
      for (int c = lane; c < n_chunks; c += 32) st = combine(st, load_stats(partial + (p0 + i) * n_chunks + c));
      st = warp_combine(st, lane);
      tok = st.idx;
      zmax = st.m;
      conf = 1.0f / st.s;
      const float ln_s = __logf(st.s);
      if (a.kind == DLM_SCORE_CONFIDENCE) score = conf;
      else if (a.kind == DLM_SCORE_NEG_ENTROPY) score = st.t / st.s - ln_s;
      else if (a.kind == DLM_SCORE_MARGIN) score = (1.0f - (st.m2 > -CUDART_INF_F ? __expf(st.m2 - st.m) : 0.f)) / st.s;
      else score = a.noise[p0 + i] - ln_s;
    }
    if (lane == 0) {
      a.tok[p0 + i] = tok;
      a.conf[p0 + i] = conf;
      a.score[p0 + i] = score;
      a.zmax[p0 + i] = zmax;
      s_score[i] = score;
      s_tok[i] = tok;
      s_on[i] = on ? 1 : 0;
      s_sel[i] = 0;
    }
  }
  if (k <= 0) return;
  __syncthreads();
  // rank among the masked positions of this batch element: (score desc, position asc)
  for (int i = tid; i < L; i += blockDim.x) {
    if (!s_on[i]) continue;
    const float mine = s_score[i];
    int rank = 0;
    for (int j = 0; j < L; ++j) {
      if (!s_on[j]) continue;
      const float sj = s_score[j];
      rank += (sj > mine || (sj == mine && j < i)) ? 1 : 0;
    }
    if (rank < k) {
      s_sel[i] = 1;
      atomicAdd(&s_count, 1);
    }
  }
  __syncthreads();
  for (int i = tid; i < L; i += blockDim.x) {
    if (!s_sel[i]) continue;
    int order = 0;
    for (int j = 0; j < i; ++j) order += s_sel[j];
    a.sel_idx[(size_t)b * k + order] = i;
    a.tokens[p0 + i] = s_tok[i];
    a.masked[p0 + i] = 0;
  }
  const int count = s_count;
  for (int j = count + tid; j < k; j += blockDim.x) a.sel_idx[(size_t)b * k + j] = -1;
  if (tid == 0) a.n_sel[b] = count;
}

__global__ void __launch_bounds__(kThreads)
vocab_stats_kernel(const float* __restrict__ logits, int vocab, int chunk_len, int n_chunks, Stats* partial,
                   unsigned int* tickets, const ScoredArgs sel) {
  dlm_grid_dependency_wait();
  dlm_trigger_dependents();
  const int row = blockIdx.y;
  if (sel.masked[row]) reduce_chunk(logits, vocab, chunk_len, n_chunks, partial, row);
  if (tickets == nullptr) return;
  __shared__ bool is_last;
  const int b = row / sel.block_len;
  if (threadIdx.x == 0) {   // thread 0 wrote this block's statistics: its release-acquire increment publishes them
    unsigned int t;
    asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(t) : "l"(tickets + b) : "memory");
    is_last = (t == (unsigned int)(n_chunks * sel.block_len) - 1u);
    if (is_last) tickets[b] = 0;
  }
  __syncthreads();
  if (!is_last) return;
  select_batch(partial, n_chunks, b, sel);
}

__global__ void __launch_bounds__(kThreads)
scored_select_kernel(const Stats* partial, int n_chunks, const ScoredArgs sel) {
  dlm_grid_dependency_wait();
  dlm_trigger_dependents();
  select_batch(partial, n_chunks, blockIdx.x, sel);
}

}  // namespace

extern "C" size_t dlm_unmask_scored_workspace_bytes(const dlm_ctx* ctx, int batch, int block_len, int vocab) {
  (void)ctx;
  if (batch <= 0 || block_len <= 0 || vocab <= 0) return 0;
  const size_t n_chunks = ((size_t)vocab + kStep - 1) / kStep;
  return (size_t)batch * block_len * n_chunks * sizeof(Stats);
}

extern "C" int dlm_unmask_select_scored(dlm_ctx* ctx, const float* logits, int batch, int block_len, int vocab,
                                        uint8_t* masked, int32_t* tokens, int k, int score_kind, const float* noise,
                                        int32_t* tok, float* conf, float* score, float* zmax, int32_t* sel_idx,
                                        int32_t* n_sel, void* workspace, size_t workspace_bytes, void* stream) {
  if (!ctx || !logits || !masked || !tok || !conf || !score || !zmax) return DLM_ERR_NULL;
  if (k > 0 && (!tokens || !sel_idx || !n_sel)) return DLM_ERR_NULL;
  if (batch <= 0 || block_len <= 0 || vocab <= 0 || k < 0) return DLM_ERR_SHAPE;
  if (score_kind < DLM_SCORE_CONFIDENCE || score_kind > DLM_SCORE_LOG_CONF_PLUS_NOISE) return DLM_ERR_SHAPE;
  if (score_kind == DLM_SCORE_LOG_CONF_PLUS_NOISE && !noise) return DLM_ERR_NULL;
  if (block_len > kMaxBlockLen || (long long)batch * block_len > 65535) return DLM_ERR_UNSUPPORTED;
  if (((uintptr_t)logits & 3) != 0) return DLM_ERR_UNSUPPORTED;
  const size_t need = dlm_unmask_scored_workspace_bytes(ctx, batch, block_len, vocab);
  if (!workspace || workspace_bytes < need || ((uintptr_t)workspace & 15)) return DLM_ERR_WORKSPACE;
  DLM_DEVICE_TRY(ctx);
  // chunks of one or two block iterations: two when even then a resident wave (4 blocks per SM) is exceeded
  const long long rows = (long long)batch * block_len;
  const long long one_pass_blocks = rows * ((vocab + kStep - 1) / kStep);
  const int passes = one_pass_blocks > 8LL * ctx->num_sms ? 2 : 1;
  const int chunk_len = kStep * passes;
  const int n_chunks = (vocab + chunk_len - 1) / chunk_len;
  ScoredArgs a;
  a.block_len = block_len; a.k = k; a.kind = score_kind; a.noise = noise; a.masked = masked; a.tokens = tokens;
  a.tok = tok; a.conf = conf; a.score = score; a.zmax = zmax; a.sel_idx = sel_idx; a.n_sel = n_sel;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  unsigned int* tickets = batch <= kDlmUnmaskTickets ? ctx->words->unmask_tickets : nullptr;
  DLM_CUDA_TRY(dlm_launch(vocab_stats_kernel, dim3(n_chunks, (unsigned)rows), dim3(kThreads), 0, s, logits, vocab, chunk_len,
                          n_chunks, static_cast<Stats*>(workspace), tickets, a));
  if (tickets != nullptr) return dlm_launch_ok(ctx, 1);
  DLM_CUDA_TRY(dlm_launch(scored_select_kernel, dim3(batch), dim3(kThreads), 0, s, static_cast<const Stats*>(workspace),
                          n_chunks, a));
  return dlm_launch_ok(ctx, 2);
}
