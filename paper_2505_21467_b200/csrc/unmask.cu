// dlm_unmask_select: confidence scoring over the vocabulary and top-k unmasking
// (Eq. 2: one logit row per masked position; Eq. 3: fill with the argmax;
//  M_{t-1} = M_t \ U_t).
//
// vocab_reduce is bound by HBM: only the logit rows of masked positions are read, once, as
// 16-byte vectors.  A row is split into chunks of kChunk logits, one block per (chunk, row); the
// block reduces its chunk to the triple (max, lowest argmax, sum of exp(z - max)) with warp
// shuffles and writes it to the workspace.  The last block of a batch element to finish (a
// ticket counter) then runs the selection for that element in the same launch: one warp per row
// merges the row's triples with a fixed shuffle tree (so the result does not depend on block
// scheduling and identical rows give identical bits), then the masked positions are ranked by
// (confidence desc, position asc).  Without ticket words (more batch elements than the context
// has counters for, or the context-free entry point) the selection runs as a second kernel.
#include <math_constants.h>

#include "common.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kVecPerThread = 4;
constexpr int kChunk = kThreads * kVecPerThread * 4;  // 4096 logits: the unit of the chunk length (and of workspace sizing)
constexpr int kMaxBlockLen = 1024;

struct Triple {
  float m;      // chunk maximum
  int idx;      // lowest index attaining it
  float s;      // sum over the chunk of exp(z - m)
  int pad;
};

struct SelectArgs {
  int block_len, k;
  uint8_t* masked;
  int32_t* tokens;
  int32_t* tok;
  float* conf;
  int32_t* sel_idx;
  int32_t* n_sel;
};

// 2^x, results below 2^-126 flushed to zero
__device__ __forceinline__ float ex2_ftz(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ void take_better(float& m, int& i, float m2, int i2) {
  if (m2 > m || (m2 == m && i2 < i)) { m = m2; i = i2; }
}

// One block reduces chunk blockIdx.x (chunk_len logits) of logit row `row` to a Triple.  Every
// thread streams its share with U independent 16-byte loads in flight and keeps a running
// (max, lowest argmax, sum of exp(z - max)); the block combines them with a fixed tree.
//
// kLazy (blocks that make several passes): the loop tracks only the running maximum and the half pass in which it
// last grew, one instruction per logit instead of three; after the block's maximum is known, the few threads that
// hold it read their 16-byte vectors of that half pass again (L2) and find its first position.  Same maximum and
// same lowest index as the eager form; the sum is taken half pass by half pass (see the pipeline below).
template <int U, bool kLazy>
__device__ __forceinline__ void reduce_chunk(const float* __restrict__ logits, int vocab, int chunk_len, int n_chunks,
                                             Triple* partial, int row) {
  const int chunk = blockIdx.x;
  const float* z = logits + (size_t)row * vocab;
  const int begin = chunk * chunk_len;
  const int end = chunk == n_chunks - 1 ? vocab : begin + chunk_len;   // the last chunk takes the remainder (it may be longer)
  const int tid = threadIdx.x;
  constexpr int kStep = kThreads * 4 * U;    // logits per block iteration

  float m = -CUDART_INF_F, s = 0.f;
  int mi = 0x7fffffff;
  int base_of_max = begin;   // kLazy: the pass in which the running maximum last grew
  const bool vec_ok = (((uintptr_t)(z + begin)) & 15) == 0;
  // thread t owns vectors t, t + 256, ... of a pass: ascending indices within a thread
  auto load_pass = [&](int base, float (&x)[U * 4], bool streaming) {
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int e = base + (u * kThreads + tid) * 4;
      if (vec_ok && e + 3 < end) {
        const float4 v = streaming ? __ldcs(reinterpret_cast<const float4*>(z + e)) : __ldcg(reinterpret_cast<const float4*>(z + e));
        x[4 * u + 0] = v.x; x[4 * u + 1] = v.y; x[4 * u + 2] = v.z; x[4 * u + 3] = v.w;
      } else {
#pragma unroll
        for (int c = 0; c < 4; ++c) x[4 * u + c] = (e + c < end) ? z[e + c] : -CUDART_INF_F;
      }
    }
  };
  int half_of_max = 0;       // kLazy: ... and the half of that pass
  // one half of a pass: vectors u in [h U/2, (h + 1) U/2) of this thread
  auto load_half = [&](int base, int h, float (&x)[U * 2], bool streaming) {
#pragma unroll
    for (int u = 0; u < U / 2; ++u) {
      const int e = base + ((h * (U / 2) + u) * kThreads + tid) * 4;
      if (vec_ok && e + 3 < end) {
        const float4 v = streaming ? __ldcs(reinterpret_cast<const float4*>(z + e)) : __ldcg(reinterpret_cast<const float4*>(z + e));
        x[4 * u + 0] = v.x; x[4 * u + 1] = v.y; x[4 * u + 2] = v.z; x[4 * u + 3] = v.w;
      } else {
#pragma unroll
        for (int c = 0; c < 4; ++c) x[4 * u + c] = (e + c < end) ? z[e + c] : -CUDART_INF_F;
      }
    }
  };
  if (kLazy) {
    // Software pipeline over half passes: while one half's arithmetic runs, the other half's loads (of this pass or
    // the next) are in flight, so a thread always has U/2 to U vectors outstanding.  With whole passes a thread had
    // nothing in flight during its arithmetic, about 40 % of the time.
    float xa[U * 2], xb[U * 2];
    auto process = [&](const float (&x)[U * 2], int base, int h) {
      float bm = m;
#pragma unroll
      for (int u = 0; u < U * 2; ++u) bm = fmaxf(bm, x[u]);   // ignores NaN, as a comparison would
      if (bm > m) {   // the running sum follows the running maximum
        base_of_max = base;
        half_of_max = h;
        s *= __expf(m - bm);
        m = bm;
      }
      if (m > -CUDART_INF_F) {
#pragma unroll
        for (int u = 0; u < U * 2; ++u) s += ex2_ftz((x[u] - m) * 1.4426950408889634f);
      }
    };
    load_half(begin, 0, xa, true);
    load_half(begin, 1, xb, true);
    for (int base = begin; base < end; base += kStep) {
      const bool more = base + kStep < end;
      process(xa, base, 0);
      if (more) load_half(base + kStep, 0, xa, true);
      process(xb, base, 1);
      if (more) load_half(base + kStep, 1, xb, true);
    }
  } else {
    for (int base = begin; base < end; base += kStep) {
      float x[U * 4];
      load_pass(base, x, true);
      float bm = m;
#pragma unroll
      for (int u = 0; u < U; ++u)
#pragma unroll
        for (int c = 0; c < 4; ++c)
          if (x[4 * u + c] > bm) { bm = x[4 * u + c]; mi = base + (u * kThreads + tid) * 4 + c; }
      if (bm > m) {   // the running sum follows the running maximum
        s *= __expf(m - bm);
        m = bm;
      }
      if (m > -CUDART_INF_F) {
        // exp(x - m) as 2^((x - m) log2(e)) with the flush-to-zero SFU instruction: the library exponential spends
        // three more instructions per logit on denormal results, and the loop is bound by instruction issue
#pragma unroll
        for (int u = 0; u < U * 4; ++u) s += ex2_ftz((x[u] - m) * 1.4426950408889634f);
      }
    }
  }
  __shared__ float sm_m[kThreads / 32];
  __shared__ int sm_i[kThreads / 32];
  __shared__ float sm_s[kThreads / 32];
  const int warp = tid >> 5, lane = tid & 31;
  float bm;
  int bi;
  if (kLazy) {
    // block maximum first ...
    float wm = m;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float m2 = __shfl_xor_sync(0xffffffffu, wm, o);
      wm = m2 > wm ? m2 : wm;
    }
    if (lane == 0) sm_m[warp] = wm;
    __syncthreads();
    bm = sm_m[0];
#pragma unroll
    for (int w = 1; w < kThreads / 32; ++w) bm = sm_m[w] > bm ? sm_m[w] : bm;
    // ... then its lowest index: a thread that holds it finds its first position in the pass where its maximum last grew
    int wi = 0x7fffffff;
    if (m == bm && bm > -CUDART_INF_F) {
      float x[U * 2];
      load_half(base_of_max, half_of_max, x, false);
#pragma unroll
      for (int u = U / 2 - 1; u >= 0; --u)
#pragma unroll
        for (int c = 3; c >= 0; --c)
          if (x[4 * u + c] == bm) wi = base_of_max + ((half_of_max * (U / 2) + u) * kThreads + tid) * 4 + c;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) wi = min(wi, __shfl_xor_sync(0xffffffffu, wi, o));
    if (lane == 0) sm_i[warp] = wi;
  } else {
    // block maximum and its lowest index
    float wm = m;
    int wi = mi;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float m2 = __shfl_xor_sync(0xffffffffu, wm, o);
      const int i2 = __shfl_xor_sync(0xffffffffu, wi, o);
      take_better(wm, wi, m2, i2);
    }
    if (lane == 0) { sm_m[warp] = wm; sm_i[warp] = wi; }
    __syncthreads();
    bm = sm_m[0];
    bi = sm_i[0];
#pragma unroll
    for (int w = 1; w < kThreads / 32; ++w) take_better(bm, bi, sm_m[w], sm_i[w]);
  }
  // sums re-based on the block maximum; a thread that saw only -inf contributes nothing
  float t = (m > -CUDART_INF_F) ? s * __expf(m - bm) : 0.f;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
  if (lane == 0) sm_s[warp] = t;
  __syncthreads();
  if (tid == 0) {
    if (kLazy) {
      bi = sm_i[0];
#pragma unroll
      for (int w = 1; w < kThreads / 32; ++w) bi = min(bi, sm_i[w]);
    }
    float total = 0.f;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) total += sm_s[w];
    __stcg(reinterpret_cast<int4*>(partial + (size_t)row * n_chunks + chunk),
           make_int4(__float_as_int(bm), bi, __float_as_int(total), 0));
  }
}

// Selection for batch element b by the whole block (any block size that is a multiple of 32).
// Reads the triples with L2 loads: other blocks of this launch wrote them.
__device__ void select_batch(const Triple* partial, int n_chunks, int b, const SelectArgs& a) {
  __shared__ float s_conf[kMaxBlockLen];
  __shared__ int32_t s_tok[kMaxBlockLen];
  __shared__ uint8_t s_sel[kMaxBlockLen];
  __shared__ int s_count;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, n_warps = blockDim.x >> 5;
  const int L = a.block_len, k = a.k;
  const size_t p0 = (size_t)b * L;
  if (tid == 0) s_count = 0;
  // (1) one warp per row: merge the row's chunk triples (lanes stride over the chunks).  Rows are
  // taken four at a time and each lane first loads its (up to) two triples of every one of them,
  // so one L2 round trip serves four rows; rows with more than 64 chunks loop instead.
  constexpr int RG = 4;
  for (int i0 = warp * RG; i0 < L; i0 += n_warps * RG) {
    int4 v[RG][2];
    bool on[RG];
#pragma unroll
    for (int r = 0; r < RG; ++r) {
      const int i = i0 + r;
      // the triples are asked for without waiting for the mask byte (a row that is not masked has stale ones,
      // which are then ignored): one round trip to L2 instead of two in the serial tail of the kernel
      const uint8_t mk = i < L ? a.masked[p0 + i] : (uint8_t)0;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int c = lane + 32 * h;
        v[r][h] = (i < L && c < n_chunks)
                      ? __ldcg(reinterpret_cast<const int4*>(partial + (p0 + i) * n_chunks) + c)
                      : make_int4(__float_as_int(-CUDART_INF_F), 0x7fffffff, 0, 0);
      }
      on[r] = mk != 0;   // uniform across the warp
    }
#pragma unroll
    for (int r = 0; r < RG; ++r) {
      const int i = i0 + r;
      if (i >= L) break;
      int my_tok = -1;
      float my_conf = -1.f;
      if (on[r]) {
        const int4* t = reinterpret_cast<const int4*>(partial + (p0 + i) * n_chunks);
        float m = __int_as_float(v[r][0].x);
        int idx = v[r][0].y;
        take_better(m, idx, __int_as_float(v[r][1].x), v[r][1].y);
        for (int c = lane + 64; c < n_chunks; c += 32) {
          const int4 w = __ldcg(t + c);
          take_better(m, idx, __int_as_float(w.x), w.y);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const float m2 = __shfl_xor_sync(0xffffffffu, m, o);
          const int i2 = __shfl_xor_sync(0xffffffffu, idx, o);
          take_better(m, idx, m2, i2);
        }
        float s = 0.f;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const float mc = __int_as_float(v[r][h].x);
          if (mc > -CUDART_INF_F) s += __int_as_float(v[r][h].z) * __expf(mc - m);
        }
        for (int c = lane + 64; c < n_chunks; c += 32) {
          const int4 w = __ldcg(t + c);
          const float mc = __int_as_float(w.x);
          if (mc > -CUDART_INF_F) s += __int_as_float(w.z) * __expf(mc - m);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        my_tok = idx;
        my_conf = 1.0f / s;
      }
      if (lane == 0) {
        a.tok[p0 + i] = my_tok;
        a.conf[p0 + i] = my_conf;
        s_conf[i] = my_conf;
        s_tok[i] = my_tok;
        s_sel[i] = 0;
      }
    }
  }
  if (k <= 0) return;
  __syncthreads();
  // (2) rank among the masked positions of this batch element: (confidence desc, position asc)
  for (int i = tid; i < L; i += blockDim.x) {
    const float my_conf = s_conf[i];
    if (my_conf < 0.f) continue;   // unmasked positions hold -1 < every confidence
    int rank = 0;
    for (int j = 0; j < L; ++j) {
      const float cj = s_conf[j];
      rank += (cj > my_conf || (cj == my_conf && j < i)) ? 1 : 0;
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

template <int U, bool kLazy>
__global__ void __launch_bounds__(kThreads)
vocab_reduce_kernel(const float* __restrict__ logits, int vocab, int chunk_len, int n_chunks, Triple* partial,
                    unsigned int* tickets, const SelectArgs sel) {
  dlm_grid_dependency_wait();
  dlm_trigger_dependents();
  const int row = blockIdx.y;
  if (sel.masked[row]) reduce_chunk<U, kLazy>(logits, vocab, chunk_len, n_chunks, partial, row);
  if (tickets == nullptr) return;
  // the last block of this batch element to get here runs its selection
  __shared__ bool is_last;
  // Thread 0 wrote this block's triple, so its release-acquire increment publishes it and, in
  // the block that sees the full count, makes every other block's triple visible.
  const int b = row / sel.block_len;
  if (threadIdx.x == 0) {
    unsigned int t;
    asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(t) : "l"(tickets + b) : "memory");
    is_last = (t == (unsigned int)(n_chunks * sel.block_len) - 1u);
    if (is_last) tickets[b] = 0;   // ready for the next launch
  }
  __syncthreads();
  if (!is_last) return;
  select_batch(partial, n_chunks, b, sel);
}

__global__ void __launch_bounds__(kThreads)
unmask_select_kernel(const Triple* partial, int n_chunks, const SelectArgs sel) {
  dlm_grid_dependency_wait();
  dlm_trigger_dependents();
  select_batch(partial, n_chunks, blockIdx.x, sel);
}

int launch_unmask(const float* logits, int batch, int block_len, int vocab, uint8_t* masked, int32_t* tokens, int k,
                  int32_t* tok, float* conf, int32_t* sel_idx, int32_t* n_sel, Triple* partial,
                  unsigned int* tickets, int num_sms, cudaStream_t s) {
  // A pass of a block covers U * 1024 logits (U vectors in flight per thread); the smaller U
  // when even one resident wave of blocks (4 per SM) would get less than 8192 logits each.
  const long long wave = 4LL * (num_sms > 0 ? num_sms : 148);
  const long long per_block = ((long long)vocab * batch * block_len + wave - 1) / wave;   // logits per block for one wave
  const int U = per_block <= 4096 ? 4 : 8;   // both variants keep 4 blocks of 256 threads on an SM
  // large problems: up to 4 passes per block (a couple of waves of fatter blocks stream better
  // than many waves of one-pass blocks)
  long long passes = per_block / (2 * 8192);
  passes = passes < 1 ? 1 : (passes > 4 ? 4 : passes);
  const int chunk_len = U * kThreads * 4 * (int)passes;
  int n_chunks = (vocab + chunk_len - 1) / chunk_len;
  // A short remainder that would push the grid just past one resident wave (Dream's vocabulary at block 32: 19 chunks
  // x 32 rows = 608 blocks against 592 slots) is folded into the chunk before it: those blocks take a second pass,
  // which costs less than a second wave in the launch's latency chain.
  const long long rows = (long long)batch * block_len;
  if (n_chunks > 1 && rows * n_chunks > wave && rows * (n_chunks - 1) <= wave &&
      vocab - (long long)(n_chunks - 1) * chunk_len <= chunk_len * 3 / 4)
    --n_chunks;
  SelectArgs a;
  a.block_len = block_len; a.k = k; a.masked = masked; a.tokens = tokens; a.tok = tok; a.conf = conf;
  a.sel_idx = sel_idx; a.n_sel = n_sel;
  const dim3 grid(n_chunks, batch * block_len);
  cudaError_t e;
  // blocks of several passes find the argmax's index after the fact (see reduce_chunk)
  if (U == 4) e = dlm_launch(vocab_reduce_kernel<4, false>, grid, dim3(kThreads), 0, s, logits, vocab, chunk_len, n_chunks, partial, tickets, a);
  else if (passes < 2) e = dlm_launch(vocab_reduce_kernel<8, false>, grid, dim3(kThreads), 0, s, logits, vocab, chunk_len, n_chunks, partial, tickets, a);
  else e = dlm_launch(vocab_reduce_kernel<8, true>, grid, dim3(kThreads), 0, s, logits, vocab, chunk_len, n_chunks, partial, tickets, a);
  if (e != cudaSuccess) return -1;
  if (tickets != nullptr) return 1;
  if (dlm_launch(unmask_select_kernel, dim3(batch), dim3(kThreads), 0, s, partial, n_chunks, a) != cudaSuccess) return -1;
  return 2;
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
  DLM_DEVICE_TRY(ctx);
  unsigned int* tickets = batch <= kDlmUnmaskTickets ? ctx->words->unmask_tickets : nullptr;
  const int n = launch_unmask(logits, batch, block_len, vocab, masked, tokens, k, tok, conf, sel_idx, n_sel,
                              static_cast<Triple*>(workspace), tickets, ctx->num_sms, static_cast<cudaStream_t>(stream));
  if (n < 0) return DLM_ERR_CUDA;
  return dlm_launch_ok(ctx, n);
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
  if (launch_unmask(logits, batch, block_len, vocab, masked, tokens, k, tok, conf, sel_idx, n_sel,
                    g_static_partial_addr[device], nullptr, 0, static_cast<cudaStream_t>(stream)) < 0)
    return DLM_ERR_CUDA;
  return cudaGetLastError() == cudaSuccess ? DLM_OK : DLM_ERR_CUDA;
}
