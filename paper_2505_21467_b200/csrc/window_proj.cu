// dlm_window_qkv_project / dlm_window_out_project: the dense projections either side of the attention
// step (Table 1 rows "Q/K/V projection" and "output projection"; Sec. 3.2.1 "Windowed Re-computation":
// the window's K/V are recomputed from its hidden states in every step).
//
// With a window of 32 .. 256 rows these products stream the weight matrix once and do little arithmetic
// per byte: HBM-bound up to about 256 rows, balanced beyond.  The tensor core wants M = 128, so the
// operands are swapped: a block computes Y^T[128 output features x R rows] = W[128 x K] X^T[K x R], the
// weights as the M x K operand (K-major as they lie in memory), the activations as the N x K operand,
// the accumulator in TMEM with one output feature per lane.  K is split across blocks so that every SM
// streams a share of the weights; the blocks of a tile leave fp32 partial tiles in the workspace and the
// last one to arrive (a ticket) adds them in a fixed order, adds the bias and writes bf16 in the layout
// the consumer reads (Q/K/V head by head for the attention step, or row-major hidden states).
//
// Block = 6 warps: warp 0 one TMA producer lane (weight panel [128 x 64] and activation panel [R x 64]
// per stage, 128-byte swizzle), warp 1 the tcgen05.mma issuer (4 MMAs of K = 16 per stage), warps 2-5 the
// epilogue (thread = TMEM lane = output feature).
#include <cuda.h>
#include <cuda_bf16.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace {

using namespace sm100;

constexpr int kThreads = 192;
constexpr int kTileN = 128;                 // output features per block
constexpr int kChunkK = 64;                 // K elements per pipeline stage (one 128-byte swizzled panel)
constexpr int kMaxRows = 256;               // activation rows per block (MMA N)
constexpr int kWBytes = kTileN * kChunkK * 2;
constexpr int kMaxStages = 8;

struct ProjParams {
  // destination: mode 0 = Q/K/V head by head ([B][heads][q_cap][D] each), mode 1 = row-major [rows][n_out]
  int mode;
  __nv_bfloat16* q_out;
  __nv_bfloat16* k_out;
  __nv_bfloat16* v_out;
  const __nv_bfloat16* bias;   // [n_out] or nullptr
  const float* rope_cos;       // mode 0: rotary embedding of the query and key heads, fp32 [B][q_cap][head_dim / 2],
  const float* rope_sin;       // or both nullptr
  // mode 0: K/V rows are also staged in the cache (one layer: [B][n_kv_heads][capacity][head_dim]) at row
  // cache_len[b] + i, the slot the commit's window mode uses; nullptr: no staging
  __nv_bfloat16* stage_k;
  __nv_bfloat16* stage_v;
  const int32_t* cache_len;    // [B]
  const int32_t* q_len;        // [B] rows of the window that are active (staged), or nullptr: all q_cap
  int capacity;
  float* partial;              // [row chunk][feature tile][split][rows_pad][128] fp32
  unsigned int* tickets;       // one per (row chunk, feature tile)
  int rows_total, q_cap, n_q_heads, n_kv_heads, head_dim, n_out, k_total;
  int batch;                   // mode 1 with head-split activations: batch elements (row chunk = all rows)
  int act_heads;               // mode 1: activations are [B][act_heads][q_cap][D] (0: plain [rows][K])
  int rows_pad;                // MMA N: rows of a chunk rounded up to 32
  int n_split, k_per_split;    // K split across blocks, elements per split (a multiple of 64)
  int n_stages;
  int* status;
};

// Waits until the counter at `addr` reaches `target` (acquire, device scope), bounded like the mbarrier waits.
__device__ __forceinline__ bool wait_count(const unsigned int* addr, unsigned int target, volatile int* abort_flag) {
  const uint64_t t0 = global_timer_ns();
  for (uint32_t spin = 1;; ++spin) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(addr) : "memory");
    if (v >= target) return true;
    if ((spin & 15u) == 0u) {
      if (*abort_flag) return false;
      if (global_timer_ns() - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        return false;
      }
    }
  }
}

__global__ void __launch_bounds__(kThreads, 1)
window_proj_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_x, const ProjParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t pad = (1024u - (smem_u32(smem_raw) & 1023u)) & 1023u;
  const uint32_t base = smem_u32(smem_raw) + pad;
  const uint32_t x_bytes = (uint32_t)p.rows_pad * 128u;
  const uint32_t stage_bytes = kWBytes + x_bytes;
  const uint32_t sm_bar = base + p.n_stages * stage_bytes;          // full[8], empty[8], done
  const uint32_t bar_full = sm_bar, bar_empty = sm_bar + 8 * kMaxStages, bar_done = sm_bar + 16 * kMaxStages;
  const uint32_t bar_red = bar_done + 8;   // the partial tiles' slices of this block's rows have landed in shared memory
  int* const flags = reinterpret_cast<int*>(smem_raw + pad + (size_t)p.n_stages * stage_bytes + 16 * kMaxStages + 16);
  volatile int* const abort_ptr = flags;
  volatile int* const never_ptr = flags + 1;
  uint32_t* const tmem_slot = reinterpret_cast<uint32_t*>(flags + 2);
  volatile int* const is_last = flags + 3;
  volatile int* const warp_ok = flags + 4;   // [4]: the epilogue warps' waits, so that all four take the same branches

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tile = blockIdx.x, split = blockIdx.y, chunk = blockIdx.z;
  const int row0 = chunk * kMaxRows;
  const int k0 = split * p.k_per_split;
  const int k1 = min(k0 + p.k_per_split, p.k_total);
  const int n_k = (k1 - k0) / kChunkK;     // stages' worth of K in this block (>= 1 by construction)
  uint32_t tmem_cols = 32;
  while ((int)tmem_cols < p.rows_pad) tmem_cols <<= 1;

  if (tid == 0) {
    *abort_ptr = 0; *never_ptr = 0; *is_last = 0;
    for (int i = 0; i < p.n_stages; ++i) {
      mbar_init(bar_full + 8 * i, 1);
      mbar_init(bar_empty + 8 * i, 1);
    }
    mbar_init(bar_done, 1);
    mbar_init(bar_red, 1);
    mbar_fence_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), tmem_cols);
    tmem_relinquish();
  }
  if (warp == 0 && lane == 0) {
    prefetch_tensormap(&tm_w);
    prefetch_tensormap(&tm_x);
  }
  dlm_grid_dependency_wait();
  dlm_trigger_dependents();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0) {
    // ================================================================= TMA producer
    if (lane == 0) {
      bool ok = true;
      int s = 0, round = 0, issued = 0;
      // bytes a stage receives: a box counts in full, also where it reaches beyond the tensor
      const uint32_t tx = kWBytes + (p.act_heads == 0 ? x_bytes : (uint32_t)(p.batch * p.q_cap) * 128u);
      for (int kc = 0; kc < n_k && ok; ++kc) {
        if (round > 0) ok = mbar_wait(bar_empty + 8 * s, (round - 1) & 1, abort_ptr);
        if (!ok) break;
        const uint32_t dst = base + s * stage_bytes;
        const int k = k0 + kc * kChunkK;
        mbar_expect_tx(bar_full + 8 * s, tx);
        tma_load_3d(dst, &tm_w, bar_full + 8 * s, k, tile * kTileN, 0);
        if (p.act_heads == 0) {
          tma_load_3d(dst + kWBytes, &tm_x, bar_full + 8 * s, k, row0, 0);
        } else {
          // activations [B][heads][q_cap][D]: K index k = head * D + d; one box of q_cap rows per batch element
          const int head = k / p.head_dim, d = k % p.head_dim;
          for (int b = 0; b < p.batch; ++b)
            tma_load_3d(dst + kWBytes + (uint32_t)(b * p.q_cap) * 128u, &tm_x, bar_full + 8 * s, d, 0, b * p.act_heads + head);
        }
        ++issued;
        if (++s == p.n_stages) { s = 0; ++round; }
      }
      if (!ok) {   // unwinding: let the copies already issued land before the block's memory is released
        for (int i = max(0, issued - p.n_stages); i < issued; ++i)
          mbar_wait(bar_full + 8 * (i % p.n_stages), (i / p.n_stages) & 1, never_ptr);
      }
    }
  } else if (warp == 1) {
    // ================================================================= MMA issuer
    bool ok = true;
    const uint32_t idesc = make_idesc_bf16(128, (uint32_t)p.rows_pad, 0);
    int s = 0, round = 0;
    for (int kc = 0; kc < n_k && ok; ++kc) {
      ok = __all_sync(0xffffffffu, mbar_wait(bar_full + 8 * s, round & 1, abort_ptr)) != 0;
      if (!ok) break;
      tc_fence_after_sync();
      const uint64_t dw = make_smem_desc_sw128(base + s * stage_bytes, 16, 1024);
      const uint64_t dx = make_smem_desc_sw128(base + s * stage_bytes + kWBytes, 16, 1024);
      if (elect_one_sync()) {
#pragma unroll
        for (int k = 0; k < kChunkK / 16; ++k) {
          if (kc == 0 && k == 0) mma_ss<false>(tmem, dw, dx, idesc);
          else mma_ss<true>(tmem, desc_offset(dw, k * 32), desc_offset(dx, k * 32), idesc);
        }
        tc_commit(bar_empty + 8 * s);
      }
      __syncwarp();
      if (++s == p.n_stages) { s = 0; ++round; }
    }
    if (elect_one_sync()) tc_commit(bar_done);
    __syncwarp();
  }

  // ================================================================= epilogue (warps 2-5)
  if (warp >= 2) {
    // TMEM lanes are tied to warp % 4: warps 2, 3, 4, 5 own lanes 64-95, 96-127, 0-31, 32-63
    const int lane_base = (warp & 3) * 32;
    const int f = lane_base + lane;                       // feature within the tile = TMEM lane
    const int n = tile * kTileN + f;                      // output feature
    bool ok = __all_sync(0xffffffffu, mbar_wait(bar_done, 0, abort_ptr)) != 0;
    tc_fence_after_sync();
    // rotary embedding (mode 0): feature d of a query or key head is paired with feature d +- head_dim / 2
    const bool rope = p.mode == 0 && p.rope_cos != nullptr;
    const int half = p.head_dim >> 1;
    const int rows_here = min(kMaxRows, p.rows_total - row0);
    const size_t tile_slot = ((size_t)chunk * gridDim.x + tile) * p.n_split;
    float* my_partial = p.partial + (tile_slot + split) * (size_t)p.rows_pad * kTileN + f;
    if (ok && p.n_split > 1) {
      // fp32 partial tile, [row][feature]: a warp's 32 lanes write 128 contiguous bytes per row
      uint32_t v[32];
      for (int c = 0; c < p.rows_pad; c += 32) {
        tmem_ld32(tmem + ((uint32_t)lane_base << 16) + c, v);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (c + j < rows_here) __stcg(my_partial + (size_t)(c + j) * kTileN, __uint_as_float(v[j]));
      }
      __threadfence();
    }
    if (lane == 0) warp_ok[warp - 2] = ok ? 1 : 0;
    named_bar_sync(1, 128);
    ok = warp_ok[0] && warp_ok[1] && warp_ok[2] && warp_ok[3];
    // Split K: the n_split blocks of a tile share its final reduction.  Block s takes rows [lo, hi) of the tile; when
    // all partial tiles are there (arrival counter; the blocks of a launch are all resident: there are no more of
    // them than SMs) it fetches those rows of every partial tile into the shared memory of the pipeline stages, which
    // are free by now, with bulk copies, all in flight at once.  (One block folding the other partial tiles with
    // loads of its own took 6 us of a 16 us call at 32 rows and 37 of 52 us at 256: every batch of loads is a trip of
    // about 2 us to data other SMs have just written.)  A second counter lets the last block to leave clear both.
    const int red_lo = p.rows_pad * split / p.n_split, red_hi = p.rows_pad * (split + 1) / p.n_split;
    const uint32_t slice_bytes = (uint32_t)(red_hi - red_lo) * kTileN * 4u;
    if (p.n_split > 1) {
      if (tid == 64) {   // first epilogue thread: every partial store above happened before the barrier
        int go = 2;
        unsigned int* const arrive = p.tickets + chunk * gridDim.x + tile;
        unsigned int* const depart = arrive + kDlmMaxSplitUnits / 2;
        if (ok) {
          unsigned int t;
          asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(t) : "l"(arrive) : "memory");
          if (wait_count(arrive, (unsigned int)p.n_split, abort_ptr)) {
            fence_proxy_async_all();
            mbar_expect_tx(bar_red, (uint32_t)p.n_split * slice_bytes);
            for (int s2 = 0; s2 < p.n_split; ++s2)
              bulk_load(base + s2 * slice_bytes, p.partial + ((tile_slot + s2) * (size_t)p.rows_pad + red_lo) * kTileN, slice_bytes,
                        bar_red);
            if (atomicAdd(depart, 1u) == (unsigned int)p.n_split - 1u) {   // every block of the tile is past its wait
              *arrive = 0;
              *depart = 0;
            }
            go = 1;
          }
        }
        *is_last = go;
      }
      named_bar_sync(1, 128);
    }
    // where output feature `feat` of row (b, i) goes: element offset of (b = 0, i = 0) and the two strides
    // ... and, for a key or value feature of a staging call, where its copy in the cache goes: element offset of
    // (b = 0, cache row 0); rows are head_dim apart, batch elements n_kv_heads * capacity * head_dim
    auto place = [&](int feat, __nv_bfloat16*& dst, size_t& row_stride, size_t& b_stride, __nv_bfloat16*& stage) {
      stage = nullptr;
      if (p.mode == 0) {
        const int head = feat / p.head_dim, d = feat % p.head_dim;
        int heads, h;
        if (head < p.n_q_heads) { dst = p.q_out; heads = p.n_q_heads; h = head; }
        else if (head < p.n_q_heads + p.n_kv_heads) { dst = p.k_out; heads = p.n_kv_heads; h = head - p.n_q_heads; stage = p.stage_k; }
        else { dst = p.v_out; heads = p.n_kv_heads; h = head - p.n_q_heads - p.n_kv_heads; stage = p.stage_v; }
        dst += (size_t)h * p.q_cap * p.head_dim + d;
        if (stage) stage += (size_t)h * p.capacity * p.head_dim + d;
        row_stride = p.head_dim;
        b_stride = (size_t)heads * p.q_cap * p.head_dim;
      } else {
        dst = p.q_out + feat;
        row_stride = p.n_out;
        b_stride = (size_t)p.q_cap * p.n_out;
      }
    };
    // cache row that window row i of batch element b is staged at, or -1: inactive row, or no room (reported)
    auto stage_row = [&](int b, int i) -> int {
      if (p.q_len && i >= __ldg(p.q_len + b)) return -1;
      const int pos = __ldg(p.cache_len + b) + i;
      if (pos < 0 || pos >= p.capacity) {
        dlm_set_status(p.status, DLM_ERR_CAPACITY);
        return -1;
      }
      return pos;
    };
    const size_t stage_b_stride = (size_t)p.n_kv_heads * p.capacity * p.head_dim;
    if (ok && p.n_split == 1) {
      // the whole sum is in TMEM: thread = feature, one 2-byte store per row (the output is small beside the weights)
      const float bias = p.bias ? __bfloat162float(p.bias[n]) : 0.f;
      __nv_bfloat16* dst;
      __nv_bfloat16* stage;
      size_t row_stride, b_stride;
      place(n, dst, row_stride, b_stride, stage);
      uint32_t v[32];
      const bool turn = rope && n / p.head_dim < p.n_q_heads + p.n_kv_heads;   // the same for a feature and its partner
      const int d = n % p.head_dim;
      // the partner's values come through shared memory (the pipeline's first stage is free: every MMA has finished);
      // [feature][33 floats]: 128 x 33 x 4 bytes fit a stage
      float* const xch = reinterpret_cast<float*>(smem_raw + pad);
      const int f_partner = d < half ? f + half : f - half;
      if (!rope && !stage) {
        // the plain projection: nothing but the bias between the accumulator and the store
        for (int c = 0; c < p.rows_pad; c += 32) {
          tmem_ld32(tmem + ((uint32_t)lane_base << 16) + c, v);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const int r = row0 + c + j;
            if (c + j < rows_here) {
              const int b = r / p.q_cap, i = r % p.q_cap;
              dst[(size_t)b * b_stride + (size_t)i * row_stride] = __float2bfloat16_rn(__uint_as_float(v[j]) + bias);
            }
          }
        }
      } else {
        for (int c = 0; c < p.rows_pad; c += 32) {
          tmem_ld32(tmem + ((uint32_t)lane_base << 16) + c, v);
          tmem_ld_wait();
          if (rope) {   // block-uniform: all four warps meet at the two barriers
#pragma unroll
            for (int j = 0; j < 32; ++j) xch[f * 33 + j] = __uint_as_float(v[j]) + bias;
            named_bar_sync(1, 128);
          }
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const int r = row0 + c + j;
            if (c + j < rows_here) {
              const int b = r / p.q_cap, i = r % p.q_cap;
              float y = __uint_as_float(v[j]) + bias;
              if (turn) {
                const size_t a = ((size_t)b * p.q_cap + i) * half + (d < half ? d : d - half);
                const float cs = p.rope_cos[a], sn = p.rope_sin[a], other = xch[f_partner * 33 + j];
                y = d < half ? y * cs - other * sn : y * cs + other * sn;
              }
              const __nv_bfloat16 yb = __float2bfloat16_rn(y);
              dst[(size_t)b * b_stride + (size_t)i * row_stride] = yb;
              if (stage) {
                const int pos = stage_row(b, i);
                if (pos >= 0) stage[(size_t)b * stage_b_stride + (size_t)pos * p.head_dim] = yb;
              }
            }
          }
          if (rope) named_bar_sync(1, 128);   // the next chunk overwrites the exchange area
        }
      }
    } else if (ok && *is_last == 1) {
      // every block adds its rows of the partial tiles in split order (the sum does not depend on the order of arrival): a
      // thread takes 4 neighbouring features of every fourth row, 16-byte loads from shared memory, 8-byte stores; a
      // warp's stores cover 128 features of one row
      const bool landed = __all_sync(0xffffffffu, mbar_wait(bar_red, 0, abort_ptr)) != 0;
      // the thread that issued the copies does not go on to the teardown before they have landed
      if (tid == 64 && !landed) mbar_wait(bar_red, 0, never_ptr);
      const int t = tid - 64;
      const int fq = (t & 31) * 4;
      const int n4 = tile * kTileN + fq;
      float b4[4] = {0.f, 0.f, 0.f, 0.f};
      if (p.bias)
        for (int j = 0; j < 4; ++j) b4[j] = __bfloat162float(p.bias[n4 + j]);
      __nv_bfloat16* dst;
      __nv_bfloat16* stage;
      size_t row_stride, b_stride;
      place(n4, dst, row_stride, b_stride, stage);
      const int red_end = landed ? min(red_hi, rows_here) : red_lo;   // rows beyond the call's hold nothing
      for (int rr0 = red_lo + (t >> 5); rr0 < red_end; rr0 += 16) {
        float4 accs[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) accs[j] = make_float4(b4[0], b4[1], b4[2], b4[3]);
        for (int s2 = 0; s2 < p.n_split; ++s2) {
#pragma unroll
          for (int j = 0; j < 4; ++j)
            if (rr0 + 4 * j < red_end) {
              const float4 x = ld_shared_f4(base + s2 * slice_bytes + (uint32_t)((rr0 + 4 * j - red_lo) * kTileN + fq) * 4u);
              accs[j].x += x.x; accs[j].y += x.y; accs[j].z += x.z; accs[j].w += x.w;
            }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int rr = rr0 + 4 * j;
          if (rr >= red_end) break;   // the same for the whole warp
          float4 acc = accs[j];
          const int r = row0 + rr;
          const int b = r / p.q_cap, i = r % p.q_cap;
          if (rope) {
            // this lane's 4 features and their partners' (head_dim / 2 features = head_dim / 8 lanes away) turn together;
            // rr is the same for the whole warp, so every lane is here for the exchange
            const int dl = p.head_dim >> 3;
            const float4 o = make_float4(__shfl_xor_sync(0xffffffffu, acc.x, dl), __shfl_xor_sync(0xffffffffu, acc.y, dl),
                                         __shfl_xor_sync(0xffffffffu, acc.z, dl), __shfl_xor_sync(0xffffffffu, acc.w, dl));
            const int d = n4 % p.head_dim;
            if (n4 / p.head_dim < p.n_q_heads + p.n_kv_heads) {
              const size_t a = ((size_t)b * p.q_cap + i) * half + (d < half ? d : d - half);
              const float4 cs = __ldg(reinterpret_cast<const float4*>(p.rope_cos + a));
              const float4 sn = __ldg(reinterpret_cast<const float4*>(p.rope_sin + a));
              const float sg = d < half ? -1.f : 1.f;
              acc.x = fmaf(sg * o.x, sn.x, acc.x * cs.x);
              acc.y = fmaf(sg * o.y, sn.y, acc.y * cs.y);
              acc.z = fmaf(sg * o.z, sn.z, acc.z * cs.z);
              acc.w = fmaf(sg * o.w, sn.w, acc.w * cs.w);
            }
          }
          const __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
          uint2 pk;
          pk.x = *reinterpret_cast<const uint32_t*>(&lo);
          pk.y = *reinterpret_cast<const uint32_t*>(&hi);
          *reinterpret_cast<uint2*>(dst + (size_t)b * b_stride + (size_t)i * row_stride) = pk;
          if (stage) {
            const int pos = stage_row(b, i);
            if (pos >= 0) *reinterpret_cast<uint2*>(stage + (size_t)b * stage_b_stride + (size_t)pos * p.head_dim) = pk;
          }
        }
      }
    }
  }
  // ---- teardown
  __syncwarp();
  if (tid == 0 && *abort_ptr) dlm_set_status(p.status, DLM_ERR_TIMEOUT);
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem, tmem_cols);
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// bf16 tensor viewed as [slabs][rows][inner]; box = 64 elements x box_rows rows x 1 slab, 128-byte swizzle.
int encode_map3(dlm_ctx* ctx, CUtensorMap* map, const void* base, long long inner, long long rows, long long slabs, int box_rows) {
  if (!ctx->encode_tiled) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn ||
        q != cudaDriverEntryPointSuccess)
      return DLM_ERR_CUDA;
    ctx->encode_tiled = fn;
  }
  const cuuint64_t dims[3] = {(cuuint64_t)inner, (cuuint64_t)rows, (cuuint64_t)slabs};
  const cuuint64_t strides[2] = {(cuuint64_t)inner * 2, (cuuint64_t)rows * inner * 2};
  const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  const cuuint32_t elem[3] = {1, 1, 1};
  const CUresult r = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled)(
      map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, elem,
      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? DLM_OK : DLM_ERR_CUDA;
}

struct ProjPlan {
  int rows_pad, chunks, tiles, n_split, k_per_split, n_stages, smem_bytes;
  size_t ws_bytes;
};

// rows: activation rows of the call; whole_rows: every block sees all rows (head-split activations)
bool make_proj_plan(const dlm_ctx* ctx, int rows, int n_out, int k_total, bool whole_rows, ProjPlan& pl) {
  if (whole_rows && rows > kMaxRows) return false;
  pl.chunks = (rows + kMaxRows - 1) / kMaxRows;
  const int rows_chunk = pl.chunks == 1 ? rows : kMaxRows;
  pl.rows_pad = (rows_chunk + 31) & ~31;
  pl.tiles = n_out / kTileN;
  const int k_chunks = k_total / kChunkK;
  // split K so that about one block per SM streams weights, each with at least four stages' worth of K
  int split = ctx->num_sms / (pl.tiles * pl.chunks);
  if (split > k_chunks / 4) split = k_chunks / 4;
  if (split < 1) split = 1;
  const int chunks_per_split = (k_chunks + split - 1) / split;
  pl.n_split = (k_chunks + chunks_per_split - 1) / chunks_per_split;
  pl.k_per_split = chunks_per_split * kChunkK;
  const int stage = kWBytes + pl.rows_pad * 128;
  const int aux = 16 * kMaxStages + 16 + 64;
  int stages = (ctx->max_smem_optin - 1024 - aux) / stage;
  if (stages > kMaxStages) stages = kMaxStages;
  if (stages > chunks_per_split) stages = chunks_per_split;
  if (stages < 2) return false;
  pl.n_stages = stages;
  // the shared final reduction parks every partial tile's slice of a block's rows in the stages' memory
  if (pl.n_split > 1 && (long long)stages * stage < (long long)(pl.rows_pad + pl.n_split) * kTileN * 4) {
    pl.n_split = 1;
    pl.k_per_split = k_chunks * kChunkK;
  }
  pl.smem_bytes = 1024 + stages * stage + aux;
  pl.ws_bytes = pl.n_split > 1 ? (size_t)pl.chunks * pl.tiles * pl.n_split * pl.rows_pad * kTileN * sizeof(float) : 0;
  return (long long)pl.tiles * pl.chunks <= kDlmMaxSplitUnits / 2;   // two counters per tile
}

int launch_proj(dlm_ctx* ctx, const ProjPlan& pl, ProjParams& p, const CUtensorMap& tm_w, const CUtensorMap& tm_x, void* workspace,
                size_t workspace_bytes, cudaStream_t s) {
  if (pl.ws_bytes > 0 && (!workspace || workspace_bytes < pl.ws_bytes || ((uintptr_t)workspace & 255))) return DLM_ERR_WORKSPACE;
  if (!ctx->proj_configured) {
    DLM_CUDA_TRY(cudaFuncSetAttribute(window_proj_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin));
    ctx->proj_configured = true;
  }
  p.partial = static_cast<float*>(workspace);
  p.tickets = ctx->words->attn_unit_tickets;
  p.rows_pad = pl.rows_pad;
  p.n_split = pl.n_split;
  p.k_per_split = pl.k_per_split;
  p.n_stages = pl.n_stages;
  p.status = &ctx->words->status;
  DLM_CUDA_TRY(dlm_launch(window_proj_kernel, dim3(pl.tiles, pl.n_split, pl.chunks), dim3(kThreads), (size_t)pl.smem_bytes, s, tm_w,
                          tm_x, p));
  return dlm_launch_ok(ctx, 1);
}

}  // namespace

extern "C" size_t dlm_window_proj_workspace_bytes(const dlm_ctx* ctx, int rows, int n_out, int k_total) {
  if (!ctx || rows <= 0 || n_out <= 0 || k_total <= 0 || n_out % kTileN != 0 || k_total % kChunkK != 0) return 0;
  ProjPlan pl;
  if (!make_proj_plan(ctx, rows, n_out, k_total, false, pl)) return 0;
  return pl.ws_bytes + 256;
}

namespace {
int qkv_project(dlm_ctx* ctx, const void* x, const void* w, const void* bias, const float* rope_cos, const float* rope_sin,
                int batch, int q_cap, int d_model, int n_q_heads, int n_kv_heads, int head_dim, void* q_out, void* k_out,
                void* v_out, const dlm_kv_cache* cache, int layer, const int32_t* q_len, void* workspace, size_t workspace_bytes,
                void* stream);
}

extern "C" int dlm_window_qkv_project(dlm_ctx* ctx, const void* x, const void* w, const void* bias, int batch, int q_cap,
                                      int d_model, int n_q_heads, int n_kv_heads, int head_dim, void* q_out, void* k_out,
                                      void* v_out, void* workspace, size_t workspace_bytes, void* stream) {
  return qkv_project(ctx, x, w, bias, nullptr, nullptr, batch, q_cap, d_model, n_q_heads, n_kv_heads, head_dim, q_out, k_out,
                     v_out, nullptr, 0, nullptr, workspace, workspace_bytes, stream);
}

extern "C" int dlm_window_qkv_project_rope(dlm_ctx* ctx, const void* x, const void* w, const void* bias, const float* rope_cos,
                                           const float* rope_sin, int batch, int q_cap, int d_model, int n_q_heads,
                                           int n_kv_heads, int head_dim, void* q_out, void* k_out, void* v_out, void* workspace,
                                           size_t workspace_bytes, void* stream) {
  if (!rope_cos || !rope_sin) return DLM_ERR_NULL;
  // a feature and its partner must lie in one 128-feature tile, and 4 neighbouring features in one half of a head
  if (head_dim != 64 && head_dim != 128) return DLM_ERR_UNSUPPORTED;
  if (((uintptr_t)rope_cos | (uintptr_t)rope_sin) & 15) return DLM_ERR_UNSUPPORTED;
  return qkv_project(ctx, x, w, bias, rope_cos, rope_sin, batch, q_cap, d_model, n_q_heads, n_kv_heads, head_dim, q_out, k_out,
                     v_out, nullptr, 0, nullptr, workspace, workspace_bytes, stream);
}

extern "C" int dlm_window_qkv_project_stage(dlm_ctx* ctx, const void* x, const void* w, const void* bias, const float* rope_cos,
                                            const float* rope_sin, int batch, int q_cap, int d_model, int n_q_heads,
                                            int n_kv_heads, int head_dim, const int32_t* q_len, void* q_out, void* k_out,
                                            void* v_out, const dlm_kv_cache* cache, int layer, void* workspace,
                                            size_t workspace_bytes, void* stream) {
  if (!cache || !cache->k || !cache->v || !cache->cache_len) return DLM_ERR_NULL;
  if ((rope_cos == nullptr) != (rope_sin == nullptr)) return DLM_ERR_NULL;
  if (rope_cos && head_dim != 64 && head_dim != 128) return DLM_ERR_UNSUPPORTED;
  if (((uintptr_t)rope_cos | (uintptr_t)rope_sin | (uintptr_t)cache->k | (uintptr_t)cache->v) & 15) return DLM_ERR_UNSUPPORTED;
  if (layer < 0 || layer >= cache->n_layers || cache->batch != batch || cache->n_kv_heads != n_kv_heads ||
      cache->head_dim != head_dim || cache->capacity <= 0)
    return DLM_ERR_SHAPE;
  return qkv_project(ctx, x, w, bias, rope_cos, rope_sin, batch, q_cap, d_model, n_q_heads, n_kv_heads, head_dim, q_out, k_out,
                     v_out, cache, layer, q_len, workspace, workspace_bytes, stream);
}

namespace {
int qkv_project(dlm_ctx* ctx, const void* x, const void* w, const void* bias, const float* rope_cos, const float* rope_sin,
                int batch, int q_cap, int d_model, int n_q_heads, int n_kv_heads, int head_dim, void* q_out, void* k_out,
                void* v_out, const dlm_kv_cache* cache, int layer, const int32_t* q_len, void* workspace, size_t workspace_bytes,
                void* stream) {
  if (!ctx || !x || !w || !q_out || !k_out || !v_out) return DLM_ERR_NULL;
  if (batch <= 0 || q_cap <= 0 || d_model <= 0 || n_q_heads <= 0 || n_kv_heads <= 0 || head_dim <= 0) return DLM_ERR_SHAPE;
  const long long n_out = (long long)(n_q_heads + 2 * n_kv_heads) * head_dim;
  const long long rows = (long long)batch * q_cap;
  if (n_out % kTileN != 0 || d_model % kChunkK != 0 || head_dim % 8 != 0 || rows > (1 << 20) || n_out > (1 << 24))
    return DLM_ERR_UNSUPPORTED;
  if (((uintptr_t)x | (uintptr_t)w | (uintptr_t)q_out | (uintptr_t)k_out | (uintptr_t)v_out) & 15) return DLM_ERR_UNSUPPORTED;
  DLM_DEVICE_TRY(ctx);
  ProjPlan pl;
  if (!make_proj_plan(ctx, (int)rows, (int)n_out, d_model, false, pl)) return DLM_ERR_UNSUPPORTED;
  CUtensorMap tm_w, tm_x;
  int rc = encode_map3(ctx, &tm_w, w, d_model, n_out, 1, kTileN);
  if (rc == DLM_OK) rc = encode_map3(ctx, &tm_x, x, d_model, rows, 1, pl.rows_pad);
  if (rc != DLM_OK) return rc;
  ProjParams p = {};
  p.mode = 0;
  p.q_out = static_cast<__nv_bfloat16*>(q_out);
  p.k_out = static_cast<__nv_bfloat16*>(k_out);
  p.v_out = static_cast<__nv_bfloat16*>(v_out);
  p.bias = static_cast<const __nv_bfloat16*>(bias);
  p.rope_cos = rope_cos;
  p.rope_sin = rope_sin;
  if (cache) {
    const size_t layer_elems = (size_t)batch * n_kv_heads * cache->capacity * head_dim;
    p.stage_k = static_cast<__nv_bfloat16*>(cache->k) + (size_t)layer * layer_elems;
    p.stage_v = static_cast<__nv_bfloat16*>(cache->v) + (size_t)layer * layer_elems;
    p.cache_len = cache->cache_len;
    p.q_len = q_len;
    p.capacity = cache->capacity;
  }
  p.rows_total = (int)rows; p.q_cap = q_cap; p.n_q_heads = n_q_heads; p.n_kv_heads = n_kv_heads; p.head_dim = head_dim;
  p.n_out = (int)n_out; p.k_total = d_model; p.batch = batch; p.act_heads = 0;
  return launch_proj(ctx, pl, p, tm_w, tm_x, workspace, workspace_bytes, static_cast<cudaStream_t>(stream));
}
}  // namespace

extern "C" int dlm_window_out_project(dlm_ctx* ctx, const void* o, const void* wo, const void* bias, int batch, int q_cap,
                                      int d_model, int n_q_heads, int head_dim, void* y, void* workspace,
                                      size_t workspace_bytes, void* stream) {
  if (!ctx || !o || !wo || !y) return DLM_ERR_NULL;
  if (batch <= 0 || q_cap <= 0 || d_model <= 0 || n_q_heads <= 0 || head_dim <= 0) return DLM_ERR_SHAPE;
  const long long k_total = (long long)n_q_heads * head_dim, rows = (long long)batch * q_cap;
  // a stage holds 64 features of one head for every row of the call: whole heads of 64-element panels, all rows in
  // one block (<= 256), and each batch element's rows starting on a swizzle-atom boundary (8 rows)
  if (d_model % kTileN != 0 || head_dim % kChunkK != 0 || rows > kMaxRows || (batch > 1 && q_cap % 8 != 0))
    return DLM_ERR_UNSUPPORTED;
  if (((uintptr_t)o | (uintptr_t)wo | (uintptr_t)y) & 15) return DLM_ERR_UNSUPPORTED;
  DLM_DEVICE_TRY(ctx);
  ProjPlan pl;
  if (!make_proj_plan(ctx, (int)rows, d_model, (int)k_total, true, pl)) return DLM_ERR_UNSUPPORTED;
  CUtensorMap tm_w, tm_x;
  int rc = encode_map3(ctx, &tm_w, wo, k_total, d_model, 1, kTileN);
  // one box per batch element: q_cap rows; the rows of the panel beyond batch * q_cap stay as they are (their
  // accumulator columns are never read)
  if (rc == DLM_OK) rc = encode_map3(ctx, &tm_x, o, head_dim, q_cap, (long long)batch * n_q_heads, q_cap);
  if (rc != DLM_OK) return rc;
  ProjParams p = {};
  p.mode = 1;
  p.q_out = static_cast<__nv_bfloat16*>(y);
  p.bias = static_cast<const __nv_bfloat16*>(bias);
  p.rows_total = (int)rows; p.q_cap = q_cap; p.n_q_heads = n_q_heads; p.n_kv_heads = 0; p.head_dim = head_dim;
  p.n_out = d_model; p.k_total = (int)k_total; p.batch = batch; p.act_heads = n_q_heads;
  return launch_proj(ctx, pl, p, tm_w, tm_x, workspace, workspace_bytes, static_cast<cudaStream_t>(stream));
}
