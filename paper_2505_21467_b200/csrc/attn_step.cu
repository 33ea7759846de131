// dlm_freecache_attn_step: attention of the active window over [cache rows ; fresh rows]
// (Sec. 3.2.1 "Windowed Re-computation"; Table 1 rows QK^T and Attention Score x Value;
// bidirectional: no causal mask).
//
// One work unit is (layer, batch element, KV head): all g = Hq/Hkv query heads of that KV
// head, q_cap rows each, form up to two 128-row M tiles that share every K/V tile, so K/V are
// read from HBM once per KV head.  Keys are visited in tiles of 128 rows: first the visible
// cache rows, then the fresh rows.
//
// Block = 10 warps, one block per SM (persistent):
//   warps 0-3   softmax of M tile 0 (thread = query row = TMEM lane)
//   warps 4-7   softmax of M tile 1
//   warp  8     TMA producer (one lane): Q once per segment, K and V tiles through two rings
//   warp  9     tcgen05.mma issuer (one lane): S = Q K^T into TMEM, then O += P V with P read
//               from TMEM (it overwrites S in place as packed bf16)
// Online softmax in fp32 with base-2 exponentials; O stays in TMEM and is rescaled only when
// a row maximum grows.
//
// Scheduling.  Every (unit, key tile) pair is one item of a global list; block c takes the
// contiguous share [c*T/G, (c+1)*T/G) of it.  A share covers whole units (result written
// directly) and at most two partial units (unnormalised O, running max and sum written to the
// workspace; a second kernel merges the partials of a unit in a fixed order, so the result is
// deterministic).  With many more units than SMs the split is not worth its traffic and units
// are dealt round-robin instead.
#include <cuda.h>
#include <cuda_bf16.h>
#include <math_constants.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace {

using namespace sm100;

constexpr int kThreads = 320;
constexpr int kTileKeys = 128;
constexpr int kPanelBytes = 128 * 128;   // one 64-element-wide panel of a 128-row tile
constexpr int kMaxBatch = 1024;
constexpr int kTmemCols = 512;

template <int D>
struct Geometry {
  static constexpr int kPanels = D / 64;
  static constexpr int kTileBytes = kPanels * kPanelBytes;      // one K tile, V tile or Q M-tile
  static constexpr int kStages = (D == 128) ? 2 : 4;            // ring depth of K and of V
  static constexpr int kSmemBytes = (2 + 2 * kStages) * kTileBytes + 1024 /*alignment*/ + 256 /*barriers*/;
  static constexpr uint32_t kColO = 0;                          // O[mt] at mt * D
  static constexpr uint32_t kColS = 2 * D;                      // S[mt] at 2D + mt * 128 (P aliases it)
};

struct AttnParams {
  const int32_t* cache_len;
  const int32_t* q_len;
  __nv_bfloat16* out;
  float* lse;
  float* ws_o;    // [2 * grid][n_mt * 128][D]   partial unnormalised O
  float* ws_ml;   // [2 * grid][n_mt * 128][2]   partial (running max in log2 units, running sum)
  int nl, layer_begin, batch, n_kv_heads, n_q_heads, group, capacity, q_cap;
  int rows;        // group * q_cap: query rows per unit
  int n_mt;        // M tiles per unit (1 or 2)
  int fresh_box;   // rows per TMA box of the fresh K/V tensors = min(128, q_cap)
  int whole_units; // 1: deal whole units round-robin, no partials
  float scale_log2;
  int* status;
};

// Per-block scheduling tables (shared memory).
struct Sched {
  int prefix[kMaxBatch + 1];  // prefix[b] = tiles of batch elements < b; prefix[batch] = sum
  int lc[kMaxBatch];          // clamped cache_len
  int lq[kMaxBatch];          // clamped q_len
};

struct Segment {
  int lc_layer, b, kvh;   // unit
  int Lc, Lq, n_ct, T;    // lengths, cache tiles, total tiles of the unit
  int t_begin, t_end;     // tile range of this segment
  int slot;               // partial slot, or -1 when the segment is the whole unit
};

__device__ __forceinline__ int tiles_of(int Lc, int Lq, int fresh_box) {
  if (Lq <= 0) return 0;
  return (Lc + kTileKeys - 1) / kTileKeys + (Lq + fresh_box - 1) / fresh_box;
}

// Walks the segments of block `cta`.  Identical in every role, so the roles agree on the
// sequence without communicating.
struct SegmentWalker {
  const AttnParams& p;
  const Sched& s;
  long long pos, end, range_begin;
  int unit, n_units;
  __device__ SegmentWalker(const AttnParams& p_, const Sched& s_, int cta, int n_cta) : p(p_), s(s_) {
    const long long sum = s.prefix[p.batch];
    const long long total = sum * p.nl * p.n_kv_heads;
    n_units = p.nl * p.n_kv_heads * p.batch;
    if (p.whole_units) {
      unit = cta;
      pos = end = range_begin = 0;
    } else {
      range_begin = pos = total * cta / n_cta;
      end = total * (cta + 1) / n_cta;
      unit = 0;
    }
  }
  __device__ bool next(Segment& g, int n_cta) {
    if (p.whole_units) {
      if (unit >= n_units) return false;
      const int grp = unit / p.batch;
      g.b = unit % p.batch;
      g.lc_layer = grp / p.n_kv_heads;
      g.kvh = grp % p.n_kv_heads;
      g.Lc = s.lc[g.b];
      g.Lq = s.lq[g.b];
      g.T = s.prefix[g.b + 1] - s.prefix[g.b];
      g.n_ct = (g.Lc + kTileKeys - 1) / kTileKeys;
      g.t_begin = 0;
      g.t_end = g.T;
      g.slot = -1;
      unit += n_cta;
      return true;
    }
    if (pos >= end) return false;
    const long long sum = s.prefix[p.batch];
    const int grp = (int)(pos / sum);
    const int rem = (int)(pos - (long long)grp * sum);
    int b = 0;
    while (s.prefix[b + 1] <= rem) ++b;   // batch is small; units with zero tiles are skipped
    const long long unit_start = (long long)grp * sum + s.prefix[b];
    g.b = b;
    g.lc_layer = grp / p.n_kv_heads;
    g.kvh = grp % p.n_kv_heads;
    g.Lc = s.lc[b];
    g.Lq = s.lq[b];
    g.T = s.prefix[b + 1] - s.prefix[b];
    g.n_ct = (g.Lc + kTileKeys - 1) / kTileKeys;
    g.t_begin = (int)(pos - unit_start);
    const long long room = end - unit_start;
    g.t_end = room < g.T ? (int)room : g.T;
    const bool whole = g.t_begin == 0 && g.t_end == g.T;
    g.slot = whole ? -1 : (pos == range_begin ? 2 * (int)blockIdx.x : 2 * (int)blockIdx.x + 1);
    pos = unit_start + g.t_end;
    return true;
  }
};

// Valid keys of tile t of a unit.
__device__ __forceinline__ int tile_valid(const Segment& g, int t, int fresh_box) {
  if (t < g.n_ct) return min(kTileKeys, g.Lc - t * kTileKeys);
  return min(fresh_box, g.Lq - (t - g.n_ct) * fresh_box);
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
attn_step_sm100_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kc,
                       const __grid_constant__ CUtensorMap tm_vc, const __grid_constant__ CUtensorMap tm_kn,
                       const __grid_constant__ CUtensorMap tm_vn, const AttnParams p) {
  using G = Geometry<D>;
  constexpr int KS = G::kStages;
  extern __shared__ uint8_t smem_raw[];
  __shared__ Sched sched;
  __shared__ int abort_flag;
  __shared__ int never_flag;   // stays 0: for waits that must not be cut short by an abort
  __shared__ uint32_t tmem_slot;

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sm_q = smem_base;                               // [2][kTileBytes]
  const uint32_t sm_k = sm_q + 2 * G::kTileBytes;                // [KS][kTileBytes]
  const uint32_t sm_v = sm_k + KS * G::kTileBytes;               // [KS][kTileBytes]
  const uint32_t sm_bar = sm_v + KS * G::kTileBytes;             // barriers, 8 bytes each
  const uint32_t bar_q_full = sm_bar, bar_q_empty = sm_bar + 8, bar_drain = sm_bar + 16;
  const uint32_t bar_k_full = sm_bar + 32, bar_k_empty = bar_k_full + 8 * KS;
  const uint32_t bar_v_full = bar_k_empty + 8 * KS, bar_v_empty = bar_v_full + 8 * KS;
  const uint32_t bar_s_ready = bar_v_empty + 8 * KS;             // [2]
  const uint32_t bar_p_ready = bar_s_ready + 16;                 // [2]
  const uint32_t bar_o_done = bar_p_ready + 16;                  // [2]

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  volatile int* abort_ptr = &abort_flag;

  // ---- set-up: lengths and tile prefix, barriers, TMEM
  if (tid == 0) { abort_flag = 0; never_flag = 0; }
  for (int b = tid; b < p.batch; b += kThreads) {
    int Lc = p.cache_len[b];
    int Lq = p.q_len ? p.q_len[b] : p.q_cap;
    if (Lc < 0 || Lc > p.capacity || Lq < 0 || Lq > p.q_cap) {
      dlm_set_status(p.status, DLM_ERR_CAPACITY);
      Lc = max(0, min(Lc, p.capacity));
      Lq = max(0, min(Lq, p.q_cap));
    }
    sched.lc[b] = Lc;
    sched.lq[b] = Lq;
  }
  __syncthreads();
  if (tid == 0) {
    int acc = 0;
    for (int b = 0; b < p.batch; ++b) {
      sched.prefix[b] = acc;
      acc += tiles_of(sched.lc[b], sched.lq[b], p.fresh_box);
    }
    sched.prefix[p.batch] = acc;
    mbar_init(bar_q_full, 1);
    mbar_init(bar_q_empty, 1);
    mbar_init(bar_drain, 1);
    for (int i = 0; i < KS; ++i) {
      mbar_init(bar_k_full + 8 * i, 1);
      mbar_init(bar_k_empty + 8 * i, 1);
      mbar_init(bar_v_full + 8 * i, 1);
      mbar_init(bar_v_empty + 8 * i, 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_s_ready + 8 * i, 1);
      mbar_init(bar_p_ready + 8 * i, 128);
      mbar_init(bar_o_done + 8 * i, 1);
    }
    mbar_fence_init();
    fence_proxy_async_smem();
  }
  if (warp == 9) {
    tmem_alloc(smem_u32(&tmem_slot), kTmemCols);
    tmem_relinquish();
  }
  if (warp == 8 && lane == 0) {
    prefetch_tensormap(&tm_q);
    prefetch_tensormap(&tm_kc);
    prefetch_tensormap(&tm_vc);
    prefetch_tensormap(&tm_kn);
    prefetch_tensormap(&tm_vn);
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = tmem_slot;
  const int n_cta = gridDim.x;

  if (sched.prefix[p.batch] > 0 || p.whole_units) {
    if (warp == 8) {
      // ================================================================= TMA producer
      if (lane == 0) {
        SegmentWalker walk(p, sched, blockIdx.x, n_cta);
        Segment g;
        uint32_t kt = 0, vt = 0, seg = 0;
        bool ok = true;
        while (ok && walk.next(g, n_cta)) {
          if (g.t_end <= g.t_begin) continue;
          const int zq = (g.lc_layer * p.batch + g.b) * p.n_kv_heads + g.kvh;
          const int zc = ((g.lc_layer + p.layer_begin) * p.batch + g.b) * p.n_kv_heads + g.kvh;
          if (seg > 0) ok = mbar_wait(bar_q_empty, (seg - 1) & 1, abort_ptr);
          if (!ok) break;
          const int q_box = min(128, p.rows);
          mbar_expect_tx(bar_q_full, (uint32_t)(p.n_mt * q_box) * 128u * G::kPanels);  // a box counts in full
          for (int mt = 0; mt < p.n_mt; ++mt)
            for (int pn = 0; pn < G::kPanels; ++pn)
              tma_load_3d(sm_q + mt * G::kTileBytes + pn * kPanelBytes, &tm_q, bar_q_full, pn * 64,
                          mt * 128, zq);
          for (int t = g.t_begin; t < g.t_end && ok; ++t) {
            const bool cache = t < g.n_ct;
            const int row = cache ? t * kTileKeys : (t - g.n_ct) * p.fresh_box;
            const int z = cache ? zc : zq;
            const uint32_t bytes = (uint32_t)(cache ? min(kTileKeys, p.capacity) : p.fresh_box) * 128u * G::kPanels;
            {
              const uint32_t s = kt % KS;
              if (kt >= (uint32_t)KS) ok = mbar_wait(bar_k_empty + 8 * s, ((kt / KS) - 1) & 1, abort_ptr);
              if (!ok) break;
              mbar_expect_tx(bar_k_full + 8 * s, bytes);
              for (int pn = 0; pn < G::kPanels; ++pn)
                tma_load_3d(sm_k + s * G::kTileBytes + pn * kPanelBytes, cache ? &tm_kc : &tm_kn, bar_k_full + 8 * s,
                            pn * 64, row, z);
              ++kt;
            }
            {
              const uint32_t s = vt % KS;
              if (vt >= (uint32_t)KS) ok = mbar_wait(bar_v_empty + 8 * s, ((vt / KS) - 1) & 1, abort_ptr);
              if (!ok) break;
              mbar_expect_tx(bar_v_full + 8 * s, bytes);
              for (int pn = 0; pn < G::kPanels; ++pn)
                tma_load_3d(sm_v + s * G::kTileBytes + pn * kPanelBytes, cache ? &tm_vc : &tm_vn, bar_v_full + 8 * s,
                            pn * 64, row, z);
              ++vt;
            }
          }
          ++seg;
        }
        if (!ok) {
          // unwinding: let the copies already issued land before the block's memory is released
          for (uint32_t i = (kt > (uint32_t)KS ? kt - KS : 0); i < kt; ++i)
            mbar_wait(bar_k_full + 8 * (i % KS), (i / KS) & 1, &never_flag);
          for (uint32_t i = (vt > (uint32_t)KS ? vt - KS : 0); i < vt; ++i)
            mbar_wait(bar_v_full + 8 * (i % KS), (i / KS) & 1, &never_flag);
        }
      }
    } else if (warp == 9) {
      // ================================================================== MMA issuer
      if (lane == 0) {
        SegmentWalker walk(p, sched, blockIdx.x, n_cta);
        Segment g;
        uint32_t kt = 0, vt = 0, gt = 0, seg = 0;
        bool ok = true;
        const uint32_t idesc_pv = make_idesc_bf16(128, D, 1);
        // S[mt] = Q[mt] K^T for the tile in K stage `ks`, N = n16 keys
        auto issue_s = [&](int mt, uint32_t ks, int n16) {
          const uint32_t idesc = make_idesc_bf16(128, (uint32_t)n16, 0);
          const uint32_t d = tmem + G::kColS + mt * 128;
#pragma unroll
          for (int k = 0; k < D / 16; ++k) {
            const uint32_t off = (k >> 2) * kPanelBytes + (k & 3) * 32;
            mma_ss(d, make_smem_desc_sw128(sm_q + mt * G::kTileBytes + off, 16, 1024),
                   make_smem_desc_sw128(sm_k + ks * G::kTileBytes + off, 16, 1024), idesc, k > 0 ? 1u : 0u);
          }
        };
        while (ok && walk.next(g, n_cta)) {
          const int n = g.t_end - g.t_begin;
          if (n <= 0) continue;
          ok = mbar_wait(bar_q_full, seg & 1, abort_ptr);
          if (!ok) break;
          {  // prologue: S of the first tile
            const uint32_t ks = kt % KS;
            ok = mbar_wait(bar_k_full + 8 * ks, (kt / KS) & 1, abort_ptr);
            if (!ok) break;
            tc_fence_after_sync();
            const int n16 = (tile_valid(g, g.t_begin, p.fresh_box) + 15) & ~15;
            for (int mt = 0; mt < p.n_mt; ++mt) {
              issue_s(mt, ks, n16);
              tc_commit(bar_s_ready + 8 * mt);
            }
            tc_commit(bar_k_empty + 8 * ks);
            if (n == 1) tc_commit(bar_q_empty);
            ++kt;
          }
          for (int it = 0; it < n && ok; ++it) {
            const uint32_t vs = vt % KS;
            const int n16 = (tile_valid(g, g.t_begin + it, p.fresh_box) + 15) & ~15;
            ok = mbar_wait(bar_v_full + 8 * vs, (vt / KS) & 1, abort_ptr);
            if (!ok) break;
            const bool more = it + 1 < n;
            uint32_t ks = 0;
            int n16_next = 0;
            for (int mt = 0; mt < p.n_mt && ok; ++mt) {
              ok = mbar_wait(bar_p_ready + 8 * mt, gt & 1, abort_ptr);
              if (!ok) break;
              tc_fence_after_sync();
              const uint32_t d = tmem + G::kColO + mt * D;
              const uint32_t a = tmem + G::kColS + mt * 128;
              for (int st = 0; st < n16 / 16; ++st)
                mma_ts(d, a + st * 8, make_smem_desc_sw128(sm_v + vs * G::kTileBytes + st * 2048, kPanelBytes, 1024),
                       idesc_pv, (it > 0 || st > 0) ? 1u : 0u);
              tc_commit(bar_o_done + 8 * mt);
              if (mt == p.n_mt - 1) tc_commit(bar_v_empty + 8 * vs);
              if (more) {
                if (mt == 0) {
                  ks = kt % KS;
                  ok = mbar_wait(bar_k_full + 8 * ks, (kt / KS) & 1, abort_ptr);
                  if (!ok) break;
                  tc_fence_after_sync();
                  n16_next = (tile_valid(g, g.t_begin + it + 1, p.fresh_box) + 15) & ~15;
                }
                issue_s(mt, ks, n16_next);
                tc_commit(bar_s_ready + 8 * mt);
                if (mt == p.n_mt - 1) {
                  tc_commit(bar_k_empty + 8 * ks);
                  if (it + 2 == n) tc_commit(bar_q_empty);
                  ++kt;
                }
              }
            }
            ++vt;
            ++gt;
          }
          ++seg;
        }
        // every MMA issued by this thread has finished before TMEM is released
        tc_commit(bar_drain);
        mbar_wait(bar_drain, 0, &never_flag);
      }
    } else {
      // ============================================================= softmax warpgroups
      const int mt = warp >> 2;
      if (mt < p.n_mt) {
        const int row = (warp & 3) * 32 + lane;                 // row of the M tile = TMEM lane
        const uint32_t t_lane = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t t_s = tmem + t_lane + G::kColS + mt * 128;
        const uint32_t t_o = tmem + t_lane + G::kColO + mt * D;
        const int r_unit = mt * 128 + row;                      // row within the unit
        const bool real_row = r_unit < p.rows;
        const int h_local = real_row ? r_unit / p.q_cap : 0;
        const int i_row = real_row ? r_unit % p.q_cap : 0;
        SegmentWalker walk(p, sched, blockIdx.x, n_cta);
        Segment g;
        uint32_t gt = 0;
        bool ok = true;
        uint32_t v[32];
        // the warp leaves a wait together, so the .sync.aligned TMEM instructions that follow
        // always see a converged warp, also when a wait is given up
        auto wait_warp = [&](uint32_t bar, uint32_t parity) {
          return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_ptr)) != 0;
        };
        while (ok && walk.next(g, n_cta)) {
          const int n = g.t_end - g.t_begin;
          const size_t qrow = (((size_t)g.lc_layer * p.batch + g.b) * p.n_q_heads + (size_t)g.kvh * p.group + h_local) *
                                  p.q_cap + i_row;
          if (n <= 0) {  // whole-unit mode, inactive batch element: the unit's rows are zero
            if (real_row) {
              uint4* o = reinterpret_cast<uint4*>(p.out + qrow * D);
#pragma unroll
              for (int c = 0; c < D / 8; ++c) o[c] = make_uint4(0, 0, 0, 0);
              if (p.lse) p.lse[qrow] = -CUDART_INF_F;
            }
            continue;
          }
          float m_run = -CUDART_INF_F, l_run = 0.f;
          for (int it = 0; it < n && ok; ++it, ++gt) {
            const int valid = tile_valid(g, g.t_begin + it, p.fresh_box);
            const int n16 = (valid + 15) & ~15;
            const int n_chunks = (valid + 31) >> 5;
            if (mt == 0 && valid < n16) {
              // V rows in [valid, n16) would be multiplied by P = 0: clear them so that stale
              // NaN / Inf bit patterns cannot reach O.
              const uint32_t vs = gt % KS;
              ok = wait_warp(bar_v_full + 8 * vs, (gt / KS) & 1);
              if (!ok) break;
              const int per_row = G::kPanels * 8;
              for (int idx = tid; idx < (n16 - valid) * per_row; idx += 128) {
                const int r = valid + idx / per_row, rem = idx % per_row;
                const uint32_t a = sm_v + vs * G::kTileBytes + (rem >> 3) * kPanelBytes + r * 128 + (rem & 7) * 16;
                asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(a), "r"(0u) : "memory");
              }
              fence_proxy_async_smem();
            }
            ok = wait_warp(bar_s_ready + 8 * mt, gt & 1);
            if (!ok) break;
            tc_fence_after_sync();
            // pass 1: row maximum over the valid keys of this tile
            float mx = -CUDART_INF_F;
            for (int c = 0; c < n_chunks; ++c) {
              tmem_ld32(t_s + c * 32, v);
              tmem_ld_wait();
              if (c * 32 + 32 <= valid) {
#pragma unroll
                for (int j = 0; j < 32; ++j) mx = fmaxf(mx, __uint_as_float(v[j]));
              } else {
#pragma unroll
                for (int j = 0; j < 32; ++j)
                  if (c * 32 + j < valid) mx = fmaxf(mx, __uint_as_float(v[j]));
              }
            }
            const float m_new = fmaxf(m_run, mx * p.scale_log2);
            if (it > 0 && __any_sync(0xffffffffu, m_new > m_run)) {
              // some row of this warp has a new maximum: rescale the warp's O rows in TMEM
              ok = wait_warp(bar_o_done + 8 * mt, (gt - 1) & 1);
              if (!ok) break;
              tc_fence_after_sync();
              const float alpha = ex2_approx(m_run - m_new);
#pragma unroll 1
              for (int c = 0; c < D / 32; ++c) {
                tmem_ld32(t_o + c * 32, v);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) * alpha);
                tmem_st32(t_o + c * 32, v);
              }
              l_run *= alpha;
            }
            m_run = m_new;
            // pass 2: P = 2^(s * scale - m), row sum, bf16 pairs written over S
            float l_add = 0.f;
            for (int c = 0; c < n_chunks; ++c) {
              tmem_ld32(t_s + c * 32, v);
              tmem_ld_wait();
              uint32_t pk[16];
#pragma unroll
              for (int j = 0; j < 16; ++j) {
                float p0 = ex2_approx(fmaf(__uint_as_float(v[2 * j]), p.scale_log2, -m_run));
                float p1 = ex2_approx(fmaf(__uint_as_float(v[2 * j + 1]), p.scale_log2, -m_run));
                if (c * 32 + 2 * j >= valid) p0 = 0.f;
                if (c * 32 + 2 * j + 1 >= valid) p1 = 0.f;
                const __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);
                // the sum uses the rounded values the tensor core will multiply with
                l_add += __low2float(h) + __high2float(h);
                pk[j] = *reinterpret_cast<const uint32_t*>(&h);
              }
              tmem_st16(t_s + c * 16, pk);
            }
            l_run += l_add;
            tmem_st_wait();
            tc_fence_before_sync();
            mbar_arrive(bar_p_ready + 8 * mt);
          }
          if (!ok) break;
          // ---- epilogue of the segment: O is complete once the last P V product has finished
          ok = wait_warp(bar_o_done + 8 * mt, (gt - 1) & 1);
          if (!ok) break;
          tc_fence_after_sync();
          const bool active = real_row && i_row < g.Lq;
          if (g.slot < 0) {
            const float inv = active ? 1.f / l_run : 0.f;
#pragma unroll 1
            for (int c = 0; c < D / 32; ++c) {
              tmem_ld32(t_o + c * 32, v);
              tmem_ld_wait();
              if (real_row) {
                uint4* o = reinterpret_cast<uint4*>(p.out + qrow * D + c * 32);
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                  uint32_t w[4];
#pragma unroll
                  for (int j = 0; j < 4; ++j) {
                    const float a0 = active ? __uint_as_float(v[q4 * 8 + 2 * j]) * inv : 0.f;
                    const float a1 = active ? __uint_as_float(v[q4 * 8 + 2 * j + 1]) * inv : 0.f;
                    const __nv_bfloat162 h = __floats2bfloat162_rn(a0, a1);
                    w[j] = *reinterpret_cast<const uint32_t*>(&h);
                  }
                  o[q4] = make_uint4(w[0], w[1], w[2], w[3]);
                }
              }
            }
            if (real_row && p.lse)
              p.lse[qrow] = active ? (m_run + lg2_approx(l_run)) * 0.6931471805599453f : -CUDART_INF_F;
          } else {
            const size_t prow = ((size_t)g.slot * p.n_mt + mt) * 128 + row;
#pragma unroll 1
            for (int c = 0; c < D / 32; ++c) {
              tmem_ld32(t_o + c * 32, v);
              tmem_ld_wait();
              if (real_row) {
                float4* o = reinterpret_cast<float4*>(p.ws_o + prow * D + c * 32);
#pragma unroll
                for (int q4 = 0; q4 < 8; ++q4)
                  o[q4] = make_float4(__uint_as_float(v[4 * q4]), __uint_as_float(v[4 * q4 + 1]),
                                      __uint_as_float(v[4 * q4 + 2]), __uint_as_float(v[4 * q4 + 3]));
              }
            }
            if (real_row) *reinterpret_cast<float2*>(p.ws_ml + prow * 2) = make_float2(m_run, l_run);
          }
        }
      }
    }
  }
  // ---- teardown: nothing of this block is in flight any more
  __syncwarp();
  if (tid == 0 && abort_flag) dlm_set_status(p.status, DLM_ERR_TIMEOUT);
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 9) {
    tc_fence_after_sync();
    tmem_dealloc(tmem, kTmemCols);
  }
}

// Merges the partial results of every unit that was split across blocks, in block order.
template <int D>
__global__ void __launch_bounds__(256)
attn_combine_kernel(const AttnParams p, int n_cta) {
  constexpr int E = D / 32;
  const int unit = blockIdx.x;
  const int r_unit = blockIdx.y * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (r_unit >= p.rows) return;
  const int grp = unit / p.batch, b = unit % p.batch;
  const int lc_layer = grp / p.n_kv_heads, kvh = grp % p.n_kv_heads;
  long long sum = 0, before = 0;
  int T = 0, Lq_b = 0;
  for (int bb = 0; bb < p.batch; ++bb) {
    int Lc = max(0, min(p.cache_len[bb], p.capacity));
    int Lq = max(0, min(p.q_len ? p.q_len[bb] : p.q_cap, p.q_cap));
    const int t = tiles_of(Lc, Lq, p.fresh_box);
    if (bb < b) before += t;
    if (bb == b) { T = t; Lq_b = Lq; }
    sum += t;
  }
  const int h_local = r_unit / p.q_cap, i_row = r_unit % p.q_cap;
  const size_t qrow = (((size_t)lc_layer * p.batch + b) * p.n_q_heads + (size_t)kvh * p.group + h_local) * p.q_cap + i_row;
  __nv_bfloat16* o = p.out + qrow * D + lane * E;
  const long long total = sum * p.nl * p.n_kv_heads;
  const long long u0 = (long long)grp * sum + before, u1 = u0 + T;
  int c_first = 0, c_last = 0;
  if (T > 0) {
    c_first = (int)(u0 * n_cta / total);
    while (total * (c_first + 1) / n_cta <= u0) ++c_first;
    while (total * c_first / n_cta > u0) --c_first;
    c_last = (int)((u1 - 1) * n_cta / total);
    while (total * (c_last + 1) / n_cta <= u1 - 1) ++c_last;
    while (total * c_last / n_cta > u1 - 1) --c_last;
    if (c_first == c_last) return;   // the unit was computed whole by one block
  }
  if (T == 0 || i_row >= Lq_b) {
#pragma unroll
    for (int e = 0; e < E; ++e) o[e] = __float2bfloat16(0.f);
    if (p.lse && lane == 0) p.lse[qrow] = -CUDART_INF_F;
    return;
  }
  const int mt = r_unit >> 7, row = r_unit & 127;
  float m_all = -CUDART_INF_F;
  for (int c = c_first; c <= c_last; ++c) {
    const long long r0 = total * c / n_cta;
    const long long s0 = r0 > u0 ? r0 : u0;
    if (s0 >= u1 || s0 >= total * (c + 1) / n_cta) continue;   // a block with an empty share
    const int slot = (s0 == r0) ? 2 * c : 2 * c + 1;
    m_all = fmaxf(m_all, p.ws_ml[(((size_t)slot * p.n_mt + mt) * 128 + row) * 2]);
  }
  float acc[E], l_all = 0.f;
#pragma unroll
  for (int e = 0; e < E; ++e) acc[e] = 0.f;
  for (int c = c_first; c <= c_last; ++c) {
    const long long r0 = total * c / n_cta;
    const long long s0 = r0 > u0 ? r0 : u0;
    if (s0 >= u1 || s0 >= total * (c + 1) / n_cta) continue;
    const int slot = (s0 == r0) ? 2 * c : 2 * c + 1;
    const size_t prow = ((size_t)slot * p.n_mt + mt) * 128 + row;
    const float2 ml = *reinterpret_cast<const float2*>(p.ws_ml + prow * 2);
    const float w = ex2_approx(ml.x - m_all);
    l_all += w * ml.y;
    const float* po = p.ws_o + prow * D + lane * E;
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] += w * po[e];
  }
  const float inv = 1.f / l_all;
#pragma unroll
  for (int e = 0; e < E; ++e) o[e] = __float2bfloat16(acc[e] * inv);
  if (p.lse && lane == 0) p.lse[qrow] = (m_all + lg2_approx(l_all)) * 0.6931471805599453f;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// bf16 tensor viewed as [slabs][rows][D]; box = 64 elements x box_rows rows x 1 slab, 128-byte swizzle.
int encode_map(dlm_ctx* ctx, CUtensorMap* map, const void* base, int D, long long rows, long long slabs, int box_rows) {
  if (!ctx->encode_tiled) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn ||
        q != cudaDriverEntryPointSuccess)
      return DLM_ERR_CUDA;
    ctx->encode_tiled = fn;
  }
  const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)rows, (cuuint64_t)slabs};
  const cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)rows * D * 2};
  const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  const cuuint32_t elem[3] = {1, 1, 1};
  const CUresult r = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled)(
      map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, elem,
      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? DLM_OK : DLM_ERR_CUDA;
}

struct Plan {
  int n_mt, rows, grid, whole_units;
  size_t ws_o_bytes, ws_ml_bytes;
};

Plan make_plan(const dlm_ctx* ctx, const dlm_kv_cache* cache, int nl, int n_q_heads, int q_cap) {
  Plan pl;
  pl.rows = (n_q_heads / cache->n_kv_heads) * q_cap;
  pl.n_mt = (pl.rows + 127) / 128;
  const long long units = (long long)nl * cache->batch * cache->n_kv_heads;
  pl.whole_units = units >= 8LL * ctx->num_sms ? 1 : 0;
  pl.grid = (int)(units < ctx->num_sms && pl.whole_units ? units : ctx->num_sms);
  const size_t slots = pl.whole_units ? 0 : 2 * (size_t)pl.grid;
  pl.ws_o_bytes = slots * pl.n_mt * 128 * cache->head_dim * sizeof(float);
  pl.ws_ml_bytes = slots * pl.n_mt * 128 * 2 * sizeof(float);
  return pl;
}

}  // namespace

extern "C" size_t dlm_attn_workspace_bytes(const dlm_ctx* ctx, const dlm_kv_cache* cache, int n_layers_in_call,
                                           int n_q_heads, int q_cap) {
  if (!ctx || !cache || n_layers_in_call <= 0 || n_q_heads <= 0 || q_cap <= 0 || cache->n_kv_heads <= 0 ||
      cache->batch <= 0 || n_q_heads % cache->n_kv_heads != 0)
    return 0;
  const Plan pl = make_plan(ctx, cache, n_layers_in_call, n_q_heads, q_cap);
  return pl.ws_o_bytes + pl.ws_ml_bytes + 256;
}

extern "C" int dlm_freecache_attn_step(dlm_ctx* ctx, const dlm_kv_cache* cache, int layer_begin, int layer_end,
                                       const void* q, const void* k_new, const void* v_new, int n_q_heads,
                                       int q_cap, const int32_t* q_len, float softmax_scale, int cache_len_hint,
                                       void* out, float* lse, void* workspace, size_t workspace_bytes,
                                       void* stream) {
  (void)cache_len_hint;  // the persistent schedule balances itself from the device-side lengths
  if (!ctx || !cache || !cache->k || !cache->v || !cache->cache_len || !q || !k_new || !v_new || !out)
    return DLM_ERR_NULL;
  if (cache->n_layers <= 0 || cache->batch <= 0 || cache->n_kv_heads <= 0 || cache->capacity <= 0 ||
      n_q_heads <= 0 || q_cap <= 0)
    return DLM_ERR_SHAPE;
  if (layer_begin < 0 || layer_end > cache->n_layers || layer_begin >= layer_end) return DLM_ERR_SHAPE;
  const int D = cache->head_dim;
  if (D != 64 && D != 128) return DLM_ERR_UNSUPPORTED;
  if (n_q_heads % cache->n_kv_heads != 0) return DLM_ERR_UNSUPPORTED;
  const int group = n_q_heads / cache->n_kv_heads;
  if ((long long)group * q_cap > 256 || cache->batch > kMaxBatch) return DLM_ERR_UNSUPPORTED;
  if (((uintptr_t)cache->k | (uintptr_t)cache->v | (uintptr_t)q | (uintptr_t)k_new | (uintptr_t)v_new |
       (uintptr_t)out) & 15)
    return DLM_ERR_UNSUPPORTED;
  const int nl = layer_end - layer_begin;
  const size_t need = dlm_attn_workspace_bytes(ctx, cache, nl, n_q_heads, q_cap);
  if (!workspace || workspace_bytes < need || ((uintptr_t)workspace & 255)) return DLM_ERR_WORKSPACE;
  const Plan pl = make_plan(ctx, cache, nl, n_q_heads, q_cap);

  AttnParams p;
  p.cache_len = cache->cache_len;
  p.q_len = q_len;
  p.out = static_cast<__nv_bfloat16*>(out);
  p.lse = lse;
  p.ws_o = static_cast<float*>(workspace);
  p.ws_ml = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + pl.ws_o_bytes);
  p.nl = nl;
  p.layer_begin = layer_begin;
  p.batch = cache->batch;
  p.n_kv_heads = cache->n_kv_heads;
  p.n_q_heads = n_q_heads;
  p.group = group;
  p.capacity = cache->capacity;
  p.q_cap = q_cap;
  p.rows = pl.rows;
  p.n_mt = pl.n_mt;
  p.fresh_box = q_cap < 128 ? q_cap : 128;
  p.whole_units = pl.whole_units;
  const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)D);
  p.scale_log2 = scale * 1.4426950408889634f;
  p.status = &ctx->words->status;

  CUtensorMap tm_q, tm_kc, tm_vc, tm_kn, tm_vn;
  const long long slabs_new = (long long)nl * cache->batch * cache->n_kv_heads;
  const long long slabs_cache = (long long)cache->n_layers * cache->batch * cache->n_kv_heads;
  const int cache_box = cache->capacity < 128 ? cache->capacity : 128;
  int rc = encode_map(ctx, &tm_q, q, D, pl.rows, slabs_new, pl.rows < 128 ? pl.rows : 128);
  if (rc == DLM_OK) rc = encode_map(ctx, &tm_kc, cache->k, D, cache->capacity, slabs_cache, cache_box);
  if (rc == DLM_OK) rc = encode_map(ctx, &tm_vc, cache->v, D, cache->capacity, slabs_cache, cache_box);
  if (rc == DLM_OK) rc = encode_map(ctx, &tm_kn, k_new, D, q_cap, slabs_new, p.fresh_box);
  if (rc == DLM_OK) rc = encode_map(ctx, &tm_vn, v_new, D, q_cap, slabs_new, p.fresh_box);
  if (rc != DLM_OK) return rc;

  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const long long units = slabs_new;
  if (D == 128) {
    auto kern = attn_step_sm100_kernel<128>;
    static bool configured = false;
    if (!configured) {
      DLM_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Geometry<128>::kSmemBytes));
      configured = true;
    }
    kern<<<pl.grid, kThreads, Geometry<128>::kSmemBytes, s>>>(tm_q, tm_kc, tm_vc, tm_kn, tm_vn, p);
    if (!pl.whole_units)
      attn_combine_kernel<128><<<dim3((unsigned)units, (unsigned)((pl.rows + 7) / 8)), 256, 0, s>>>(p, pl.grid);
  } else {
    auto kern = attn_step_sm100_kernel<64>;
    static bool configured = false;
    if (!configured) {
      DLM_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Geometry<64>::kSmemBytes));
      configured = true;
    }
    kern<<<pl.grid, kThreads, Geometry<64>::kSmemBytes, s>>>(tm_q, tm_kc, tm_vc, tm_kn, tm_vn, p);
    if (!pl.whole_units)
      attn_combine_kernel<64><<<dim3((unsigned)units, (unsigned)((pl.rows + 7) / 8)), 256, 0, s>>>(p, pl.grid);
  }
  return dlm_launch_ok(ctx, pl.whole_units ? 1 : 2);
}
