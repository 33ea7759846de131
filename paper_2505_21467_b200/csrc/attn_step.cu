// dlm_freecache_attn_step: attention of the active window over [cache rows ; fresh rows]
// (Sec. 3.2.1 "Windowed Re-computation"; Table 1 rows QK^T and Attention Score x Value;
// bidirectional: no causal mask).
//
// One work unit is (layer, batch element, KV head, chunk of up to 256 query rows): the g = Hq/Hkv
// query heads of a KV head, q_cap rows each, are cut into chunks of 256 rows = two 128-row M
// tiles that share every K/V tile (at the block sizes of the configs, g * q_cap <= 256: one chunk,
// K/V read from HBM once per KV head; larger windows re-read them per chunk, normally from L2;
// calls with very few units use chunks of 128 rows, one M tile, to have more units to spread).
// Keys are loaded in tiles of 128 rows, first the visible cache rows, then the fresh rows, and
// processed in half-steps of 64.
//
// Block = 12 warps (three warpgroups), one block per SM (persistent):
//   warps 0-3   softmax of M tile 0 (thread = query row = TMEM lane)
//   warps 4-7   softmax of M tile 1
//   warp  8     TMA producer (one lane): Q once per segment, K and V tiles through two rings
//   warp  9/10  tcgen05.mma issuer of M tile 0 / 1 (one elected lane each): S = Q K^T into one of two
//               64-column score buffers in TMEM, two half-steps ahead of the softmax; then
//               O += P V with P read from TMEM (it overwrites S in place as packed bf16)
//   warp  11    publisher (one lane): makes a finished partial result visible device-wide and
//               bumps its unit's counter, so the softmax warps need not wait for that
// Online softmax in fp32 with base-2 exponentials; a half-step's scores sit in registers; O stays
// in TMEM and is rescaled only when a row's scores have outgrown the maximum in use by a lot.
//
// Scheduling.  Every (unit, key tile) pair is one item of a global list; block c takes the
// contiguous share [c*T/G, (c+1)*T/G) of it.  A share covers whole units (result written
// directly) and at most two partial units (unnormalised O, running max and sum written to the
// workspace).  A block walks its share from the end to the start, so the piece at the start of a
// share (the last piece of its unit) is the last thing the block computes; that block merges the
// unit: it waits for the counter the other pieces' blocks bump after publishing their partial
// results (they have lower block indices and computed those pieces first), then folds them into
// its own O, which is still in TMEM, in block order: the result is deterministic.  When the split
// would cost more than it saves (the host estimates both) units are dealt whole, round-robin.
#include <cuda.h>
#include <cuda_bf16.h>
#include <math_constants.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace {

using namespace sm100;

constexpr int kThreads = 384;          // 3 warpgroups: two of softmax warps, one with the producer and the MMA issuers
constexpr int kTileKeys = 128;
constexpr int kPanelBytes = 128 * 128;   // one 64-element-wide panel of a 128-row tile
constexpr int kMaxBatch = 1024;
constexpr int kTmemCols = 512;
constexpr int kRegsSoftmax = 216;     // registers per thread of the softmax warpgroups after setmaxnreg.inc
constexpr int kRegsOther = 72;        // ... of the producer / MMA warpgroup after setmaxnreg.dec
constexpr int kMaxQCap = 4096;         // active rows per call
constexpr double kTeamMergeTiles = 3.0;   // cost of the team schedule's exchange and reduction per M tile, in key tiles
                                          // (measured: about 5 us from the last MMA to the output stores, a key tile 1.7 us)
constexpr int kTeamMax = 16;              // most blocks of a team
constexpr int kMaxGrid = 256;          // blocks of the persistent grid (one per SM)
constexpr int kMaxStages = 8;          // barrier slots reserved per ring
constexpr int kBarrierBytes = 512;     // mbarriers of a block
constexpr int kFlagBytes = 64;         // abort / never flags, TMEM slot, merge flag

template <int D>
struct Geometry {
  static constexpr int kPanels = D / 64;
  static constexpr int kTileBytes = kPanels * kPanelBytes;      // one K tile, V tile or Q M-tile
  static constexpr int kStages = (D == 128) ? 2 : 4;            // ring depth of K and of V
  static constexpr uint32_t kColO = 0;                          // O[mt] at mt * D
  static constexpr uint32_t kColS = 2 * D;                      // S[mt] at 2D + mt * 128 (P aliases it)
};

struct AttnParams {
  const int32_t* cache_len;
  const int32_t* q_len;
  __nv_bfloat16* out;
  float* lse;
  float* ws_o;    // [2 * grid][n_mt][D/4][128][4]  partial unnormalised O: 4 columns of a row per 16-byte vector
  float* ws_ml;   // [2 * grid][n_mt][128][2]    partial (running max in log2 units, running sum)
  int nl, layer_begin, batch, n_kv_heads, n_q_heads, group, capacity, q_cap;
  int rows_total;  // group * q_cap: query rows per (layer, batch element, KV head)
  int n_rc;        // row chunks: rows_total cut into units of up to 256 rows (each re-reads the K/V tiles)
  int rows;        // query rows per unit = min(chunk_rows, rows_total)
  int chunk_rows;  // 256 (two M tiles share every K/V tile) or 128 (one M tile per unit)
  int n_mt;        // M tiles per unit (1 or 2)
  int fresh_box;   // rows per TMA box of the fresh K/V tensors = min(128, q_cap)
  int whole_units; // 1: deal whole units round-robin, no partials
  int team;        // > 1 (with whole_units): blocks [u * team, (u + 1) * team) share unit u, key tiles dealt by rank;
                   // every block then reduces its share of the unit's outputs over all the team's pieces
  int smem_bytes;           // dynamic shared memory of the launch
  float scale_log2;
  int* status;
  unsigned int* tickets;   // one zero-initialised counter per unit: pieces finished
};

// Per-block scheduling tables (in the block's dynamic shared memory, sized by batch and grid).
struct Sched {
  int* prefix;    // [batch + 1]  prefix[b] = tiles of batch elements < b; prefix[batch] = sum
  int* lc;        // [batch]      clamped cache_len
  int* lq;        // [batch]      clamped q_len
  int* share_lo;  // [grid + 1]   split mode: block c owns items [share_lo[c], share_lo[c + 1])
};
__host__ __device__ inline int sched_ints(int batch, int grid) { return 3 * (batch + 1) + 2 * (grid + 1); }

struct Segment {
  int lc_layer, b, kvh, rc;   // unit: layer within the call, batch element, KV head, row chunk
  int Lc, Lq, n_ct, T;    // lengths, cache tiles, total tiles of the unit
  int t_begin, t_end;     // tile range of this segment
  int slot;               // partial slot; -1 when the segment is the whole unit; -2 for a piece of the team schedule
  int merger;             // partial segment holding the unit's last tile: this block merges the unit
};

__device__ __forceinline__ int tiles_of(int Lc, int Lq, int fresh_box) {
  if (Lq <= 0) return 0;
  return (Lc + kTileKeys - 1) / kTileKeys + (Lq + fresh_box - 1) / fresh_box;
}

// Walks the segments of block `cta`.  Identical in every role, so the roles agree on the
// sequence without communicating.  Item counts fit 32 bits (the host refuses larger launches).
struct SegmentWalker {
  const AttnParams& p;
  const Sched& s;
  int end, range_begin;   // split mode: items [range_begin, end) are still to do
  int unit, n_units;
  __device__ SegmentWalker(const AttnParams& p_, const Sched& s_, int cta) : p(p_), s(s_) {
    n_units = p.nl * p.n_kv_heads * p.n_rc * p.batch;
    if (p.whole_units) {
      unit = p.team > 1 ? cta / p.team : cta;
      end = range_begin = 0;
    } else {
      range_begin = s.share_lo[cta];
      end = s.share_lo[cta + 1];
      unit = 0;
    }
  }
  __device__ bool next(Segment& g, int n_cta) {
    if (p.whole_units) {
      if (unit >= n_units) return false;
      const int grp = unit / p.batch;
      g.b = unit % p.batch;
      g.rc = grp % p.n_rc;
      g.lc_layer = (grp / p.n_rc) / p.n_kv_heads;
      g.kvh = (grp / p.n_rc) % p.n_kv_heads;
      g.Lc = s.lc[g.b];
      g.Lq = s.lq[g.b];
      g.T = s.prefix[g.b + 1] - s.prefix[g.b];
      g.n_ct = (g.Lc + kTileKeys - 1) / kTileKeys;
      g.t_begin = 0;
      g.t_end = g.T;
      g.slot = -1;
      g.merger = 0;
      if (p.team > 1) {   // this block's share of the unit's key tiles; the launch has one team per unit
        const int rank = (int)blockIdx.x % p.team;
        g.t_begin = g.T * rank / p.team;
        g.t_end = g.T * (rank + 1) / p.team;
        g.slot = -2;
        unit = n_units;
        return true;
      }
      unit += n_cta;
      return true;
    }
    // split mode: from the end of the share towards its start
    if (end <= range_begin) return false;
    const int sum = s.prefix[p.batch];
    const int item = end - 1;
    const int grp = item / sum;
    const int rem = item - grp * sum;
    int b = 0;
    while (s.prefix[b + 1] <= rem) ++b;   // batch is small; units with zero tiles are skipped
    const int unit_start = grp * sum + s.prefix[b];
    g.b = b;
    g.rc = grp % p.n_rc;
    g.lc_layer = (grp / p.n_rc) / p.n_kv_heads;
    g.kvh = (grp / p.n_rc) % p.n_kv_heads;
    g.Lc = s.lc[b];
    g.Lq = s.lq[b];
    g.T = s.prefix[b + 1] - s.prefix[b];
    g.n_ct = (g.Lc + kTileKeys - 1) / kTileKeys;
    const int seg_lo = unit_start > range_begin ? unit_start : range_begin;
    g.t_begin = seg_lo - unit_start;
    g.t_end = end - unit_start;
    const bool whole = g.t_begin == 0 && g.t_end == g.T;
    g.slot = whole ? -1 : (seg_lo == range_begin ? 2 * (int)blockIdx.x : 2 * (int)blockIdx.x + 1);
    g.merger = (!whole && g.t_end == g.T) ? 1 : 0;
    end = seg_lo;
    return true;
  }
};

// Valid keys of tile t of a unit.
__device__ __forceinline__ int tile_valid(const Segment& g, int t, int fresh_box) {
  if (t < g.n_ct) return min(kTileKeys, g.Lc - t * kTileKeys);
  return min(fresh_box, g.Lq - (t - g.n_ct) * fresh_box);
}

// The blocks whose shares overlap the unit of segment g (this block is one of them), and where
// each of them left its partial result.
struct UnitPieces {
  const Sched& s;
  int u0, u1, c_first, c_last;
  __device__ UnitPieces(const AttnParams& p, const Sched& s_, const Segment& g, int cta) : s(s_) {
    const int sum = s.prefix[p.batch];
    u0 = ((g.lc_layer * p.n_kv_heads + g.kvh) * p.n_rc + g.rc) * sum + s.prefix[g.b];
    u1 = u0 + g.T;
    c_first = c_last = cta;
    while (s.share_lo[c_first] > u0) --c_first;
    while (s.share_lo[c_last + 1] < u1) ++c_last;
  }
  // slot of the piece computed by block c (c_first <= c <= c_last): the block's first segment
  // if the piece starts where the block's share starts, else its second one
  __device__ __forceinline__ int slot_of(int c) const { return s.share_lo[c] >= u0 ? 2 * c : 2 * c + 1; }
};

// Waits until the counter at `addr` reaches `target` (acquire, device scope).  Bounded like the
// mbarrier waits: gives up after the same wall-time limit or when the block is aborting.
__device__ __forceinline__ bool wait_counter(const unsigned int* addr, unsigned int target, volatile int* abort_flag,
                                             uint64_t limit_ns) {
  const uint64_t t0 = global_timer_ns();
  for (uint32_t spin = 1;; ++spin) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(addr) : "memory");
    if (v >= target) return true;
    if ((spin & 15u) == 0u) {
      if (*abort_flag) return false;
      if (global_timer_ns() - t0 > limit_ns) {
        *abort_flag = 1;
        return false;
      }
    }
  }
}

// Team schedule: what a block of a team works on after its share of the key tiles.  The team's pieces lie
// in the workspace as [rank][M tile][head_dim / 4][128 rows] 16-byte vectors (4 columns of a row) and
// [rank][M tile][128 rows] (m, l) pairs; the unit's n_mt * head_dim / 4 * 128 output vectors are dealt to
// the ranks in that storage order, rank r reducing vectors [lo, hi) over all pieces.
// The launch parameters the team schedule's exchange needs, handed to its functions by value.
struct TeamArgs {
  __nv_bfloat16* out;
  float* lse;
  float* ws_o;
  float* ws_ml;
  unsigned int* tickets;
  int team, n_mt, batch, n_rc, n_kv_heads, n_q_heads, group, q_cap, rows, rows_total;
  __device__ explicit TeamArgs(const AttnParams& p)
      : out(p.out), lse(p.lse), ws_o(p.ws_o), ws_ml(p.ws_ml), tickets(p.tickets), team(p.team), n_mt(p.n_mt),
        batch(p.batch), n_rc(p.n_rc), n_kv_heads(p.n_kv_heads), n_q_heads(p.n_q_heads), group(p.group), q_cap(p.q_cap),
        rows(p.rows), rows_total(p.rows_total) {}
};

struct TeamShare {
  int rank, unit, b, rc, lc_layer, kvh, lo, hi;
  bool has_keys;
  size_t piece0;               // index of the team's first piece
  uint32_t ml_bytes, o_bytes;  // bytes fetched from each piece: all its (m, l) rows; this block's share of its vectors
  __device__ TeamShare(const TeamArgs& p, const int* prefix, int D) {
    const int C = p.team;
    rank = (int)blockIdx.x % C;
    unit = (int)blockIdx.x / C;
    b = unit % p.batch;
    const int grp = unit / p.batch;
    rc = grp % p.n_rc;
    lc_layer = (grp / p.n_rc) / p.n_kv_heads;
    kvh = (grp / p.n_rc) % p.n_kv_heads;
    has_keys = prefix[b + 1] > prefix[b];
    const int n_vec = p.n_mt * (D / 4) * 128;
    lo = n_vec * rank / C;          // n_vec <= 8192, C <= 16
    hi = n_vec * (rank + 1) / C;
    piece0 = (size_t)unit * C * p.n_mt;
    ml_bytes = (uint32_t)p.n_mt * 128u * 8u;
    o_bytes = (uint32_t)(hi - lo) * 16u;
  }
};

// The two halves of the team schedule's exchange are functions of their own, not inlined: they run once per
// launch, and inlined they changed the register allocation of the kernel's main loops (measured: 2 - 3 % on the
// layer-batched calls, which never run them).
//
// Publisher warp, one thread: once every softmax thread of this block has stored its row of the block's piece
// (bar_pub), count the block in the unit's arrival counter; when the whole team has arrived, fetch this
// block's share of every piece, and every piece's (m, l) rows, into the shared memory the Q, K and V buffers no
// longer need (all of the block's MMAs have finished by then: every softmax thread waited for its last one).
// bar_team = bar_pub + 8 completes when all of it has landed.
template <int D, bool kNoWait>
__device__ __noinline__ void team_publish(const TeamArgs p, const int* prefix, uint32_t sm_q, uint32_t bar_pub,
                                          volatile int* abort_ptr) {
  constexpr uint64_t kLimit = kNoWait ? 0ull : kWaitLimitNs;
  const uint32_t bar_team = bar_pub + 8;
  const TeamShare ts(p, prefix, D);
  if (!ts.has_keys || !mbar_wait_limit(bar_pub, 0, abort_ptr, kLimit)) return;
  unsigned int* const arrive = p.tickets + ts.unit;
  unsigned int* const depart = p.tickets + kDlmMaxSplitUnits / 2 + ts.unit;
  __threadfence();
  atomicAdd(arrive, 1u);
  if (!wait_counter(arrive, (unsigned int)p.team, abort_ptr, kLimit)) return;
  fence_proxy_async_all();
  mbar_expect_tx(bar_team, (uint32_t)p.team * (ts.ml_bytes + ts.o_bytes));
  for (int c = 0; c < p.team; ++c) {
    bulk_load(sm_q + c * ts.ml_bytes, p.ws_ml + (ts.piece0 + (size_t)c * p.n_mt) * 256, ts.ml_bytes, bar_team);
    bulk_load(sm_q + p.team * ts.ml_bytes + c * ts.o_bytes,
              p.ws_o + ((ts.piece0 + (size_t)c * p.n_mt) * (size_t)(D / 4 * 128) + ts.lo) * 4, ts.o_bytes, bar_team);
  }
  // every block of the team is past its wait on the arrival counter when the last one gets here: the last
  // one clears both counters for the next launch
  if (atomicAdd(depart, 1u) == (unsigned int)p.team - 1u) {
    *arrive = 0;
    *depart = 0;
  }
  // the copies issued above land in this block's shared memory: this thread does not leave before they have (the
  // softmax threads wait on the same barrier, but may have given up); abort_ptr + 1 is the flag that stays 0
  mbar_wait(bar_team, 0, abort_ptr + 1);
}

// Softmax threads (all live ones of the block, whole warps): store this thread's row of the block's piece --
// unnormalised O from TMEM at t_o if the block had key tiles, and (m, l), which is (-inf, 0) if it had none
// (that piece's O is then never read) -- then wait for the publisher's fetch and reduce this block's share of
// the unit's output vectors over the C pieces, in rank order.  Returns false when a wait was given up.
template <int D, int kChunk, bool kNoWait>
__device__ __noinline__ bool team_exchange(const TeamArgs p, const int* prefix, uint32_t sm_q, uint32_t bar_pub,
                                           volatile int* abort_ptr, uint32_t t_o, bool has_tiles, float m_used, float l_run) {
  constexpr uint64_t kLimit = kNoWait ? 0ull : kWaitLimitNs;
  constexpr int kVecs = D / 4 * 128;          // vectors of one M tile's piece
  const int tid = threadIdx.x, warp = tid >> 5;
  const int mt = warp >> 2, row = tid & 127;
  const int n_live = (p.rows + 31) & ~31;
  const uint32_t bar_team = bar_pub + 8;
  const TeamShare ts(p, prefix, D);
  const int C = p.team;
  const int Lq = prefix[p.batch + 1 + p.batch + ts.b];   // the clamped q_len table follows the prefix and cache_len tables
  {
    const size_t mine = ts.piece0 + (size_t)ts.rank * p.n_mt + mt;
    if (has_tiles) {
      float4* po = reinterpret_cast<float4*>(p.ws_o) + mine * (size_t)kVecs + row;
      uint32_t v[32];
#pragma unroll 1
      for (int c = 0; c < D / 32; ++c) {
        tmem_ld32(t_o + c * 32, v);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 8; ++j)
          __stcg(po + (c * 8 + j) * 128, make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                                     __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3])));
      }
    }
    __stcg(reinterpret_cast<float2*>(p.ws_ml) + mine * 128 + row, make_float2(m_used, l_run));
  }
  // no fence here: the arrival below orders the stores before the publisher's wait (block scope), and the
  // publisher's fence before it counts the block in carries them to device scope
  mbar_arrive(bar_pub);
  if (__all_sync(0xffffffffu, mbar_wait_limit(bar_team, 0, abort_ptr, kLimit)) == 0) return false;
  const uint32_t sm_ml = sm_q, sm_o = sm_q + C * ts.ml_bytes;
  for (int i = ts.lo + tid; i < ts.hi; i += n_live) {
    const int mt_i = i / kVecs, rem = i % kVecs, qd = rem / 128, row_i = rem % 128;
    const int r_unit_i = mt_i * 128 + row_i;
    const int r_kv_i = ts.rc * kChunk + r_unit_i;
    if (r_unit_i >= n_live || r_kv_i >= p.rows_total) continue;
    const int hl = r_kv_i / p.q_cap, ir = r_kv_i % p.q_cap;
    const size_t qrow_i = (((size_t)ts.lc_layer * p.batch + ts.b) * p.n_q_heads + (size_t)ts.kvh * p.group + hl) * p.q_cap + ir;
    const bool active_i = ir < Lq;
    const uint32_t a_ml = sm_ml + (uint32_t)r_unit_i * 8u, a_o = sm_o + (uint32_t)(i - ts.lo) * 16u;
    float m_all = -CUDART_INF_F;
#pragma unroll 4
    for (int c = 0; c < C; ++c) {
      const float2 ml = ld_shared_f2(a_ml + c * ts.ml_bytes);
      if (ml.y > 0.f) m_all = fmaxf(m_all, ml.x);
    }
    float l_all = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
    for (int c = 0; c < C; ++c) {
      const float2 ml = ld_shared_f2(a_ml + c * ts.ml_bytes);
      const float4 x = ld_shared_f4(a_o + c * ts.o_bytes);
      if (ml.y > 0.f) {   // a piece without keys holds no O
        const float w = ex2_approx(ml.x - m_all);
        l_all = fmaf(w, ml.y, l_all);
        acc.x = fmaf(w, x.x, acc.x);
        acc.y = fmaf(w, x.y, acc.y);
        acc.z = fmaf(w, x.z, acc.z);
        acc.w = fmaf(w, x.w, acc.w);
      }
    }
    const float inv = active_i ? 1.f / l_all : 0.f;
    const __nv_bfloat162 h0 = __floats2bfloat162_rn(active_i ? acc.x * inv : 0.f, active_i ? acc.y * inv : 0.f);
    const __nv_bfloat162 h1 = __floats2bfloat162_rn(active_i ? acc.z * inv : 0.f, active_i ? acc.w * inv : 0.f);
    *reinterpret_cast<uint2*>(p.out + qrow_i * D + qd * 4) =
        make_uint2(*reinterpret_cast<const uint32_t*>(&h0), *reinterpret_cast<const uint32_t*>(&h1));
    if (qd == 0 && p.lse) p.lse[qrow_i] = active_i ? (m_all + lg2_approx(l_all)) * 0.6931471805599453f : -CUDART_INF_F;
  }
  __syncwarp();
  return true;
}

// A key tile is processed in half-steps of up to 64 keys.  Each M tile has two 64-column score
// buffers in TMEM used alternately, so the scores of the half-step after next are computed by the
// tensor pipe while the softmax warps work on the current one: they never wait for scores in the
// steady state.  All roles enumerate the half-steps of a segment with this iterator.
constexpr int kHalfKeys = 64;
struct HalfStep {
  int t;          // key tile
  int k0;         // first key of the half-step within the tile (0 or 64)
  int nkeys;      // valid keys (1..64)
  bool first_of_tile, last_of_tile;
};
struct HalfIter {
  const Segment& g;
  int fresh_box, t, h;
  __device__ HalfIter(const Segment& g_, int fresh_box_) : g(g_), fresh_box(fresh_box_), t(g_.t_begin), h(0) {}
  __device__ __forceinline__ bool get(HalfStep& s) const {
    if (t >= g.t_end) return false;
    const int valid = tile_valid(g, t, fresh_box);
    s.t = t;
    s.k0 = h * kHalfKeys;
    s.nkeys = min(kHalfKeys, valid - s.k0);
    s.first_of_tile = (h == 0);
    s.last_of_tile = (h == 1) || valid <= kHalfKeys;
    return true;
  }
  __device__ __forceinline__ void advance(const HalfStep& s) {
    if (s.last_of_tile) { ++t; h = 0; } else { h = 1; }
  }
};

// Softmax of one half-step for the query row held by this thread (S row in TMEM -> P row in TMEM).
// O is rescaled only when the scores have outgrown the maximum in use by a lot: until then P is
// formed against the older, smaller maximum and may exceed 1 by a few powers of two, which bf16
// and the fp32 accumulators hold just as well; the final division by the row sum, taken against
// the same maximum, cancels it.  Ragged half-steps compare maxima (kRescaleThreshold, log2 units);
// full ones look at the row sum (kSumLimit).
constexpr float kRescaleThreshold = 8.0f;

// Rare path shared by both kinds of half-step: some row of the warp outgrew its maximum by more
// than the threshold, so the warp's O rows in TMEM are rescaled (rows that did not grow keep
// factor 1).  The P V product of the previous half-step may still be running: wait for it first.
template <int D>
__device__ __noinline__ bool rescale_o(uint32_t t_o, bool grow, float m_new, float& m_used, float& l_run,
                                       uint32_t bar_pv_done, uint32_t parity, volatile int* abort_ptr) {
  const bool ok = __all_sync(0xffffffffu, mbar_wait(bar_pv_done, parity, abort_ptr)) != 0;
  if (!ok) return false;
  tc_fence_after_sync();
  const float alpha = grow ? ex2_approx(m_used - m_new) : 1.0f;
  uint32_t v[32];
#pragma unroll 1
  for (int c = 0; c < D / 32; ++c) {
    tmem_ld32(t_o + c * 32, v);
    tmem_ld_wait();
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) * alpha);
    tmem_st32(t_o + c * 32, v);
  }
  tmem_st_wait();
  l_run *= alpha;
  if (grow) m_used = m_new;
  return true;
}

// Full half-step (64 valid keys): the score row sits in registers, so TMEM is read once and with a
// single wait.  Only the first half-step of a segment takes the row maximum before the
// exponentials; later ones form P against the maximum in use and look at the row sum afterwards:
// a sum above kSumLimit means some score outgrew that maximum by a lot, and only then (rare)
// is the maximum taken, O rescaled and P formed again.  The maximum pass, half-rate ALU work
// that both softmax groups of an SMSP would do at the same time, is gone from the steady state.
constexpr float kSumLimit = 1024.0f;   // 64 keys: some P is then above 16, and none was above 1024 before

template <int D>
__device__ __forceinline__ float row_max64(const uint32_t (&s)[64]) {
  float mx[8];   // independent chains: the maximum is latency-bound otherwise
#pragma unroll
  for (int c = 0; c < 8; ++c) mx[c] = __uint_as_float(s[c]);
#pragma unroll
  for (int j = 8; j < 64; j += 8) {
#pragma unroll
    for (int c = 0; c < 8; ++c) mx[c] = fmaxf(mx[c], __uint_as_float(s[j + c]));
  }
  return fmaxf(fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])), fmaxf(fmaxf(mx[4], mx[5]), fmaxf(mx[6], mx[7])));
}

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// P = 2^(s * scale - m) for 32 scores, packed to bf16 pairs and written to 16 TMEM columns at t_p;
// adds to the two partial row sums.  (Variants measured in the kernel and found no faster at the
// configs' shapes: all 32 exponentials issued before the sums, and packing by integer add and byte
// permute instead of the conversion instruction, which shares the SFU's pipe.)
__device__ __forceinline__ void exp32_store(const uint32_t* s, float scale_log2, float m_used, uint32_t t_p, float& l0,
                                            float& l1) {
  uint32_t pk[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const float p0 = ex2_approx(fmaf(__uint_as_float(s[2 * j]), scale_log2, -m_used));
    const float p1 = ex2_approx(fmaf(__uint_as_float(s[2 * j + 1]), scale_log2, -m_used));
    l0 += p0;
    l1 += p1;
    pk[j] = pack_bf16(p0, p1);
  }
  tmem_st16(t_p, pk);
}

// The same for 64 scores (32 TMEM columns at t_p); returns the row sum.
__device__ __forceinline__ float exp64_store(const uint32_t (&s)[64], float scale_log2, float m_used, uint32_t t_p) {
  float l0 = 0.f, l1 = 0.f;
  exp32_store(s, scale_log2, m_used, t_p, l0, l1);
  exp32_store(s + 32, scale_log2, m_used, t_p + 16, l0, l1);
  return l0 + l1;
}

template <int D>
__device__ __forceinline__ bool softmax_half_full(uint32_t t_s, uint32_t t_o, bool first, float scale_log2,
                                                  float& m_used, float& l_run, uint32_t bar_pv_done,
                                                  uint32_t pv_parity, volatile int* abort_ptr) {
  uint32_t s[64];
  tmem_ld32(t_s, s);
  tmem_ld32(t_s + 32, s + 32);
  tmem_ld_wait();
  if (first) {
    m_used = row_max64<D>(s) * scale_log2;
    l_run = 0.f;
  }
  float l_half = exp64_store(s, scale_log2, m_used, t_s);
  if (!first) {
    const bool grow = !(l_half <= kSumLimit);   // also catches a NaN sum
    if (__any_sync(0xffffffffu, grow)) {
      const float m_new = row_max64<D>(s) * scale_log2;
      tmem_st_wait();   // the P just written is replaced below
      if (!rescale_o<D>(t_o, grow, m_new, m_used, l_run, bar_pv_done, pv_parity, abort_ptr)) return false;
      l_half = exp64_store(s, scale_log2, m_used, t_s);
    }
  }
  l_run += l_half;
  tmem_st_wait();
  return true;
}

// Ragged half-step (fewer than 64 valid keys: the end of the cache rows, or the fresh rows): 32
// columns at a time, keys at or beyond `valid` masked out.
template <int D>
__device__ __noinline__ bool softmax_half_ragged(uint32_t t_s, uint32_t t_o, int valid, bool first, float scale_log2,
                                                 float& m_used, float& l_run, uint32_t bar_pv_done,
                                                 uint32_t pv_parity, volatile int* abort_ptr) {
  const int n_chunks = (valid + 31) >> 5;
  uint32_t v[32];
  float mx = -CUDART_INF_F;
  for (int c = 0; c < n_chunks; ++c) {
    tmem_ld32(t_s + c * 32, v);
    tmem_ld_wait();
#pragma unroll
    for (int j = 0; j < 32; ++j)
      if (c * 32 + j < valid) mx = fmaxf(mx, __uint_as_float(v[j]));
  }
  const float m_new = mx * scale_log2;
  if (first) {
    m_used = m_new;
    l_run = 0.f;
  } else {
    const bool grow = m_new > m_used + kRescaleThreshold;
    if (__any_sync(0xffffffffu, grow)) {
      if (!rescale_o<D>(t_o, grow, m_new, m_used, l_run, bar_pv_done, pv_parity, abort_ptr)) return false;
    }
  }
  float l_add = 0.f;
  for (int c = 0; c < n_chunks; ++c) {
    tmem_ld32(t_s + c * 32, v);
    tmem_ld_wait();
    uint32_t pk[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      float p0 = ex2_approx(fmaf(__uint_as_float(v[2 * j]), scale_log2, -m_used));
      float p1 = ex2_approx(fmaf(__uint_as_float(v[2 * j + 1]), scale_log2, -m_used));
      if (c * 32 + 2 * j >= valid) p0 = 0.f;
      if (c * 32 + 2 * j + 1 >= valid) p1 = 0.f;
      l_add += p0 + p1;
      pk[j] = pack_bf16(p0, p1);
    }
    tmem_st16(t_s + c * 16, pk);
  }
  l_run += l_add;
  tmem_st_wait();
  return true;
}

// kNoWait = true is the instantiation a test selects to run the give-up path: every wait on work still to come tests
// its barrier once and gives up if the data is not there yet (waits that let issued copies and MMAs finish keep the
// 2 s limit).  The limit is a compile-time constant because the waits sit on the critical path of the MMA issuers
// (a run-time limit cost 2 % at the Dream shape).
template <int D, int kChunk, bool kNoWait>
__global__ void __launch_bounds__(kThreads, 1)
attn_step_sm100_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kc,
                       const __grid_constant__ CUtensorMap tm_vc, const __grid_constant__ CUtensorMap tm_kn,
                       const __grid_constant__ CUtensorMap tm_vn, const AttnParams p) {
  using G = Geometry<D>;
  constexpr uint64_t kLimit = kNoWait ? 0ull : kWaitLimitNs;
  // Shared memory of the block, all of it dynamic (the scheduling tables are sized by batch and grid):
  // [Q: n_mt tiles][K ring][V ring][barriers][flags][scheduling tables], from the first 1024-byte
  // boundary (the swizzled tiles need that alignment).
  extern __shared__ uint8_t smem_raw[];
  // compile-time ring depths: the MMA issuers' scalar code is on the critical path, and divisions by a
  // run-time depth in it cost 10 % at the LLaDA shape
  constexpr int KS = G::kStages, VS = G::kStages;
  const uint32_t smem_pad = (1024u - (smem_u32(smem_raw) & 1023u)) & 1023u;
  const uint32_t smem_base = smem_u32(smem_raw) + smem_pad;
  const uint32_t sm_q = smem_base;                               // [n_mt][kTileBytes]
  const uint32_t sm_k = sm_q + p.n_mt * G::kTileBytes;           // [KS][kTileBytes]
  const uint32_t sm_v = sm_k + KS * G::kTileBytes;               // [VS][kTileBytes]
  const uint32_t sm_bar = sm_v + VS * G::kTileBytes;             // barriers, 8 bytes each
  int* const flags = reinterpret_cast<int*>(smem_raw + smem_pad + (size_t)(p.n_mt + KS + VS) * G::kTileBytes + kBarrierBytes);
  volatile int* const abort_ptr = flags;        // raised by the first wait that gives up
  volatile int* const never_ptr = flags + 1;    // stays 0: for waits that must not be cut short by an abort
  uint32_t* const tmem_slot = reinterpret_cast<uint32_t*>(flags + 2);
  volatile int* const merge_ok = flags + 3;
  Sched sched;
  sched.prefix = flags + kFlagBytes / 4;
  sched.lc = sched.prefix + p.batch + 1;
  sched.lq = sched.lc + p.batch;
  sched.share_lo = sched.lq + p.batch;
  if (smem_pad + (uint32_t)(p.n_mt + KS + VS) * G::kTileBytes + kBarrierBytes + kFlagBytes +
          4u * (uint32_t)sched_ints(p.batch, gridDim.x) > (uint32_t)p.smem_bytes) {
    // cannot happen with the host's sizing (it leaves room for the largest pad); nothing has been touched yet
    if (threadIdx.x == 0) dlm_set_status(p.status, DLM_ERR_WORKSPACE);
    return;
  }

  const uint32_t bar_q_full = sm_bar, bar_q_empty = sm_bar + 8, bar_drain = sm_bar + 16;   // drain: [2]
  const uint32_t bar_k_full = sm_bar + 32, bar_k_empty = bar_k_full + 8 * kMaxStages;
  const uint32_t bar_v_full = bar_k_empty + 8 * kMaxStages, bar_v_empty = bar_v_full + 8 * kMaxStages;
  const uint32_t bar_s_ready = bar_v_empty + 8 * kMaxStages;             // [M tile][score buffer]: scores of a half-step written
  const uint32_t bar_p_ready = bar_s_ready + 32;                 // [M tile][score buffer]: P of a half-step written
  const uint32_t bar_pv_done = bar_p_ready + 32;                 // [M tile][half-step parity] P V product finished.  Two P V
                                                                 // products can be in flight, so consecutive half-steps use different
                                                                 // barriers: a parity wait cannot tell phases two apart
  const uint32_t bar_pub = bar_pv_done + 32;                     // partial result of a segment stored by every softmax thread
  const uint32_t bar_team = bar_pub + 8;                         // team schedule: the team's pieces of this block's share have landed

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // softmax threads that own a real query row, rounded up to whole warps (they are tid 0 .. n_live-1)
  const int n_live = (p.rows + 31) & ~31;

  // ---- set-up: barriers, TMEM and descriptor prefetch first (they need no data), so that they overlap
  // the cold read of the lengths; then the tile prefix
  if (tid == 0) {
    *abort_ptr = 0; *never_ptr = 0; *merge_ok = 0;
    mbar_init(bar_q_full, 1);
    mbar_init(bar_q_empty, (uint32_t)p.n_mt);       // one commit per MMA issuer
    mbar_init(bar_drain, 1);
    mbar_init(bar_drain + 8, 1);
    mbar_init(bar_pub, (uint32_t)n_live);
    mbar_init(bar_team, 1);
    for (int i = 0; i < KS; ++i) {
      mbar_init(bar_k_full + 8 * i, 1);
      mbar_init(bar_k_empty + 8 * i, (uint32_t)p.n_mt);
    }
    for (int i = 0; i < VS; ++i) {
      mbar_init(bar_v_full + 8 * i, 1);
      mbar_init(bar_v_empty + 8 * i, (uint32_t)p.n_mt);
    }
    for (int i = 0; i < 2; ++i) {
      const uint32_t live_i = (uint32_t)max(32, min(128, n_live - 128 * i)) / 32;   // one arrival per live warp
      for (int u = 0; u < 2; ++u) {
        mbar_init(bar_s_ready + 16 * i + 8 * u, 1);
        mbar_init(bar_p_ready + 16 * i + 8 * u, live_i);
      }
      mbar_init(bar_pv_done + 16 * i, 1);
      mbar_init(bar_pv_done + 16 * i + 8, 1);
    }
    mbar_fence_init();
    fence_proxy_async_smem();
  }
  if (warp == 9) {
    tmem_alloc(smem_u32(tmem_slot), kTmemCols);
    tmem_relinquish();
  }
  if (warp == 8 && lane == 0) {
    prefetch_tensormap(&tm_q);
    prefetch_tensormap(&tm_kc);
    prefetch_tensormap(&tm_vc);
    prefetch_tensormap(&tm_kn);
    prefetch_tensormap(&tm_vn);
  }
  // everything above needed no data; from here on the inputs of the call are read
  __syncthreads();   // the barriers exist for the producer's first copy below
  dlm_grid_dependency_wait();
  dlm_trigger_dependents();
  // Whole units and teams: which unit a block starts with does not depend on the lengths, so the copy of its Q
  // rows starts now, while the lengths are read and the tile prefix is built (about 1 us, and Q no longer queues
  // in front of the first K tile).  The roles below consume this Q also when the unit turns out to have no key
  // tile for this block.
  const bool early_q = p.whole_units != 0;
  if (early_q && warp == 8 && lane == 0) {
    const int unit = p.team > 1 ? (int)blockIdx.x / p.team : (int)blockIdx.x;
    const int grp = unit / p.batch, b = unit % p.batch, rc = grp % p.n_rc;
    const int zq = (((grp / p.n_rc) / p.n_kv_heads) * p.batch + b) * p.n_kv_heads + (grp / p.n_rc) % p.n_kv_heads;
    mbar_expect_tx(bar_q_full, (uint32_t)(p.n_mt * min(128, p.rows)) * 128u * G::kPanels);
    for (int mt = 0; mt < p.n_mt; ++mt)
      for (int pn = 0; pn < G::kPanels; ++pn)
        tma_load_3d(sm_q + mt * G::kTileBytes + pn * kPanelBytes, &tm_q, bar_q_full, pn * 64, rc * kChunk + mt * 128, zq);
  }
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
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;
  // number of shares the item list is cut into (every share holds at least one item)
  const int total_items = sched.prefix[p.batch] * p.nl * p.n_kv_heads * p.n_rc;
  const int n_cta = p.whole_units ? (int)gridDim.x : min((int)gridDim.x, total_items);
  const bool has_work = p.whole_units || (int)blockIdx.x < n_cta;
  if (!p.whole_units) {
    for (int c = tid; c <= n_cta; c += kThreads)
      sched.share_lo[c] = (int)((long long)total_items * c / max(n_cta, 1));
    __syncthreads();
  }

  // The softmax warps keep a whole score row in registers; the other warpgroup needs few.
  // setmaxnreg.inc waits, without a bound, until the registers it asks for are free: the host
  // checks before the first launch that what the third warpgroup gives up covers what the two
  // softmax warpgroups take (kRegsSoftmax, kRegsOther against the kernel's register count).
  if (warp >= 8) {
    setmaxnreg_dec<kRegsOther>();
    if (warp == 8) {
      // ================================================================= TMA producer
      if (lane == 0 && has_work) {
        SegmentWalker walk(p, sched, blockIdx.x);
        Segment g;
        uint32_t kt = 0, vt = 0, seg = 0, q_issued = early_q ? 1 : 0;
        bool ok = true;
        bool q_ahead = early_q;   // the Q of the block's first unit is already on its way
        while (ok && walk.next(g, n_cta)) {
          const bool q_here = q_ahead;
          q_ahead = false;
          if (g.t_end <= g.t_begin) {
            if (q_here) ++seg;   // the issuers take and release that Q all the same
            continue;
          }
          const int zq = (g.lc_layer * p.batch + g.b) * p.n_kv_heads + g.kvh;
          const int zc = ((g.lc_layer + p.layer_begin) * p.batch + g.b) * p.n_kv_heads + g.kvh;
          if (!q_here) {
            if (seg > 0) ok = mbar_wait_limit(bar_q_empty, (seg - 1) & 1, abort_ptr, kLimit);
            if (!ok) break;
            const int q_box = min(128, p.rows);
            mbar_expect_tx(bar_q_full, (uint32_t)(p.n_mt * q_box) * 128u * G::kPanels);  // a box counts in full
            for (int mt = 0; mt < p.n_mt; ++mt)
              for (int pn = 0; pn < G::kPanels; ++pn)
                tma_load_3d(sm_q + mt * G::kTileBytes + pn * kPanelBytes, &tm_q, bar_q_full, pn * 64,
                            g.rc * kChunk + mt * 128, zq);
            ++q_issued;
          }
          for (int t = g.t_begin; t < g.t_end && ok; ++t) {
            const bool cache = t < g.n_ct;
            const int row = cache ? t * kTileKeys : (t - g.n_ct) * p.fresh_box;
            const int z = cache ? zc : zq;
            const uint32_t bytes = (uint32_t)(cache ? min(kTileKeys, p.capacity) : p.fresh_box) * 128u * G::kPanels;
            {
              const uint32_t s = kt % KS;
              if (kt >= (uint32_t)KS) ok = mbar_wait_limit(bar_k_empty + 8 * s, ((kt / KS) - 1) & 1, abort_ptr, kLimit);
              if (!ok) break;
              mbar_expect_tx(bar_k_full + 8 * s, bytes);
              for (int pn = 0; pn < G::kPanels; ++pn)
                tma_load_3d(sm_k + s * G::kTileBytes + pn * kPanelBytes, cache ? &tm_kc : &tm_kn, bar_k_full + 8 * s,
                            pn * 64, row, z);
              ++kt;
            }
            {
              const uint32_t s = vt % VS;
              if (vt >= (uint32_t)VS) ok = mbar_wait_limit(bar_v_empty + 8 * s, ((vt / VS) - 1) & 1, abort_ptr, kLimit);
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
            mbar_wait(bar_k_full + 8 * (i % KS), (i / KS) & 1, never_ptr);
          for (uint32_t i = (vt > (uint32_t)VS ? vt - VS : 0); i < vt; ++i)
            mbar_wait(bar_v_full + 8 * (i % VS), (i / VS) & 1, never_ptr);
          if (q_issued > 0) mbar_wait(bar_q_full, (q_issued - 1) & 1, never_ptr);
        }
      }
    } else if (warp == 9 || warp == 10) {
      // ============================================ MMA issuers: warp 9 for M tile 0, warp 10 for M tile 1
      // One warp per M tile, so that the scalar work around one tile's MMAs (barrier waits and
      // commits) runs while the tensor pipe executes the other tile's.  The whole warp runs the
      // loop and one elected lane issues: in warp-uniform code the descriptors live in uniform
      // registers, which is what tcgen05.mma reads; issued from a divergent single-lane branch
      // every MMA paid for moving its operands there.  The K, V and Q buffers are
      // released when every issuer has committed (their "empty" barriers count n_mt arrivals).
      const int mt = warp - 9;
      if (has_work && mt < p.n_mt) {
        auto wait_warp = [&](uint32_t bar, uint32_t parity) {
          return __all_sync(0xffffffffu, mbar_wait_limit(bar, parity, abort_ptr, kLimit)) != 0;
        };
        SegmentWalker walk(p, sched, blockIdx.x);
        Segment g;
        uint32_t kt = 0, vt = 0, gt = 0, seg = 0;
        bool ok = true;
        const uint32_t idesc_pv = make_idesc_bf16(128, D, 1);
        // descriptors of the first K-step of each operand buffer; the loops only add constants
        const uint64_t desc_q = make_smem_desc_sw128(sm_q + mt * G::kTileBytes, 16, 1024);
        const uint64_t desc_k0 = make_smem_desc_sw128(sm_k, 16, 1024);
        const uint64_t desc_v0 = make_smem_desc_sw128(sm_v, kPanelBytes, 1024);
        const uint32_t t_o = tmem + G::kColO + mt * D;
        const uint32_t t_s = tmem + G::kColS + mt * 128;
        // S = Q K^T for the keys [k0, k0 + n16) of the tile in K stage `ks`, into score buffer `buf`
        auto issue_s = [&](uint32_t ks, int k0, int n16, uint32_t buf) {
          const uint32_t idesc = make_idesc_bf16(128, (uint32_t)n16, 0);
          const uint64_t dk = desc_offset(desc_k0, ks * G::kTileBytes + k0 * 128);
          const uint32_t d = t_s + buf * kHalfKeys;
          if (elect_one_sync()) {
            mma_ss<false>(d, desc_q, dk, idesc);
#pragma unroll
            for (int k = 1; k < D / 16; ++k) {
              const uint32_t off = (k >> 2) * kPanelBytes + (k & 3) * 32;
              mma_ss<true>(d, desc_offset(desc_q, off), desc_offset(dk, off), idesc);
            }
          }
          __syncwarp();
        };
        // O (+)= P V for the same keys, P in score buffer `buf`, V tile in stage `vs`
        auto issue_pv = [&](uint32_t vs, int k0, int n16, uint32_t buf, bool first) {
          const uint64_t dv = desc_offset(desc_v0, vs * G::kTileBytes + k0 * 128);
          const uint32_t a = t_s + buf * kHalfKeys;
          if (elect_one_sync()) {
            if (first) mma_ts<false>(t_o, a, dv, idesc_pv); else mma_ts<true>(t_o, a, dv, idesc_pv);
            if (n16 == kHalfKeys) {
#pragma unroll
              for (int st = 1; st < kHalfKeys / 16; ++st) mma_ts<true>(t_o, a + st * 8, desc_offset(dv, st * 2048), idesc_pv);
            } else {
              for (int st = 1; st < n16 / 16; ++st) mma_ts<true>(t_o, a + st * 8, desc_offset(dv, st * 2048), idesc_pv);
            }
          }
          __syncwarp();
        };
        auto commit = [&](uint32_t bar) {
          if (elect_one_sync()) tc_commit(bar);
          __syncwarp();
        };
        uint32_t js = 0;   // half-steps whose scores have been issued (global count: buffer = js & 1)
        bool q_ahead = early_q;   // the Q of the block's first unit was copied before the lengths were known
        while (ok && walk.next(g, n_cta)) {
          const bool q_here = q_ahead;
          q_ahead = false;
          if (g.t_end <= g.t_begin) {
            if (q_here) {   // no key tile for this block after all: take that Q and release it
              ok = wait_warp(bar_q_full, seg & 1);
              if (!ok) break;
              if (lane == 0) mbar_arrive(bar_q_empty);
              __syncwarp();
              ++seg;
            }
            continue;
          }
          ok = wait_warp(bar_q_full, seg & 1);
          if (!ok) break;
          HalfIter si(g, p.fresh_box), pi(g, p.fresh_box);
          // scores of the next half-step of the segment that has none yet, into buffer js & 1
          auto issue_next_s = [&]() -> bool {
            HalfStep hs;
            if (!si.get(hs)) return true;
            const uint32_t ks = kt % KS;
            if (hs.first_of_tile) {
              if (!wait_warp(bar_k_full + 8 * ks, (kt / KS) & 1)) return false;
              tc_fence_after_sync();
            }
            issue_s(ks, hs.k0, (hs.nkeys + 15) & ~15, js & 1);
            commit(bar_s_ready + 16 * mt + 8 * (js & 1));
            ++js;
            si.advance(hs);
            if (hs.last_of_tile) {
              commit(bar_k_empty + 8 * ks);
              ++kt;
              if (si.t >= g.t_end) commit(bar_q_empty);   // Q is not read again in this segment
            }
            return true;
          };
          ok = issue_next_s() && issue_next_s();   // both score buffers filled ahead
          bool first = true;
          HalfStep hs;
          while (ok && pi.get(hs)) {
            const uint32_t vs = vt % VS;
            if (hs.first_of_tile) {
              ok = wait_warp(bar_v_full + 8 * vs, (vt / VS) & 1);
              if (!ok) break;
            }
            ok = wait_warp(bar_p_ready + 16 * mt + 8 * (gt & 1), (gt >> 1) & 1);
            if (!ok) break;
            tc_fence_after_sync();
            issue_pv(vs, hs.k0, (hs.nkeys + 15) & ~15, gt & 1, first);
            commit(bar_pv_done + 16 * mt + 8 * (gt & 1));
            first = false;
            if (hs.last_of_tile) {
              commit(bar_v_empty + 8 * vs);
              ++vt;
            }
            ++gt;
            pi.advance(hs);
            ok = issue_next_s();   // the buffer just consumed takes the half-step after next
          }
          ++seg;
        }
        // every MMA issued by this warp has finished before TMEM is released
        if (elect_one_sync()) tc_commit(bar_drain + 8 * mt);
        __syncwarp();
        mbar_wait(bar_drain + 8 * mt, 0, never_ptr);
      }
    } else {
      // ================================================================= publisher (warp 11)
      // A piece that some other block will merge: once every softmax thread has stored its row
      // (they arrive on bar_pub and move on), make the stores visible device-wide and count the
      // piece in its unit's counter.
      if (lane == 0 && p.team > 1) {
        team_publish<D, kNoWait>(TeamArgs(p), sched.prefix, sm_q, bar_pub, abort_ptr);
      } else if (lane == 0 && has_work && !p.whole_units) {
        SegmentWalker walk(p, sched, blockIdx.x);
        Segment g;
        uint32_t pub = 0;
        while (walk.next(g, n_cta)) {
          if (g.slot < 0 || g.merger || g.t_end <= g.t_begin) continue;
          if (!mbar_wait_limit(bar_pub, pub & 1, abort_ptr, kLimit)) break;
          ++pub;
          __threadfence();
          atomicAdd(p.tickets + ((g.lc_layer * p.n_kv_heads + g.kvh) * p.n_rc + g.rc) * p.batch + g.b, 1u);
        }
      }
    }
  } else {
    setmaxnreg_inc<kRegsSoftmax>();
    if (tid < n_live) {
      // ================================================= softmax warps (those that own real rows)
      const int mt = warp >> 2;
      const int row = (warp & 3) * 32 + lane;                 // row of the M tile = TMEM lane
      const uint32_t t_lane = (uint32_t)((warp & 3) * 32) << 16;
      const uint32_t t_s = tmem + t_lane + G::kColS + mt * 128;
      const uint32_t t_o = tmem + t_lane + G::kColO + mt * D;
      const int r_unit = mt * 128 + row;                      // row within the unit (== tid)
      const int n_live_mt = min(128, n_live - 128 * mt);   // live softmax threads of this M tile
      // the warp leaves a wait together, so the .sync.aligned TMEM instructions that follow
      // always see a converged warp, also when a wait is given up
      auto wait_warp = [&](uint32_t bar, uint32_t parity) {
        return __all_sync(0xffffffffu, mbar_wait_limit(bar, parity, abort_ptr, kLimit)) != 0;
      };
      // this thread's query row in row chunk rc of a KV head: which of its query heads, which active row
      auto out_row_of = [&](int lc_layer, int b, int kvh, int rc) {
        const int r = rc * kChunk + r_unit;
        const int hl = r < p.rows_total ? r / p.q_cap : 0, ir = r < p.rows_total ? r % p.q_cap : 0;
        return (((size_t)lc_layer * p.batch + b) * p.n_q_heads + (size_t)kvh * p.group + hl) * p.q_cap + ir;
      };
      auto zero_my_row = [&](size_t qrow, bool real_row) {
        if (real_row) {
          uint4* o = reinterpret_cast<uint4*>(p.out + qrow * D);
#pragma unroll
          for (int c = 0; c < D / 8; ++c) o[c] = make_uint4(0, 0, 0, 0);
          if (p.lse) p.lse[qrow] = -CUDART_INF_F;
        }
      };
      if (!p.whole_units) {
        // units without any key (inactive batch elements) appear in no share: zero them here
        const int n_units = p.nl * p.n_kv_heads * p.n_rc * p.batch;
        for (int unit = blockIdx.x; unit < n_units; unit += gridDim.x) {
          const int b = unit % p.batch, grp = unit / p.batch, rc = grp % p.n_rc;
          if (sched.prefix[b + 1] == sched.prefix[b])
            zero_my_row(out_row_of((grp / p.n_rc) / p.n_kv_heads, b, (grp / p.n_rc) % p.n_kv_heads, rc),
                        rc * kChunk + r_unit < p.rows_total);
        }
      }
      if (has_work) {
        SegmentWalker walk(p, sched, blockIdx.x);
        Segment g;
        uint32_t gt = 0, vt = 0;   // half-steps and key tiles done so far
        bool ok = true;
        while (ok && walk.next(g, n_cta)) {
          const int n = g.t_end - g.t_begin;
          const size_t qrow = out_row_of(g.lc_layer, g.b, g.kvh, g.rc);
          const int r_kv = g.rc * kChunk + r_unit;               // row among all query rows of the KV head
          const bool real_row = r_kv < p.rows_total;
          const int i_row = real_row ? r_kv % p.q_cap : 0;
          if (n <= 0) {  // inactive batch element: the unit's rows are zero (team schedule: or no tile for this rank)
            if (g.T == 0) {
              zero_my_row(qrow, real_row);
            } else if (g.slot == -2) {   // a piece without key tiles
              ok = team_exchange<D, kChunk, kNoWait>(TeamArgs(p), sched.prefix, sm_q, bar_pub, abort_ptr, t_o, false, -CUDART_INF_F, 0.f);
            }
            continue;
          }
          float m_used = -CUDART_INF_F, l_run = 0.f;
          bool first = true;
          for (int t = g.t_begin; t < g.t_end && ok; ++t, ++vt) {
            const int valid = tile_valid(g, t, p.fresh_box);
            const int n16 = (valid + 15) & ~15;
            if (valid < n16) {
              // V rows in [valid, n16) would be multiplied by P = 0: clear them so that stale
              // NaN / Inf bit patterns cannot reach O.  Each M tile's warps do it before they
              // announce the P of the tile's first half-step, so it precedes that tile's P V
              // products (the two M tiles write the same zeros).
              const uint32_t vs = vt % VS;
              ok = wait_warp(bar_v_full + 8 * vs, (vt / VS) & 1);
              if (!ok) break;
              const int per_row = G::kPanels * 8;
              for (int idx = row; idx < (n16 - valid) * per_row; idx += n_live_mt) {
                const int r = valid + idx / per_row, rem = idx % per_row;
                const uint32_t a = sm_v + vs * G::kTileBytes + (rem >> 3) * kPanelBytes + r * 128 + (rem & 7) * 16;
                asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(a), "r"(0u) : "memory");
              }
              fence_proxy_async_smem();
            }
            // the tile's half-steps (the same enumeration as HalfIter, which the MMA warps use)
            for (int k0 = 0; k0 < valid && ok; k0 += kHalfKeys, ++gt) {
              const int nkeys = min(kHalfKeys, valid - k0);
              const uint32_t buf = gt & 1;
              ok = wait_warp(bar_s_ready + 16 * mt + 8 * buf, (gt >> 1) & 1);
              if (!ok) break;
              tc_fence_after_sync();
              if (nkeys == kHalfKeys)
                ok = softmax_half_full<D>(t_s + buf * kHalfKeys, t_o, first, p.scale_log2, m_used, l_run,
                                          bar_pv_done + 16 * mt + 8 * ((gt - 1) & 1), ((gt - 1) >> 1) & 1, abort_ptr);
              else
                ok = softmax_half_ragged<D>(t_s + buf * kHalfKeys, t_o, nkeys, first, p.scale_log2, m_used, l_run,
                                            bar_pv_done + 16 * mt + 8 * ((gt - 1) & 1), ((gt - 1) >> 1) & 1, abort_ptr);
              if (!ok) break;
              // every lane's P is stored (tcgen05.wait::st inside the softmax); one lane announces the warp's rows
              __syncwarp();
              if (lane == 0) {
                tc_fence_before_sync();
                mbar_arrive(bar_p_ready + 16 * mt + 8 * buf);
              }
              first = false;
            }
          }
          if (!ok) break;
          // ---- epilogue of the segment: O is complete once the last P V product has finished
          ok = wait_warp(bar_pv_done + 16 * mt + 8 * ((gt - 1) & 1), ((gt - 1) >> 1) & 1);
          if (!ok) break;
          tc_fence_after_sync();
          const bool active = real_row && i_row < g.Lq;
          uint32_t v[32];
          if (g.slot == -2) {
            ok = team_exchange<D, kChunk, kNoWait>(TeamArgs(p), sched.prefix, sm_q, bar_pub, abort_ptr, t_o, true, m_used, l_run);
          } else if (g.slot < 0) {
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
              p.lse[qrow] = active ? (m_used + lg2_approx(l_run)) * 0.6931471805599453f : -CUDART_INF_F;
          } else {
            // ---- a piece of a split unit.  Partial O is stored as 16-byte vectors of 4 columns,
            // [D/4][128 rows][4]: a warp's 32 rows of one vector are 512 contiguous bytes, for the
            // stores here and for the loads of the merge.
            if (!g.merger) {
              float4* po = reinterpret_cast<float4*>(p.ws_o) + ((size_t)g.slot * p.n_mt + mt) * (size_t)(D / 4 * 128) + row;
#pragma unroll 1
              for (int c = 0; c < D / 32; ++c) {
                tmem_ld32(t_o + c * 32, v);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 8; ++j)
                  __stcg(po + (c * 8 + j) * 128, make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                                             __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3])));
              }
              __stcg(reinterpret_cast<float2*>(p.ws_ml) + ((size_t)g.slot * p.n_mt + mt) * 128 + row,
                     make_float2(m_used, l_run));
              mbar_arrive(bar_pub);   // the publisher warp takes it from here
            } else {
              // ---- the unit's last piece: this block merges.  The other pieces belong to blocks
              // c_first .. this - 1, which computed them first thing; wait for their count, then fold
              // them into O (own piece first, then block order: the result does not depend on timing).
              const UnitPieces up(p, sched, g, blockIdx.x);
              const int n_others = up.c_last - up.c_first;
              const int unit = ((g.lc_layer * p.n_kv_heads + g.kvh) * p.n_rc + g.rc) * p.batch + g.b;
              if (tid == 0) {
                const bool came = wait_counter(p.tickets + unit, (unsigned int)n_others, abort_ptr, kLimit);
                if (came) p.tickets[unit] = 0;   // ready for the next launch
                *merge_ok = came ? 1 : 2;
              }
              // The other threads wait for thread 0's verdict on a flag, not on a hardware barrier: a warp that
              // gave up earlier never gets here, and a barrier would then wait for it for ever.  Thread 0 always
              // writes the flag within its own bounded wait; if its warp gave up before, the abort flag is up.
              for (uint32_t spin = 1; *merge_ok == 0; ++spin)
                if ((spin & 63u) == 0u && *abort_ptr) break;
              __syncwarp();
              const int verdict = __shfl_sync(0xffffffffu, *merge_ok, 0);   // one answer per warp: the code below is .aligned
              if (verdict != 1) { ok = false; break; }
              __threadfence();
              // maximum and sum over all pieces
              float m_all = m_used, l_all = l_run;
              for (int ib = 0; ib < n_others; ib += 4) {
                float2 ml[4];
#pragma unroll
                for (int j = 0; j < 4; ++j)
                  ml[j] = (ib + j < n_others)
                              ? __ldcg(reinterpret_cast<const float2*>(p.ws_ml) +
                                       ((size_t)up.slot_of(up.c_first + ib + j) * p.n_mt + mt) * 128 + row)
                              : make_float2(-CUDART_INF_F, 0.f);
                const float m_new = fmaxf(fmaxf(fmaxf(ml[0].x, ml[1].x), fmaxf(ml[2].x, ml[3].x)), m_all);
                l_all *= ex2_approx(m_all - m_new);
#pragma unroll
                for (int j = 0; j < 4; ++j) l_all += ml[j].y * ex2_approx(ml[j].x - m_new);
                m_all = m_new;
              }
              const float inv = active ? 1.f / l_all : 0.f;
              const float w_own = ex2_approx(m_used - m_all);
              if (real_row && p.lse)
                p.lse[qrow] = active ? (m_all + lg2_approx(l_all)) * 0.6931471805599453f : -CUDART_INF_F;
              // O: one other piece at a time, all of its row in flight at once (L2 latency, not
              // bandwidth, bounds a narrower loop); the running sum lives in TMEM between pieces
              for (int i = 0; i < n_others; ++i) {
                const size_t piece = (size_t)up.slot_of(up.c_first + i) * p.n_mt + mt;
                const float4* src = reinterpret_cast<const float4*>(p.ws_o) + piece * (size_t)(D / 4 * 128) + row;
                float4 x[D / 4];
#pragma unroll
                for (int j = 0; j < D / 4; ++j) x[j] = __ldcg(src + j * 128);
                const float w = ex2_approx(__ldcg(p.ws_ml + (piece * 128 + row) * 2) - m_all);
                const float w0 = (i == 0) ? w_own : 1.f;
                const bool last = (i == n_others - 1);
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                  tmem_ld32(t_o + c * 32, v);
                  tmem_ld_wait();
#pragma unroll
                  for (int j = 0; j < 8; ++j) {
                    v[4 * j + 0] = __float_as_uint(fmaf(w, x[c * 8 + j].x, w0 * __uint_as_float(v[4 * j + 0])));
                    v[4 * j + 1] = __float_as_uint(fmaf(w, x[c * 8 + j].y, w0 * __uint_as_float(v[4 * j + 1])));
                    v[4 * j + 2] = __float_as_uint(fmaf(w, x[c * 8 + j].z, w0 * __uint_as_float(v[4 * j + 2])));
                    v[4 * j + 3] = __float_as_uint(fmaf(w, x[c * 8 + j].w, w0 * __uint_as_float(v[4 * j + 3])));
                  }
                  if (!last) {
                    tmem_st32(t_o + c * 32, v);
                  } else if (real_row) {
                    uint4* o = reinterpret_cast<uint4*>(p.out + qrow * D + c * 32);
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                      uint32_t wd[4];
#pragma unroll
                      for (int j = 0; j < 4; ++j) {
                        const __nv_bfloat162 h =
                            __floats2bfloat162_rn(active ? __uint_as_float(v[q4 * 8 + 2 * j]) * inv : 0.f,
                                                  active ? __uint_as_float(v[q4 * 8 + 2 * j + 1]) * inv : 0.f);
                        wd[j] = *reinterpret_cast<const uint32_t*>(&h);
                      }
                      o[q4] = make_uint4(wd[0], wd[1], wd[2], wd[3]);
                    }
                  }
                }
                if (!last) tmem_st_wait();
              }
            }
          }
        }
      }
    }
  }
  // ---- teardown: nothing of this block is in flight any more
  __syncwarp();
  if (tid == 0 && *abort_ptr) dlm_set_status(p.status, DLM_ERR_TIMEOUT);
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 9) {
    tc_fence_after_sync();
    tmem_dealloc(tmem, kTmemCols);
  }
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

// The kernel starts with `numRegs` registers per thread in all 12 warps.  The 8 softmax warps then
// ask for kRegsSoftmax each and block until they get them; only what the other 4 warps release
// is certain to be free, so the request must fit inside that.
bool register_budget_ok(const cudaFuncAttributes& a) {
  return a.numRegs >= kRegsOther && 8 * (kRegsSoftmax - a.numRegs) <= 4 * (a.numRegs - kRegsOther);
}

// The eight instantiations: head_dim 128 / 64, row chunks of 256 / 128, normal / no-wait (test) waits.
using AttnKernel = void (*)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const CUtensorMap, const CUtensorMap,
                            const AttnParams);
inline int kernel_index(int head_dim, int chunk_rows, bool no_wait) {
  return (head_dim == 128 ? 0 : 1) + (chunk_rows == 256 ? 0 : 2) + (no_wait ? 4 : 0);
}
AttnKernel kernel_of(int which) {
  switch (which) {
    case 0: return attn_step_sm100_kernel<128, 256, false>;
    case 1: return attn_step_sm100_kernel<64, 256, false>;
    case 2: return attn_step_sm100_kernel<128, 128, false>;
    case 3: return attn_step_sm100_kernel<64, 128, false>;
    case 4: return attn_step_sm100_kernel<128, 256, true>;
    case 5: return attn_step_sm100_kernel<64, 256, true>;
    case 6: return attn_step_sm100_kernel<128, 128, true>;
    default: return attn_step_sm100_kernel<64, 128, true>;
  }
}

// First use of an attention kernel on a context's device: checks the register budget and opts in to
// all the dynamic shared memory the device allows a block (less the kernel's static part).
int configure_kernel(dlm_ctx* ctx, int which, const void* kern) {
  if (ctx->attn_smem_limit[which] > 0) return DLM_OK;
  cudaFuncAttributes a;
  DLM_CUDA_TRY(cudaFuncGetAttributes(&a, kern));
  if (!register_budget_ok(a)) return DLM_ERR_UNSUPPORTED;
  const int limit = ctx->max_smem_optin - (int)a.sharedSizeBytes;
  if (limit <= 0) return DLM_ERR_UNSUPPORTED;
  DLM_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, limit));
  ctx->attn_smem_limit[which] = limit;
  return DLM_OK;
}

struct Plan {
  int n_mt, rows, rows_total, n_rc, grid, whole_units, chunk_rows, team;
  int smem_bytes;
  size_t ws_o_bytes, ws_ml_bytes;
};

// Shared memory of a block: Q tiles, the K and V rings, barriers, flags, scheduling tables and up to
// 1023 bytes of alignment.  (Deeper rings were measured: 2 + 3 and 3 + 3 stages at head_dim 128 were
// 3 - 10 % slower on the configs' shapes, so the rest of the shared memory stays unused.)
bool plan_shared_memory(int smem_limit, int head_dim, int batch, Plan& pl) {
  const int tile = head_dim / 64 * kPanelBytes;
  const int stages = head_dim == 128 ? Geometry<128>::kStages : Geometry<64>::kStages;
  pl.smem_bytes = 1024 + (pl.n_mt + 2 * stages) * tile + kBarrierBytes + kFlagBytes + 4 * sched_ints(batch, pl.grid);
  return pl.smem_bytes <= smem_limit;
}

// Splitting units across blocks balances the load but costs each block a partial store and each
// unit a wait and a merge that grows with its number of pieces (measured: about 3 key tiles' worth
// plus 0.7 per further piece); dealing units whole costs idle SMs when the units do not fill a
// whole number of waves.  The number of shares (= blocks) is chosen to minimise the estimated
// time in key tiles per block, from the caller's cache length hint; one share per unit or fewer
// means whole units.
Plan make_plan(const dlm_ctx* ctx, const dlm_kv_cache* cache, int nl, int n_q_heads, int q_cap, int cache_len_hint) {
  Plan pl;
  pl.rows_total = (n_q_heads / cache->n_kv_heads) * q_cap;
  // Row chunks of 256 (two M tiles sharing every K/V tile) read K/V once per KV head.  When a call has
  // only a handful of such units (one layer of a small batch), chunks of 128 double the units that can
  // be spread over the SMs and halve every partial result; the second read of K/V comes from L2
  // (measured on one Dream-shaped layer at batch 1: 15.9 us against 20.9).
  const long long units256 = (long long)nl * cache->batch * cache->n_kv_heads * ((pl.rows_total + 255) / 256);
  pl.chunk_rows = (pl.rows_total > 128 && units256 * 8 <= ctx->num_sms) ? 128 : 256;
  pl.n_rc = (pl.rows_total + pl.chunk_rows - 1) / pl.chunk_rows;
  pl.rows = pl.rows_total < pl.chunk_rows ? pl.rows_total : pl.chunk_rows;
  pl.n_mt = (pl.rows + 127) / 128;
  const long long units = (long long)nl * cache->batch * cache->n_kv_heads * pl.n_rc;
  const int sms = ctx->num_sms < kMaxGrid ? ctx->num_sms : kMaxGrid;
  const bool may_split = units < 8LL * sms && units <= kDlmMaxSplitUnits;
  const int len = (cache_len_hint > 0 && cache_len_hint < cache->capacity) ? cache_len_hint : cache->capacity;
  const long long tiles_unit = (len + 127) / 128 + (q_cap + 127) / 128;
  const double t_whole = (double)(((units + sms - 1) / sms) * tiles_unit);
  double best = t_whole;
  int best_shares = 0;   // 0: whole units
  if (may_split) {
    for (long long shares = units + 1; shares <= sms; ++shares) {
      if (shares > units * tiles_unit) break;   // a share holds at least one item
      const double pieces = (double)shares / (double)units;
      const double t = (double)((units * tiles_unit + shares - 1) / shares) + 3.0 + 0.7 * (pieces - 1.0);
      if (t < best) { best = t; best_shares = (int)shares; }
    }
    if (units > sms) {   // more units than SMs: the only split is over all SMs
      const double t = (double)((units * tiles_unit + sms - 1) / sms) + 3.0 + 0.7;
      if (t < best) { best = t; best_shares = sms; }
    }
  }
  pl.whole_units = best_shares == 0 ? 1 : 0;
  pl.grid = pl.whole_units ? (int)(units < sms ? units : sms) : best_shares;
  // Team schedule for calls with few units: C blocks per unit, the unit's key tiles dealt among them, every
  // block reducing a C-th of the outputs over all pieces in parallel (the split schedule's merging block
  // folds the other pieces one after the other).  The smallest C that reaches the fewest tiles per block.
  pl.team = 1;
  if (ctx->attn_team_max > 1 && may_split && units * 2 <= sms) {
    long long C = ctx->attn_team_max < kTeamMax ? ctx->attn_team_max : kTeamMax;
    if (C > sms / units) C = sms / units;
    if (C > tiles_unit) C = tiles_unit;
    if (C > 1) {
      const long long per_block = (tiles_unit + C - 1) / C;
      C = (tiles_unit + per_block - 1) / per_block;
      const double t = (double)per_block + kTeamMergeTiles * pl.n_mt;   // a piece of two M tiles is twice the bytes
      if (C > 1 && (t < best || ctx->attn_team_force)) {
        pl.team = (int)C;
        pl.whole_units = 1;
        pl.grid = (int)(units * C);
      }
    }
  }
  // the workspace is sized for the split schedule whenever that schedule is possible at all, so
  // that its size does not depend on the hint
  const size_t slots = may_split ? 2 * (size_t)sms : 0;
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
  const Plan pl = make_plan(ctx, cache, n_layers_in_call, n_q_heads, q_cap, 0);
  return pl.ws_o_bytes + pl.ws_ml_bytes + 256;
}

extern "C" int dlm_selftest_attn_schedule(const dlm_ctx* ctx, const dlm_kv_cache* cache, int n_layers_in_call, int n_q_heads,
                                          int q_cap, int cache_len_hint, int* grid, int* team, int* whole_units,
                                          int* chunk_rows) {
  if (!ctx || !cache || !grid || !team || !whole_units || !chunk_rows) return DLM_ERR_NULL;
  if (n_layers_in_call <= 0 || n_q_heads <= 0 || q_cap <= 0 || cache->n_kv_heads <= 0 || cache->batch <= 0 ||
      cache->capacity <= 0 || n_q_heads % cache->n_kv_heads != 0)
    return DLM_ERR_SHAPE;
  const Plan pl = make_plan(ctx, cache, n_layers_in_call, n_q_heads, q_cap, cache_len_hint);
  *grid = pl.grid;
  *team = pl.team;
  *whole_units = pl.whole_units;
  *chunk_rows = pl.chunk_rows;
  return DLM_OK;
}

extern "C" int dlm_freecache_attn_step(dlm_ctx* ctx, const dlm_kv_cache* cache, int layer_begin, int layer_end,
                                       const void* q, const void* k_new, const void* v_new, int n_q_heads,
                                       int q_cap, const int32_t* q_len, float softmax_scale, int cache_len_hint,
                                       void* out, float* lse, void* workspace, size_t workspace_bytes,
                                       void* stream) {
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
  if (q_cap > kMaxQCap || (long long)group * q_cap > (1 << 20) || cache->batch > kMaxBatch) return DLM_ERR_UNSUPPORTED;
  if (((uintptr_t)cache->k | (uintptr_t)cache->v | (uintptr_t)q | (uintptr_t)k_new | (uintptr_t)v_new |
       (uintptr_t)out) & 15)
    return DLM_ERR_UNSUPPORTED;
  DLM_DEVICE_TRY(ctx);
  const int nl = layer_end - layer_begin;
  const size_t need = dlm_attn_workspace_bytes(ctx, cache, nl, n_q_heads, q_cap);
  if (!workspace || workspace_bytes < need || ((uintptr_t)workspace & 255)) return DLM_ERR_WORKSPACE;
  const Plan pl = make_plan(ctx, cache, nl, n_q_heads, q_cap, cache_len_hint);
  {
    const bool nw = ctx->wait_limit_ns == 0;
    const int which = kernel_index(D, pl.chunk_rows, nw);
    const int rc = configure_kernel(ctx, which, reinterpret_cast<const void*>(kernel_of(which)));
    if (rc != DLM_OK) return rc;
  }
  Plan pl_mut = pl;
  if (!plan_shared_memory(ctx->attn_smem_limit[kernel_index(D, pl.chunk_rows, ctx->wait_limit_ns == 0)], D, cache->batch, pl_mut)) return DLM_ERR_UNSUPPORTED;
  {  // the split schedule counts (unit, key tile) items in 32 bits
    const long long tiles_per_unit = (cache->capacity + 127) / 128 + (q_cap + 127) / 128 + 1;
    if (!pl.whole_units && (long long)nl * cache->batch * cache->n_kv_heads * pl.n_rc * tiles_per_unit >= (1LL << 30))
      return DLM_ERR_UNSUPPORTED;
  }

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
  p.chunk_rows = pl.chunk_rows;
  p.rows_total = pl.rows_total;
  p.n_rc = pl.n_rc;
  p.n_mt = pl.n_mt;
  p.fresh_box = q_cap < 128 ? q_cap : 128;
  p.whole_units = pl.whole_units;
  p.team = pl.team;
  p.smem_bytes = pl_mut.smem_bytes;
  const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)D);
  p.scale_log2 = scale * 1.4426950408889634f;
  p.status = &ctx->words->status;
  p.tickets = ctx->words->attn_unit_tickets;

  CUtensorMap tm_q, tm_kc, tm_vc, tm_kn, tm_vn;
  const long long slabs_new = (long long)nl * cache->batch * cache->n_kv_heads;
  const long long slabs_cache = (long long)cache->n_layers * cache->batch * cache->n_kv_heads;
  const int cache_box = cache->capacity < 128 ? cache->capacity : 128;
  int rc = encode_map(ctx, &tm_q, q, D, pl.rows_total, slabs_new, pl.rows < 128 ? pl.rows : 128);
  if (rc == DLM_OK) rc = encode_map(ctx, &tm_kc, cache->k, D, cache->capacity, slabs_cache, cache_box);
  if (rc == DLM_OK) rc = encode_map(ctx, &tm_vc, cache->v, D, cache->capacity, slabs_cache, cache_box);
  if (rc == DLM_OK) rc = encode_map(ctx, &tm_kn, k_new, D, q_cap, slabs_new, p.fresh_box);
  if (rc == DLM_OK) rc = encode_map(ctx, &tm_vn, v_new, D, q_cap, slabs_new, p.fresh_box);
  if (rc != DLM_OK) return rc;

  cudaStream_t s = static_cast<cudaStream_t>(stream);
  DLM_CUDA_TRY(dlm_launch(kernel_of(kernel_index(D, pl.chunk_rows, ctx->wait_limit_ns == 0)), dim3(pl.grid), dim3(kThreads),
                          (size_t)p.smem_bytes, s, tm_q, tm_kc, tm_vc, tm_kn, tm_vn, p));
  return dlm_launch_ok(ctx, 1);
}
