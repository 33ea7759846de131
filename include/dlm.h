/*
 * dlm.h — C-ABI of the FreeCache denoising-step library for NVIDIA B200 (sm_100a).
 *
 * The library implements the per-step hot path of a diffusion language model (DLM) served
 * with FreeCache and Guided Diffusion:
 *
 *   dlm_freecache_attn_step  bidirectional GQA attention of the active window over
 *                            [frozen cache rows ; freshly recomputed rows]   (Sec. 3.2.1)
 *   dlm_kv_cache_commit      writes K/V rows into the device-resident cache  (Sec. 3.2.1)
 *   dlm_unmask_select        confidence = max softmax probability, argmax token,
 *                            top-k unmasking                                (Eq. 1-3)
 *   dlm_guided_accept        longest agreeing prefix between the DLM proposals and an
 *                            autoregressive guider's argmax                 (Algorithm 1)
 *
 * Conventions
 *   - Every function returns an int: DLM_OK (0) or a negative DLM_ERR_* code.  When an
 *     argument error is returned nothing has been launched.
 *   - Pointers documented "device" are caller-owned device pointers on the context's GPU and
 *     must stay valid until the enqueued work has finished.  The library never allocates,
 *     frees or retains tensor memory; the only device memory it owns is about 12 KB of
 *     status and ticket words inside the context.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  All calls
 *     only enqueue work; none synchronises except dlm_get_status.
 *   - Data-dependent errors (an index out of range, an append beyond capacity, a bounded
 *     device-side wait that expired) cannot be detected on the host without a round trip.
 *     The kernels suppress the offending writes, record the first such error in the
 *     context's device status word, and dlm_get_status reports it.
 *   - All tensors are contiguous, row-major, innermost dimension last.  bf16 means the
 *     16-bit brain-float bit pattern.
 *   - There is no CPU fallback: on a machine without a usable sm_100 device dlm_create fails.
 */
#ifndef DLM_H_
#define DLM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  DLM_OK = 0,
  DLM_ERR_NULL = -1,        /* a required pointer is NULL                                  */
  DLM_ERR_SHAPE = -2,       /* a size is non-positive or inconsistent                       */
  DLM_ERR_UNSUPPORTED = -3, /* valid but not implemented (head_dim, group size, ...)        */
  DLM_ERR_CAPACITY = -4,    /* cache_len + rows would exceed the cache capacity             */
  DLM_ERR_WORKSPACE = -5,   /* workspace NULL, misaligned or too small                      */
  DLM_ERR_CUDA = -6,        /* a CUDA runtime / driver call failed                          */
  DLM_ERR_TIMEOUT = -7,     /* a bounded device-side wait expired (kernel gave up cleanly)  */
  DLM_ERR_INDEX = -8,       /* a row index read from device memory is out of range          */
  DLM_ERR_DEVICE = -9       /* the calling thread's current CUDA device is not the context's */
};

enum { DLM_DST_APPEND = 0, DLM_DST_WINDOW = 1 }; /* dlm_kv_cache_commit: where rows go when dst_pos is NULL */

typedef struct dlm_ctx dlm_ctx;

/* Creates a context bound to CUDA device `device` (must be compute capability 10.x).
 * Every later call that takes the context must be made with that device current on the
 * calling thread (else DLM_ERR_DEVICE, nothing launched).
 * The context owns only its status / ticket words.  Not thread-safe: use one context per
 * host thread or serialise calls.  Kernels enqueued through one context on different
 * streams must not overlap in time (they share the context's ticket words). */
int dlm_create(dlm_ctx** out, int device);
int dlm_destroy(dlm_ctx* ctx);

/* Synchronises `stream`, returns the first data-dependent error recorded by any kernel
 * since the last call (DLM_OK if none) and clears it. */
int dlm_get_status(dlm_ctx* ctx, void* stream);

/* Static, human-readable text for a return code. */
const char* dlm_strerror(int code);

/* Number of kernels this context has launched so far (host-side counter). */
int64_t dlm_launch_count(const dlm_ctx* ctx);

/* Diagnostic: enqueues a one-warp kernel that waits, with the library's bounded device-side wait and a
 * limit of `limit_ns` nanoseconds (1 .. 1e9), on a barrier nobody arrives at.  The wait gives up, the
 * kernel ends normally and dlm_get_status then reports DLM_ERR_TIMEOUT; the context stays usable.  This is
 * how the give-up path of every wait in the kernels is exercised without hanging a GPU. */
int dlm_selftest_wait_timeout(dlm_ctx* ctx, uint64_t limit_ns, void* stream);

/* Diagnostic: sets the limit of the attention kernel's device-side waits on work still to come (TMA copies, MMAs,
 * other blocks' partial results) for the calls that follow.  Two values are compiled in: 2 000 000 000 (2 s, the
 * default) and 0; anything else up to 2 s is DLM_ERR_UNSUPPORTED, anything above DLM_ERR_SHAPE.
 * 0 means "do not wait at all": the first wait whose data has not arrived yet gives up, every role of the block
 * unwinds (copies and MMAs already issued are still waited for, with the 2 s limit, before the block releases its
 * shared memory and TMEM), the kernel ends normally, its outputs are unspecified and dlm_get_status reports
 * DLM_ERR_TIMEOUT.  This runs the kernel's own give-up path without hanging or faulting anything. */
int dlm_selftest_set_wait_limit(dlm_ctx* ctx, uint64_t limit_ns);

/* Diagnostic: the most blocks (>= 1, else DLM_ERR_SHAPE; unlimited by default, the schedule's own maximum is 16)
 * that dlm_freecache_attn_step may give one unit in its team schedule, in the calls that follow.  That schedule
 * serves calls with few (layer, batch element, KV head, row chunk) units: a team of blocks per unit, the unit's
 * key tiles dealt among them, every block reducing its share of the unit's outputs over all the team's partial
 * results.  It is chosen when a cost estimate prefers it to the other schedules; force = 1 (0 by default; other
 * values DLM_ERR_SHAPE) takes it wherever it is possible at all: at most half as many units as SMs and more than
 * one key tile per unit.  max_blocks = 1 switches the schedule off, so that the same call can be run through the
 * other schedules and the results compared; they agree to rounding, not bit for bit (the order of the merge
 * differs). */
int dlm_selftest_set_attn_team_max(dlm_ctx* ctx, int max_blocks, int force);

/* View of a caller-owned KV cache (Sec. 3.2.1: K/V of the prompt and of frozen blocks).
 *   k, v       device, bf16 [n_layers][batch][n_kv_heads][capacity][head_dim]
 *   cache_len  device, int32 [batch]: rows [0, cache_len[b]) are visible to attention.
 * Rows at or beyond cache_len[b] may hold anything (stale, staged, NaN) and never
 * influence a result. */
typedef struct {
  void* k;
  void* v;
  int32_t* cache_len;
  int32_t n_layers, batch, n_kv_heads, capacity, head_dim;
} dlm_kv_cache;

/*
 * dlm_kv_cache_commit — cache fill, refresh and freeze (Sec. 3.2.1: the initial pass "saves"
 * K/V for the whole sequence; a finished block's K/V are "frozen").
 *
 * For every layer in [layer_begin, layer_end), batch element b, r < n(b), KV head, and both
 * tensors:   cache[layer][b][head][dst(b,r)][:] = new[layer-layer_begin][b][head][src(b,r)][:]
 *   src(b,r) = src_idx ? src_idx[b*n_max + r] : r
 *   dst(b,r) = dst_pos ? dst_pos[b*n_max + r]
 *            : dst_mode == DLM_DST_WINDOW ? cache_len[b] + src(b,r)   (row p of the active window
 *                                            is staged at its own slot behind the visible rows)
 *            : cache_len[b] + r                                       (DLM_DST_APPEND)
 *   n(b)     = n_rows  ? n_rows[b]            : n_max
 * If advance_len != 0, cache_len[b] += n(b) once all rows of the call are written.
 *
 *   k_new, v_new  device, bf16 [layer_end-layer_begin][batch][n_kv_heads][src_len][head_dim]
 *   src_idx       device, int32 [batch][n_max] or NULL
 *   dst_pos       device, int32 [batch][n_max] or NULL; destinations within one batch element
 *                 must be distinct (duplicates race: the row written is then unspecified and may
 *                 mix 16-byte pieces of several sources, K and V independently)
 *   n_rows        device, int32 [batch] or NULL
 * Argument errors: NULL cache / tensors, src_len <= 0, n_max <= 0, bad layer range,
 * head_dim * 2 bytes not a multiple of 16.
 * dst_mode other than the two constants is DLM_ERR_SHAPE; it is ignored when dst_pos is given.
 * Data-dependent: n(b) outside [0, n_max], or an append / advance with cache_len[b] + n(b) >
 * capacity: nothing is written for b, status DLM_ERR_CAPACITY; an index outside [0, src_len) /
 * [0, capacity): that row is skipped, status DLM_ERR_INDEX.
 */
int dlm_kv_cache_commit(dlm_ctx* ctx, const dlm_kv_cache* cache, const void* k_new,
                        const void* v_new, int src_len, const int32_t* src_idx,
                        const int32_t* dst_pos, int dst_mode, const int32_t* n_rows, int n_max,
                        int advance_len, int layer_begin, int layer_end, void* stream);

/* Bytes of device scratch dlm_freecache_attn_step needs for `n_layers_in_call` layers,
 * `n_q_heads` query heads and `q_cap` active rows on this cache (split-KV partial results).
 * Returns 0 on invalid arguments. */
size_t dlm_attn_workspace_bytes(const dlm_ctx* ctx, const dlm_kv_cache* cache,
                                int n_layers_in_call, int n_q_heads, int q_cap);

/* Diagnostic: the schedule dlm_freecache_attn_step would choose for a call with these arguments (host only,
 * launches nothing; only the cache's shape fields are read).  Outputs (host): the grid size; the blocks per
 * team (1 = no teams); whether units are dealt whole (1) or split across blocks (0); query rows per unit
 * (256 or 128).  DLM_ERR_NULL / DLM_ERR_SHAPE as for the call itself. */
int dlm_selftest_attn_schedule(const dlm_ctx* ctx, const dlm_kv_cache* cache, int n_layers_in_call, int n_q_heads,
                               int q_cap, int cache_len_hint, int* grid, int* team, int* whole_units,
                               int* chunk_rows);

/*
 * dlm_freecache_attn_step — attention of the active window (Sec. 3.2.1 "Windowed
 * Re-computation"; Table 1 rows QK^T and Attention Score x Value; no causal mask).
 *
 * For each layer l in [layer_begin, layer_end), batch element b, query head h (KV head
 * h / (n_q_heads / n_kv_heads)) and active row i < q_len(b):
 *     keys/values = cache rows [0, cache_len[b]) of layer l, then fresh rows [0, q_len(b))
 *     out[l][b][h][i][:] = sum_j softmax_j(scale * <q_i, k_j>) v_j      (fp32 accumulate)
 *     lse[l][b][h][i]    = log sum_j exp(scale * <q_i, k_j>)            (natural log)
 * Rows i >= q_len(b) get out = 0 and lse = -inf.  More than one layer per call is only
 * meaningful when all layers' Q/K/V exist up front (a synthetic stack); a real model calls
 * it once per layer.
 *
 *   q            device, bf16 [layers][batch][n_q_heads][q_cap][head_dim]
 *   k_new, v_new device, bf16 [layers][batch][n_kv_heads][q_cap][head_dim]
 *   q_len        device, int32 [batch] or NULL (= q_cap for all)
 *   softmax_scale  <= 0 selects 1/sqrt(head_dim)
 *   cache_len_hint host estimate of max_b cache_len[b], used only to choose between the two work
 *                  schedules (units split across SMs, or dealt whole); <= 0 means "capacity".
 *                  A poor hint costs speed, never correctness.
 *   out          device, bf16 [layers][batch][n_q_heads][q_cap][head_dim]
 *   lse          device, fp32 [layers][batch][n_q_heads][q_cap] or NULL
 *   workspace    device, 256-byte aligned, at least dlm_attn_workspace_bytes(...)
 * Supported: head_dim in {64, 128}; n_q_heads a multiple of n_kv_heads; 1 <= q_cap <= 4096.
 * Otherwise DLM_ERR_UNSUPPORTED.  The (n_q_heads / n_kv_heads) * q_cap query rows that share a KV head
 * are processed 256 at a time; each group of 256 reads that head's K/V once (the repeats normally hit L2).
 * q_cap = the whole remaining generation is the windowed re-computation of Sec. 3.2.1; cache_len = 0 with
 * q_cap = the whole sequence is the initial full pass that fills the cache.
 * Data-dependent: cache_len[b] outside [0, capacity] or q_len[b] outside [0, q_cap] is
 * clamped and recorded as DLM_ERR_CAPACITY; an expired device wait as DLM_ERR_TIMEOUT.
 */
int dlm_freecache_attn_step(dlm_ctx* ctx, const dlm_kv_cache* cache, int layer_begin,
                            int layer_end, const void* q, const void* k_new, const void* v_new,
                            int n_q_heads, int q_cap, const int32_t* q_len, float softmax_scale,
                            int cache_len_hint, void* out, float* lse, void* workspace,
                            size_t workspace_bytes, void* stream);

/* Bytes of device scratch dlm_unmask_select needs (per-row partial reductions). */
size_t dlm_unmask_workspace_bytes(const dlm_ctx* ctx, int batch, int block_len, int vocab);

/*
 * dlm_unmask_select — confidence scoring and top-k unmasking (Eq. 2: one logit row per masked
 * position; Eq. 3: fill with the argmax; M_{t-1} = M_t \ U_t).
 *
 * For each masked (b, i):  tok = lowest v attaining max_v z_v,  conf = 1 / sum_v exp(z_v - max z)
 * (the maximum softmax probability).  Unmasked positions get tok = -1, conf = -1.
 * If k > 0, per batch element: k_eff = min(k, number of masked positions); U = the k_eff masked
 * positions of largest conf, ties to the lowest position; tokens[U] = tok[U]; masked[U] = 0;
 * sel_idx[b][0..k_eff) = U ascending, remaining entries -1; n_sel[b] = k_eff.
 * If k == 0 ("propose only") only tok and conf are written; sel_idx / n_sel may be NULL.
 *
 *   logits   device, fp32 [batch][block_len][vocab]; -inf entries allowed (they contribute 0); a masked
 *            row that is -inf throughout, NaN and +inf are caller errors with unspecified results
 *   masked   device, uint8 [batch][block_len], in/out (non-zero = masked)
 *   tokens   device, int32 [batch][block_len], in/out
 *   tok      device, int32 [batch][block_len], out
 *   conf     device, fp32  [batch][block_len], out
 *   sel_idx  device, int32 [batch][k], out;   n_sel device, int32 [batch], out
 *   workspace device, 16-byte aligned, at least dlm_unmask_workspace_bytes(...)
 * Supported: block_len <= 1024.
 */
int dlm_unmask_select(dlm_ctx* ctx, const float* logits, int batch, int block_len, int vocab,
                      uint8_t* masked, int32_t* tokens, int k, int32_t* tok, float* conf,
                      int32_t* sel_idx, int32_t* n_sel, void* workspace, size_t workspace_bytes,
                      void* stream);

/*
 * dlm_unmask_select_static — dlm_unmask_select for callers that cannot allocate device memory.
 * (The paper has no counterpart: this is a deployment variant of the call above, with the same
 * arithmetic and the same results.)
 *
 * Some hosts of this library may not call cudaMalloc at all: code that runs under a fixed
 * memory plan handed out by an outer runtime, plug-ins whose allocator belongs to another
 * component, or processes started after the device's memory has been given away.  Such a
 * caller can own neither a context (dlm_create allocates) nor a workspace.  This entry point
 * needs neither: the per-row partial reductions live in a 1 MiB array that is part of the
 * library's device image (every GPU that loads the library holds it until the process exits).
 * It calls no allocating routine, takes no context and reports errors only by return code.
 *
 * Arguments and results are those of dlm_unmask_select (device pointers, same layouts), for
 * the device that is current on the calling thread.
 * Limit: batch * block_len * ceil(vocab / 4096) <= 65536, otherwise DLM_ERR_WORKSPACE and
 * nothing is launched.
 * The first call on each device looks up the array's device address (a driver query, made
 * with that device current); make that first call before starting any stream capture.
 * Every call on a device shares the one array and leaves its last contents in it.  Nothing
 * in it has to start at zero (each call overwrites the entries it later reads), but two
 * calls that may overlap on the GPU, from different streams or threads, race on it: order them.
 * Not thread-safe for the first call on a device; serialise that one.
 */
int dlm_unmask_select_static(const float* logits, int batch, int block_len, int vocab,
                             uint8_t* masked, int32_t* tokens, int k, int32_t* tok, float* conf,
                             int32_t* sel_idx, int32_t* n_sel, void* stream);

/*
 * dlm_guided_accept — Guided Diffusion accept rule (Sec. 3.2.2 and Algorithm 1).
 *
 * Per batch element, with M = [i_1 < ... < i_m] the masked positions: k = the largest prefix
 * length such that tok_dlm[i_j] == tok_ar[i_j] for all j <= k.  Positions i_1..i_k are
 * accepted; if k == 0 and m > 0, i_1 alone is accepted.  Accepted positions receive the DLM
 * token (fallback_source == 1: the lone fallback position receives the AR token instead),
 * and their mask is cleared.
 *
 *   tok_dlm, tok_ar device, int32 [batch][block_len]  (tok_ar[i] is the guider's prediction
 *                   FOR position i)
 *   masked, tokens  device, in/out as in dlm_unmask_select
 *   accept          device, uint8 [batch][block_len], out (1 = accepted)
 *   acc_idx         device, int32 [batch][block_len], out: accepted positions ascending, rest -1
 *   n_acc           device, int32 [batch], out
 * Supported: block_len <= 1024.
 */
int dlm_guided_accept(dlm_ctx* ctx, const int32_t* tok_dlm, const int32_t* tok_ar, int batch,
                      int block_len, uint8_t* masked, int32_t* tokens, int fallback_source,
                      uint8_t* accept, int32_t* acc_idx, int32_t* n_acc, void* stream);

/*
 * dlm_guided_accept_topk — the "Top-K Match" variant of the accept rule (App. C.1, Table 7: Top-1 / Top-2 /
 * Top-5 match; App. C.3 configuration table: "Top-K Assisted Tokens Selection", default 2).
 *
 * As dlm_guided_accept, except that position i counts as agreeing when tok_dlm[i] equals ANY of the
 * guider's top_k tokens for position i.  The paper names the variant without a formula; this is the reading
 * taken.  top_k = 1 is dlm_guided_accept.
 *
 *   tok_ar_topk  device, int32 [batch][block_len][top_k], the guider's tokens for each position in rank
 *                order (entry 0 is its argmax, which is also the AR token of fallback_source == 1)
 * Supported: block_len <= 1024, 1 <= top_k <= 64.
 */
int dlm_guided_accept_topk(dlm_ctx* ctx, const int32_t* tok_dlm, const int32_t* tok_ar_topk, int top_k, int batch,
                           int block_len, uint8_t* masked, int32_t* tokens, int fallback_source,
                           uint8_t* accept, int32_t* acc_idx, int32_t* n_acc, void* stream);

/*
 * dlm_unmask_select_scored — top-k unmasking ranked by a choice of score, all computed in one pass over the
 * vocabulary (Sec. 3.1 and the figure on accuracy against the number of denoising steps name, as baselines, a
 * MaskGIT-style sampler, an entropy-based one and a Top-K margin one; Eq. 3 still fills with the argmax).
 * The paper prints no formula for them.  READINGS taken here (parity is pinned to these readings), for a masked
 * position with logit row z, p = softmax(z), p_(1) >= p_(2) its two largest entries (a value that occurs twice
 * counts twice):
 *   DLM_SCORE_CONFIDENCE           score = p_(1)                               (= dlm_unmask_select)
 *   DLM_SCORE_NEG_ENTROPY          score = sum_v p_v ln p_v                    (most certain distribution first)
 *   DLM_SCORE_MARGIN               score = p_(1) - p_(2)                       (Top-K margin with K = 2)
 *   DLM_SCORE_LOG_CONF_PLUS_NOISE  score = ln p_(1) + noise[b][i]              (MaskGIT-style: the caller draws the
 *                                   noise, e.g. temperature * Gumbel, so the call itself stays deterministic)
 * Per batch element the k_eff = min(k, number of masked positions) masked positions of largest score are unmasked,
 * ties to the lowest position; outputs as dlm_unmask_select, plus
 *   score  device, fp32 [batch][block_len], out: the ranking score (0 at unmasked positions)
 *   zmax   device, fp32 [batch][block_len], out: the largest logit of the row (0 at unmasked positions); this is
 *          the "maximum token logit of the diffusion output" that dlm_guided_accept_threshold takes
 *   noise  device, fp32 [batch][block_len]; read only for DLM_SCORE_LOG_CONF_PLUS_NOISE, may be NULL otherwise
 * k == 0 writes tok, conf, score and zmax only.  Workspace from dlm_unmask_scored_workspace_bytes, 16-byte aligned.
 * Supported: block_len <= 1024.  score_kind outside the four constants is DLM_ERR_SHAPE.
 */
enum { DLM_SCORE_CONFIDENCE = 0, DLM_SCORE_NEG_ENTROPY = 1, DLM_SCORE_MARGIN = 2, DLM_SCORE_LOG_CONF_PLUS_NOISE = 3 };
size_t dlm_unmask_scored_workspace_bytes(const dlm_ctx* ctx, int batch, int block_len, int vocab);
int dlm_unmask_select_scored(dlm_ctx* ctx, const float* logits, int batch, int block_len, int vocab,
                             uint8_t* masked, int32_t* tokens, int k, int score_kind, const float* noise,
                             int32_t* tok, float* conf, float* score, float* zmax, int32_t* sel_idx,
                             int32_t* n_sel, void* workspace, size_t workspace_bytes, void* stream);

/*
 * dlm_guided_accept_threshold — the accept rule with the guidance confidence threshold (App. C.3 "Stochastic
 * Guided Unmasking"; configuration table: Top-K Assisted Tokens Selection = 2, Guidance Confidence Threshold
 * tau = 0.5).  The passage is short and refers to an "Algorithm 2" that the paper does not contain.  READING taken
 * (parity is pinned to this reading): the result is the union of
 *   (1) the deterministic rule: dlm_guided_accept_topk with the same top_k, fallback included, and
 *   (2) every masked position i with  zmax_dlm[i] > tau * max_j logit_ar_topk[i][j]   (raw logits, as the passage
 *       says; product and comparison in fp32),
 * reported in ascending position order.  Accepted positions receive the DLM token; a position accepted by the
 * fallback alone receives the guider's first token when fallback_source == 1.  The accepted set is in general not
 * a prefix: commit it with its index list (dlm_kv_cache_commit with src_idx = acc_idx).
 *
 *   zmax_dlm       device, fp32 [batch][block_len]: largest DLM logit per position (dlm_unmask_select_scored)
 *   tok_ar_topk    device, int32 [batch][block_len][top_k], the guider's tokens in rank order
 *   logit_ar_topk  device, fp32  [batch][block_len][top_k], their logits
 *   other arguments as dlm_guided_accept_topk.
 * Supported: block_len <= 1024, 1 <= top_k <= 64; a NaN tau is DLM_ERR_UNSUPPORTED.
 */
int dlm_guided_accept_threshold(dlm_ctx* ctx, const int32_t* tok_dlm, const float* zmax_dlm,
                                const int32_t* tok_ar_topk, const float* logit_ar_topk, int top_k, float tau,
                                int batch, int block_len, uint8_t* masked, int32_t* tokens, int fallback_source,
                                uint8_t* accept, int32_t* acc_idx, int32_t* n_acc, void* stream);

/*
 * dlm_window_qkv_project / dlm_window_out_project — the dense projections either side of the attention step
 * (Table 1 rows "Q/K/V projection" and "output projection"; Sec. 3.2.1 "Windowed Re-computation": the window's
 * K/V are recomputed from its hidden states in every step).  bf16 inputs, fp32 accumulation, bf16 outputs.
 *
 * dlm_window_qkv_project: for output feature n = head * head_dim + d, with the heads ordered query heads, key
 * heads, value heads:      y[b][i][n] = bias[n] + sum_c x[b][i][c] * w[n][c]
 * written head by head in the layout dlm_freecache_attn_step reads, so no transpose sits between the two calls:
 *   x      device, bf16 [batch][q_cap][d_model]
 *   w      device, bf16 [(n_q_heads + 2 n_kv_heads) * head_dim][d_model]   (the three matrices stacked by output row)
 *   bias   device, bf16 [(n_q_heads + 2 n_kv_heads) * head_dim] or NULL
 *   q_out  device, bf16 [batch][n_q_heads][q_cap][head_dim];  k_out, v_out  bf16 [batch][n_kv_heads][q_cap][head_dim]
 * Supported: d_model a multiple of 64, (n_q_heads + 2 n_kv_heads) * head_dim a multiple of 128, head_dim a multiple
 * of 8, 16-byte aligned pointers.
 *
 * dlm_window_out_project: y[b][i][m] = bias[m] + sum_{h,d} o[b][h][i][d] * wo[m][h * head_dim + d]
 *   o      device, bf16 [batch][n_q_heads][q_cap][head_dim]   (the attention step's output, read in place)
 *   wo     device, bf16 [d_model][n_q_heads * head_dim];  bias bf16 [d_model] or NULL
 *   y      device, bf16 [batch][q_cap][d_model]
 * Supported: d_model a multiple of 128, head_dim a multiple of 64, batch * q_cap <= 256, and q_cap a multiple of 8
 * when batch > 1.
 *
 * workspace: device, 256-byte aligned, at least dlm_window_proj_workspace_bytes(ctx, rows = batch * q_cap,
 * n_out = output features, k_total = contraction length) bytes: fp32 partial tiles of the K split.
 */
size_t dlm_window_proj_workspace_bytes(const dlm_ctx* ctx, int rows, int n_out, int k_total);
int dlm_window_qkv_project(dlm_ctx* ctx, const void* x, const void* w, const void* bias, int batch, int q_cap,
                           int d_model, int n_q_heads, int n_kv_heads, int head_dim, void* q_out, void* k_out,
                           void* v_out, void* workspace, size_t workspace_bytes, void* stream);
int dlm_window_out_project(dlm_ctx* ctx, const void* o, const void* wo, const void* bias, int batch, int q_cap,
                           int d_model, int n_q_heads, int head_dim, void* y, void* workspace,
                           size_t workspace_bytes, void* stream);

/*
 * dlm_window_qkv_project_rope — dlm_window_qkv_project with the rotary position embedding of the query and key heads
 * applied in the projection's epilogue, before the one rounding to bf16, so that no separate pass over Q and K sits
 * between the projection and dlm_freecache_attn_step.  The paper does not describe the models' position encoding (it
 * runs stock Dream-7B and LLaDA-8B, Sec. 4); both use the rotary embedding of Su et al. (RoFormer) in the half-split
 * layout.  READING taken (the oracle states the same): within a head, feature d < head_dim / 2 is paired with feature
 * d + head_dim / 2 and, with the row's angles,
 *     out[d]                = y[d] * cos[d] - y[d + head_dim / 2] * sin[d]
 *     out[d + head_dim / 2] = y[d + head_dim / 2] * cos[d] + y[d] * sin[d]          (y includes the bias; fp32)
 * for the query heads and the key heads; the value heads are written as they are.
 *   rope_cos, rope_sin   device, fp32 [batch][q_cap][head_dim / 2], 16-byte aligned: cosine and sine of the angle of
 *                        every (row, pair); the caller computes them from the rows' positions (a window row of
 *                        sequence b at position t has angle t * base^(-2 d / head_dim) in the usual parametrisation)
 *   other arguments, workspace and supported shapes as dlm_window_qkv_project; in addition head_dim in {64, 128}
 *   (DLM_ERR_UNSUPPORTED otherwise), rope_cos and rope_sin not NULL (DLM_ERR_NULL).
 */
int dlm_window_qkv_project_rope(dlm_ctx* ctx, const void* x, const void* w, const void* bias, const float* rope_cos,
                                const float* rope_sin, int batch, int q_cap, int d_model, int n_q_heads,
                                int n_kv_heads, int head_dim, void* q_out, void* k_out, void* v_out, void* workspace,
                                size_t workspace_bytes, void* stream);

/*
 * dlm_window_qkv_project_stage — the projection (with the rotary embedding when rope_cos / rope_sin are given, as
 * dlm_window_qkv_project_rope; both NULL: none) that also stages the window's K/V rows in the cache from its epilogue
 * (Sec. 3.2.1 "Windowed Re-computation": the active block's K/V are recomputed in every step; "upon completion of
 * block B_i, its KV projections are frozen").  Beside k_out / v_out, row i of sequence b is written to cache row
 * cache_len[b] + i of layer `layer` (K and V), the slot dlm_kv_cache_commit's DLM_DST_WINDOW mode uses, with the
 * same bits as in k_out / v_out.  cache_len is not changed: the staged rows stay invisible to
 * dlm_freecache_attn_step until the caller advances cache_len[b] by the block's length when the block is complete,
 * and the rows staged by the block's last step are then the frozen ones; no separate copy of the block is needed.
 *   q_len   device, int32 [batch] or NULL: only rows i < q_len[b] are staged (NULL: all q_cap rows); q_out, k_out
 *           and v_out hold all q_cap rows either way
 *   cache   its k / v / cache_len are device pointers as for dlm_kv_cache_commit; batch, n_kv_heads and head_dim
 *           must match the call's (DLM_ERR_SHAPE), 0 <= layer < n_layers
 * Data-dependent: a row whose slot lies at or beyond the capacity is not staged and DLM_ERR_CAPACITY is recorded.
 * A step of a model then needs no dlm_kv_cache_commit call at all; the commit entry point remains for refreshes
 * and for rows chosen after the fact.
 */
int dlm_window_qkv_project_stage(dlm_ctx* ctx, const void* x, const void* w, const void* bias, const float* rope_cos,
                                 const float* rope_sin, int batch, int q_cap, int d_model, int n_q_heads,
                                 int n_kv_heads, int head_dim, const int32_t* q_len, void* q_out, void* k_out,
                                 void* v_out, const dlm_kv_cache* cache, int layer, void* workspace,
                                 size_t workspace_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* DLM_H_ */
