/*
 * CPU oracle for the FreeCache denoising-step hot path of a diffusion language model.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, obviously-correct statement of
 * what the hot path computes.  It shares no code, header, table or helper with the CUDA
 * library, and the CUDA library never calls it.  Only the tests, the smoke check and the
 * CPU-baseline leg of the benchmark may load it.
 *
 * Precision: floating-point inputs are fp32 (bf16 bit patterns widened exactly by the
 * caller); every sum, dot product and exponential is carried in fp64 and the result is
 * rounded once to fp32.  Integer / byte work is exact.
 *
 * Every function below is pinned by CPU tests to something other than itself (fp64 brute
 * force over the full sequence, closed forms, a library SDPA, hand-worked examples,
 * exhaustive enumeration); none is "parity unpinned".
 *
 * Notation follows the paper: M_t masked set (Eq. 1), z_t logits (Eq. 2), U_t selected set
 * (Eq. 3), blocks B_1..B_N with frozen K/V (Sec. 3.2.1), tok_DLM / tok_AR and the masked
 * index list M = [i_1..i_m] (Algorithm 1).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_ERR_CAPACITY 1 /* bit: an append would run past the cache capacity      */
#define ORACLE_ERR_INDEX 2    /* bit: a source or destination row index is out of range */

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/*
 * One attention step of one layer (Sec. 3.2.1, "Windowed Re-computation"; Table 1 rows
 * QK^T and Attention Score x Value).
 *
 * For batch element b, query head h (KV head h / (Hq/Hkv)) and active row i < q_len[b]:
 * the keys are the visible cached rows j < cache_len[b] (prompt and frozen blocks) followed
 * by the freshly recomputed rows of the active window j' < q_len[b].  There is no causal
 * mask (the model is bidirectional).  With s_j = scale * <q_i, k_j>:
 *     out_i = sum_j softmax(s)_j * v_j,        lse_i = log sum_j exp(s_j).
 * Rows i >= q_len[b] are defined as zero (lse = -inf).
 *
 * Layouts (row-major, innermost last):
 *   cache_k, cache_v : [B][Hkv][Lcap][D]      q   : [B][Hq][q_cap][D]
 *   k_new, v_new     : [B][Hkv][q_cap][D]     out : [B][Hq][q_cap][D]   lse : [B][Hq][q_cap]
 *   cache_len, q_len : [B]  (q_len may be NULL: every row active)
 * Rows of the cache at or beyond cache_len[b] are never read.
 */
int oracle_attn_step(int B, int Hq, int Hkv, int D, int Lcap, int q_cap,
                     const float* cache_k, const float* cache_v, const int32_t* cache_len,
                     const int32_t* q_len, const float* q, const float* k_new,
                     const float* v_new, float scale, float* out, float* lse) {
  if (Hkv <= 0 || Hq % Hkv != 0) return -1;
  const int g = Hq / Hkv;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
  for (int b = 0; b < B; ++b) {
    for (int h = 0; h < Hq; ++h) {
      const int kvh = h / g;
      const int Lc = cache_len[b];
      const int Lq = q_len ? q_len[b] : q_cap;
      const int L = Lc + Lq;
      double* s = (double*)malloc(sizeof(double) * (size_t)(L > 0 ? L : 1));
      double* acc = (double*)malloc(sizeof(double) * (size_t)D);
      const float* Kc = cache_k + ((size_t)b * Hkv + kvh) * (size_t)Lcap * D;
      const float* Vc = cache_v + ((size_t)b * Hkv + kvh) * (size_t)Lcap * D;
      const float* Kn = k_new + ((size_t)b * Hkv + kvh) * (size_t)q_cap * D;
      const float* Vn = v_new + ((size_t)b * Hkv + kvh) * (size_t)q_cap * D;
      for (int i = 0; i < q_cap; ++i) {
        float* o = out + (((size_t)b * Hq + h) * q_cap + i) * D;
        float* l = lse + ((size_t)b * Hq + h) * q_cap + i;
        if (i >= Lq) {
          for (int d = 0; d < D; ++d) o[d] = 0.0f;
          *l = -INFINITY;
          continue;
        }
        const float* qi = q + (((size_t)b * Hq + h) * q_cap + i) * D;
        double m = -INFINITY;
        for (int j = 0; j < L; ++j) {
          const float* kj = (j < Lc) ? Kc + (size_t)j * D : Kn + (size_t)(j - Lc) * D;
          double dot = 0.0;
          for (int d = 0; d < D; ++d) dot += (double)qi[d] * (double)kj[d];
          s[j] = (double)scale * dot;
          if (s[j] > m) m = s[j];
        }
        double denom = 0.0;
        for (int d = 0; d < D; ++d) acc[d] = 0.0;
        for (int j = 0; j < L; ++j) {
          const float* vj = (j < Lc) ? Vc + (size_t)j * D : Vn + (size_t)(j - Lc) * D;
          const double p = exp(s[j] - m);
          denom += p;
          for (int d = 0; d < D; ++d) acc[d] += p * (double)vj[d];
        }
        for (int d = 0; d < D; ++d) o[d] = (float)(acc[d] / denom);
        *l = (float)(m + log(denom));
      }
      free(s);
      free(acc);
    }
  }
  return ORACLE_OK;
}

/*
 * KV-cache commit / refresh (Sec. 3.2.1, "Initialization and Partitioning" saves K/V,
 * "Progressive Caching" freezes them).  Pure data movement on 16-bit patterns.
 *
 * For every layer in [layer_begin, layer_end), batch element b, r < n[b], KV head and both
 * tensors:   cache[layer][b][head][dst(b,r)][:] = new[layer - layer_begin][b][head][src(b,r)][:]
 * with src(b,r) = src_idx ? src_idx[b][r] : r   and
 *      dst(b,r) = dst_pos ? dst_pos[b][r]
 *               : dst_mode == 1 ? cache_len[b] + src(b,r)   (row p of the active window is staged
 *                                                            at its own slot behind the visible rows)
 *               : cache_len[b] + r                          (append),
 * n[b] = n_rows ? n_rows[b] : n_max.  If advance_len != 0, cache_len[b] += n[b] afterwards.
 *
 * Layouts: cache_k/v [NL][B][Hkv][Lcap][D]; k_new/v_new [layer_end-layer_begin][B][Hkv][src_len][D];
 *          src_idx, dst_pos [B][n_max]; n_rows, cache_len [B].
 *
 * Input errors (returned as a bit mask, other batch elements unaffected):
 *   - n[b] outside [0, n_max], or an append / advance that would pass Lcap: nothing is
 *     written for b and cache_len[b] is left alone (ORACLE_ERR_CAPACITY);
 *   - a source index outside [0, src_len) or a destination outside [0, Lcap): that row is
 *     skipped (ORACLE_ERR_INDEX).
 */
int oracle_kv_cache_commit(int NL, int B, int Hkv, int Lcap, int D, uint16_t* cache_k,
                           uint16_t* cache_v, int32_t* cache_len, const uint16_t* k_new,
                           const uint16_t* v_new, int src_len, const int32_t* src_idx,
                           const int32_t* dst_pos, int dst_mode, const int32_t* n_rows, int n_max,
                           int advance_len, int layer_begin, int layer_end) {
  int status = ORACLE_OK;
  if (layer_begin < 0 || layer_end > NL || layer_begin > layer_end) return -1;
  for (int b = 0; b < B; ++b) {
    const int n = n_rows ? n_rows[b] : n_max;
    const int len0 = cache_len[b];
    if (n < 0 || n > n_max) { status |= ORACLE_ERR_CAPACITY; continue; }
    const int append = (dst_pos == NULL && dst_mode == 0);
    if ((append || advance_len) && (len0 < 0 || (int64_t)len0 + n > Lcap)) {
      status |= ORACLE_ERR_CAPACITY;
      continue;
    }
    for (int r = 0; r < n; ++r) {
      const int64_t src = src_idx ? src_idx[(size_t)b * n_max + r] : r;
      const int64_t dst = dst_pos ? dst_pos[(size_t)b * n_max + r]
                                  : (dst_mode == 1 ? (int64_t)len0 + src : (int64_t)len0 + r);
      if (src < 0 || src >= src_len || dst < 0 || dst >= Lcap) { status |= ORACLE_ERR_INDEX; continue; }
      for (int layer = layer_begin; layer < layer_end; ++layer) {
        for (int h = 0; h < Hkv; ++h) {
          const size_t to = ((((size_t)layer * B + b) * Hkv + h) * (size_t)Lcap + (size_t)dst) * D;
          const size_t from = ((((size_t)(layer - layer_begin) * B + b) * Hkv + h) * (size_t)src_len + (size_t)src) * D;
          memcpy(cache_k + to, k_new + from, sizeof(uint16_t) * (size_t)D);
          memcpy(cache_v + to, v_new + from, sizeof(uint16_t) * (size_t)D);
        }
      }
    }
    if (advance_len) cache_len[b] = len0 + n;
  }
  return status;
}

/*
 * Confidence scoring and top-k unmasking (Eq. 2, Eq. 3 and M_{t-1} = M_t \ U_t).
 *
 * For each masked position (b, i) with logit row z over the vocabulary:
 *     tok  = lowest v attaining max_v z_v        (argmax of the softmax = argmax of z),
 *     conf = max softmax probability = 1 / sum_v exp(z_v - max z)   (fp64 sum, rounded to fp32).
 * Unmasked positions get tok = -1, conf = -1.
 * If k > 0: with k_eff = min(k, |M_t| in this batch element), U_t is the k_eff masked
 * positions of largest conf (compared as fp32), ties to the lowest position; then
 * tokens[pos] = tok[pos], masked[pos] = 0, sel_idx[b][0..n_sel) = U_t ascending (rest -1),
 * n_sel[b] = k_eff.  If k == 0 ("propose only") nothing but tok and conf is written,
 * and sel_idx / n_sel may be NULL.
 *
 * Layouts: logits [B][Lblk][V] fp32; masked uint8 [B][Lblk]; tokens, tok int32 [B][Lblk];
 *          conf fp32 [B][Lblk]; sel_idx int32 [B][k]; n_sel int32 [B].
 */
int oracle_unmask_select(int B, int Lblk, int V, const float* logits, uint8_t* masked,
                         int32_t* tokens, int k, int32_t* tok, float* conf, int32_t* sel_idx,
                         int32_t* n_sel) {
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
  for (int b = 0; b < B; ++b) {
    for (int i = 0; i < Lblk; ++i) {
      const size_t p = (size_t)b * Lblk + i;
      if (!masked[p]) { tok[p] = -1; conf[p] = -1.0f; continue; }
      const float* z = logits + p * (size_t)V;
      int best = 0;
      for (int v = 1; v < V; ++v)
        if (z[v] > z[best]) best = v; /* strict: the lowest index wins a tie */
      double sum = 0.0;
      for (int v = 0; v < V; ++v) sum += exp((double)z[v] - (double)z[best]);
      tok[p] = best;
      conf[p] = (float)(1.0 / sum);
    }
  }
  if (k <= 0) return ORACLE_OK;
  for (int b = 0; b < B; ++b) {
    uint8_t* mk = masked + (size_t)b * Lblk;
    const float* cf = conf + (size_t)b * Lblk;
    uint8_t* chosen = (uint8_t*)calloc((size_t)Lblk, 1);
    int n = 0;
    for (int round = 0; round < k; ++round) {
      int best = -1;
      for (int i = 0; i < Lblk; ++i) {
        if (!mk[i] || chosen[i]) continue;
        if (best < 0 || cf[i] > cf[best]) best = i; /* strict: lowest position wins a tie */
      }
      if (best < 0) break;
      chosen[best] = 1;
      ++n;
    }
    int w = 0;
    for (int i = 0; i < Lblk; ++i) {
      if (!chosen[i]) continue;
      sel_idx[(size_t)b * k + w++] = i;
      tokens[(size_t)b * Lblk + i] = tok[(size_t)b * Lblk + i];
      mk[i] = 0;
    }
    for (; w < k; ++w) sel_idx[(size_t)b * k + w] = -1;
    n_sel[b] = n;
    free(chosen);
  }
  return ORACLE_OK;
}

/*
 * Guided Diffusion accept rule (Sec. 3.2.2; Algorithm 1).
 *
 * Per batch element, let M = [i_1 < ... < i_m] be the masked positions.  k is the largest
 * prefix length with tok_dlm[i_j] == tok_ar[i_j] for all j <= k.  If k > 0 positions
 * i_1..i_k are unmasked with the DLM proposals; otherwise only i_1 is unmasked (with the
 * DLM proposal, or with the AR token when fallback_source == 1).  m == 0 accepts nothing.
 * Outputs: accept[b][i] in {0,1}; acc_idx[b][0..n_acc) ascending accepted positions (rest -1);
 * tokens[accepted] written, masked[accepted] cleared.
 *
 * Layouts: tok_dlm, tok_ar, tokens, acc_idx int32 [B][Lblk]; masked, accept uint8 [B][Lblk];
 *          n_acc int32 [B].
 */
int oracle_guided_accept(int B, int Lblk, const int32_t* tok_dlm, const int32_t* tok_ar,
                         uint8_t* masked, int32_t* tokens, int fallback_source,
                         uint8_t* accept, int32_t* acc_idx, int32_t* n_acc) {
  for (int b = 0; b < B; ++b) {
    const size_t o = (size_t)b * Lblk;
    int n = 0, first = -1, still_agreeing = 1;
    for (int i = 0; i < Lblk; ++i) { accept[o + i] = 0; acc_idx[o + i] = -1; }
    for (int i = 0; i < Lblk; ++i) {
      if (!masked[o + i]) continue;
      if (first < 0) first = i;
      if (!still_agreeing) continue;
      if (tok_dlm[o + i] == tok_ar[o + i]) {
        accept[o + i] = 1;
        acc_idx[o + n++] = i;
      } else {
        still_agreeing = 0;
      }
    }
    int fallback = 0;
    if (n == 0 && first >= 0) { /* no agreement at i_1: accept it alone */
      accept[o + first] = 1;
      acc_idx[o + n++] = first;
      fallback = 1;
    }
    for (int j = 0; j < n; ++j) {
      const int i = acc_idx[o + j];
      tokens[o + i] = (fallback && fallback_source == 1) ? tok_ar[o + i] : tok_dlm[o + i];
      masked[o + i] = 0;
    }
    n_acc[b] = n;
  }
  return ORACLE_OK;
}

/*
 * "Top-K Match" variant of the accept rule (App. C.1, Table 7; configuration table of App. C.3).
 * The paper names it without a formula; the reading taken: position i_j agrees when tok_dlm[i_j] equals any
 * of the guider's K tokens for that position.  Everything else is the rule above: longest agreeing prefix
 * over the masked positions in ascending order, the first masked position alone if it does not agree.
 * tok_ar_topk is [B][Lblk][K] in rank order; entry 0 is the guider's argmax (the AR fallback token).
 */
int oracle_guided_accept_topk(int B, int Lblk, int K, const int32_t* tok_dlm, const int32_t* tok_ar_topk,
                              uint8_t* masked, int32_t* tokens, int fallback_source,
                              uint8_t* accept, int32_t* acc_idx, int32_t* n_acc) {
  if (K <= 0) return -1;
  for (int b = 0; b < B; ++b) {
    const size_t o = (size_t)b * Lblk;
    int n = 0, first = -1, still_agreeing = 1;
    for (int i = 0; i < Lblk; ++i) { accept[o + i] = 0; acc_idx[o + i] = -1; }
    for (int i = 0; i < Lblk; ++i) {
      if (!masked[o + i]) continue;
      if (first < 0) first = i;
      if (!still_agreeing) continue;
      int among = 0;
      for (int j = 0; j < K; ++j)
        if (tok_ar_topk[(o + i) * K + j] == tok_dlm[o + i]) among = 1;
      if (among) {
        accept[o + i] = 1;
        acc_idx[o + n++] = i;
      } else {
        still_agreeing = 0;
      }
    }
    int fallback = 0;
    if (n == 0 && first >= 0) {
      accept[o + first] = 1;
      acc_idx[o + n++] = first;
      fallback = 1;
    }
    for (int j = 0; j < n; ++j) {
      const int i = acc_idx[o + j];
      tokens[o + i] = (fallback && fallback_source == 1) ? tok_ar_topk[(o + i) * K] : tok_dlm[o + i];
      masked[o + i] = 0;
    }
    n_acc[b] = n;
  }
  return ORACLE_OK;
}

/*
 * Per-position statistics for the other ways of choosing U_t that the paper names as baselines
 * (Sec. 3.1 and the figure on accuracy against the number of denoising steps: a MaskGIT-style sampler, an
 * entropy-based one and a Top-K margin one).  The paper prints no formula for any of them; the readings taken,
 * for a masked position with logit row z, p = softmax(z), z_(1) >= z_(2) the two largest entries (a value that
 * occurs twice counts twice):
 *     zmax        = z_(1)                                   (the maximum logit)
 *     conf        = p_(1) = 1 / sum_v exp(z_v - z_(1))      (as in oracle_unmask_select)
 *     neg_entropy = sum_v p_v log p_v = -(log S - T / S),   S = sum_v exp(z_v - z_(1)), T = sum_v (z_v - z_(1)) exp(z_v - z_(1))
 *     margin      = p_(1) - p_(2) = (1 - exp(z_(2) - z_(1))) / S        (V == 1: p_(2) = 0)
 * All sums in fp64, each result rounded once to fp32.  -inf entries contribute nothing (0 * -inf is taken as 0).
 * Unmasked positions get tok = -1 and -1 in conf; zmax, neg_entropy and margin are written as 0 there.
 */
int oracle_unmask_scores(int B, int Lblk, int V, const float* logits, const uint8_t* masked, int32_t* tok,
                         float* conf, float* zmax, float* neg_entropy, float* margin) {
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
  for (int b = 0; b < B; ++b) {
    for (int i = 0; i < Lblk; ++i) {
      const size_t p = (size_t)b * Lblk + i;
      if (!masked[p]) { tok[p] = -1; conf[p] = -1.0f; zmax[p] = 0.f; neg_entropy[p] = 0.f; margin[p] = 0.f; continue; }
      const float* z = logits + p * (size_t)V;
      int best = 0;
      for (int v = 1; v < V; ++v)
        if (z[v] > z[best]) best = v;
      double second = -INFINITY; /* largest entry once one occurrence of the maximum is set aside */
      for (int v = 0; v < V; ++v)
        if (v != best && (double)z[v] > second) second = (double)z[v];
      double S = 0.0, T = 0.0;
      for (int v = 0; v < V; ++v) {
        const double d = (double)z[v] - (double)z[best];
        const double e = exp(d);
        S += e;
        if (e > 0.0) T += d * e;
      }
      tok[p] = best;
      zmax[p] = z[best];
      conf[p] = (float)(1.0 / S);
      neg_entropy[p] = (float)(-(log(S) - T / S));
      margin[p] = (float)((1.0 - (V > 1 ? exp(second - (double)z[best]) : 0.0)) / S);
    }
  }
  return ORACLE_OK;
}

/*
 * Top-k unmasking with a choice of score (the readings above; Eq. 3 still fills with the argmax):
 *   kind 0  score = conf                            (oracle_unmask_select)
 *   kind 1  score = neg_entropy                     (entropy-based: most certain distributions first)
 *   kind 2  score = margin                          (Top-K margin with K = 2)
 *   kind 3  score = log(conf) + noise[b][i]         (MaskGIT-style: confidence perturbed by noise that the caller
 *                                                    draws, e.g. temperature * Gumbel; fp64 log, one rounding)
 * The k_eff = min(k, |M_t|) masked positions of largest score (compared as fp32) are unmasked, ties to the lowest
 * position; outputs as in oracle_unmask_select plus score [B][Lblk] (-inf... unmasked positions get score 0) and zmax.
 */
int oracle_unmask_select_scored(int B, int Lblk, int V, const float* logits, uint8_t* masked, int32_t* tokens, int k,
                                int kind, const float* noise, int32_t* tok, float* conf, float* score, float* zmax,
                                int32_t* sel_idx, int32_t* n_sel) {
  if (kind < 0 || kind > 3 || (kind == 3 && !noise)) return -1;
  float* ne = (float*)malloc(sizeof(float) * (size_t)B * Lblk);
  float* mg = (float*)malloc(sizeof(float) * (size_t)B * Lblk);
  oracle_unmask_scores(B, Lblk, V, logits, masked, tok, conf, zmax, ne, mg);
  for (size_t p = 0; p < (size_t)B * Lblk; ++p) {
    if (!masked[p]) { score[p] = 0.f; continue; }
    if (kind == 0) score[p] = conf[p];
    else if (kind == 1) score[p] = ne[p];
    else if (kind == 2) score[p] = mg[p];
    else score[p] = (float)(log((double)conf[p]) + (double)noise[p]);
  }
  free(ne);
  free(mg);
  if (k <= 0) return ORACLE_OK;
  for (int b = 0; b < B; ++b) {
    uint8_t* mk = masked + (size_t)b * Lblk;
    const float* sc = score + (size_t)b * Lblk;
    uint8_t* chosen = (uint8_t*)calloc((size_t)Lblk, 1);
    int n = 0;
    for (int round = 0; round < k; ++round) {
      int best = -1;
      for (int i = 0; i < Lblk; ++i) {
        if (!mk[i] || chosen[i]) continue;
        if (best < 0 || sc[i] > sc[best]) best = i;
      }
      if (best < 0) break;
      chosen[best] = 1;
      ++n;
    }
    int w = 0;
    for (int i = 0; i < Lblk; ++i) {
      if (!chosen[i]) continue;
      sel_idx[(size_t)b * k + w++] = i;
      tokens[(size_t)b * Lblk + i] = tok[(size_t)b * Lblk + i];
      mk[i] = 0;
    }
    for (; w < k; ++w) sel_idx[(size_t)b * k + w] = -1;
    n_sel[b] = n;
    free(chosen);
  }
  return ORACLE_OK;
}

/*
 * Guided accept with the confidence threshold (App. C.3, "Stochastic Guided Unmasking"; configuration table:
 * Top-K Assisted Tokens Selection = 2, Guidance Confidence Threshold tau = 0.5).
 *
 * The passage says, in short: only the guider's Top-K logits count as guidance logits; besides the deterministic
 * rule, a token whose largest diffusion logit exceeds tau times the largest guidance logit is unmasked, and
 * otherwise it stays as it is.  The reading taken:
 *   1. the deterministic rule is the Top-K match accept above, including its fallback (K = 1: Algorithm 1);
 *   2. in addition every masked position i with  zmax_dlm[i] > tau * max_j logit_ar_topk[i][j]  is accepted
 *      (raw logits, as the passage says; the product and the comparison in fp32);
 *   3. the accepted set is the union, reported in ascending position order; accepted positions receive the DLM
 *      token, except a position accepted by the fallback alone, which receives the guider's first token when
 *      fallback_source == 1.
 * Layouts as oracle_guided_accept_topk, plus zmax_dlm fp32 [B][Lblk] and logit_ar_topk fp32 [B][Lblk][K].
 */
int oracle_guided_accept_threshold(int B, int Lblk, int K, const int32_t* tok_dlm, const float* zmax_dlm,
                                   const int32_t* tok_ar_topk, const float* logit_ar_topk, float tau,
                                   uint8_t* masked, int32_t* tokens, int fallback_source, uint8_t* accept,
                                   int32_t* acc_idx, int32_t* n_acc) {
  if (K <= 0) return -1;
  for (int b = 0; b < B; ++b) {
    const size_t o = (size_t)b * Lblk;
    int first = -1, still_agreeing = 1, n_prefix = 0;
    for (int i = 0; i < Lblk; ++i) { accept[o + i] = 0; acc_idx[o + i] = -1; }
    /* 1. deterministic rule: longest prefix of masked positions whose DLM token is among the guider's K */
    for (int i = 0; i < Lblk; ++i) {
      if (!masked[o + i]) continue;
      if (first < 0) first = i;
      if (!still_agreeing) continue;
      int among = 0;
      for (int j = 0; j < K; ++j)
        if (tok_ar_topk[(o + i) * K + j] == tok_dlm[o + i]) among = 1;
      if (among) { accept[o + i] = 1; ++n_prefix; } else still_agreeing = 0;
    }
    int fallback_pos = -1;
    if (n_prefix == 0 && first >= 0) { accept[o + first] = 1; fallback_pos = first; }
    /* 2. threshold rule on every masked position */
    for (int i = 0; i < Lblk; ++i) {
      if (!masked[o + i]) continue;
      float g = logit_ar_topk[(o + i) * K];
      for (int j = 1; j < K; ++j)
        if (logit_ar_topk[(o + i) * K + j] > g) g = logit_ar_topk[(o + i) * K + j];
      const float bound = tau * g;
      if (zmax_dlm[o + i] > bound) {
        accept[o + i] = 1;
        if (i == fallback_pos) fallback_pos = -1; /* accepted in its own right */
      }
    }
    /* 3. union, ascending */
    int n = 0;
    for (int i = 0; i < Lblk; ++i) {
      if (!accept[o + i]) continue;
      acc_idx[o + n++] = i;
      tokens[o + i] = (i == fallback_pos && fallback_source == 1) ? tok_ar_topk[(o + i) * K] : tok_dlm[o + i];
      masked[o + i] = 0;
    }
    n_acc[b] = n;
  }
  return ORACLE_OK;
}

/*
 * Fused Q/K/V projection of the active window (Table 1 row "Q/K/V projection"; Sec. 3.2.1 "Windowed
 * Re-computation": the window's K/V are recomputed in every step).
 *
 * x is the window's hidden states [B][q_cap][d_model]; w holds the three projection matrices stacked by output
 * feature, [(Hq + 2 Hkv) * D][d_model] (rows: the Hq query heads, then the Hkv key heads, then the Hkv value heads;
 * within a head the D features in order), bias [(Hq + 2 Hkv) * D] or NULL.  For output feature n = head * D + d:
 *     y[b][i][n] = bias[n] + sum_c x[b][i][c] * w[n][c]              (fp64 sum, one rounding to fp32)
 * and the result is written head by head in the layout the attention step reads:
 *     q_out [B][Hq][q_cap][D],   k_out, v_out [B][Hkv][q_cap][D].
 */
int oracle_qkv_project(int B, int q_cap, int d_model, int Hq, int Hkv, int D, const float* x, const float* w,
                       const float* bias, float* q_out, float* k_out, float* v_out) {
  const int n_out = (Hq + 2 * Hkv) * D;
#pragma omp parallel for collapse(2) schedule(static)
  for (int b = 0; b < B; ++b) {
    for (int n = 0; n < n_out; ++n) {
      const int head = n / D, d = n % D;
      float* dst;
      int heads, h;
      if (head < Hq) { dst = q_out; heads = Hq; h = head; }
      else if (head < Hq + Hkv) { dst = k_out; heads = Hkv; h = head - Hq; }
      else { dst = v_out; heads = Hkv; h = head - Hq - Hkv; }
      for (int i = 0; i < q_cap; ++i) {
        const float* xr = x + ((size_t)b * q_cap + i) * d_model;
        const float* wr = w + (size_t)n * d_model;
        double acc = bias ? (double)bias[n] : 0.0;
        for (int c = 0; c < d_model; ++c) acc += (double)xr[c] * (double)wr[c];
        dst[(((size_t)b * heads + h) * q_cap + i) * D + d] = (float)acc;
      }
    }
  }
  return ORACLE_OK;
}

/*
 * The same projection followed by the rotary position embedding of the query and key heads.  The paper does not
 * describe the models' position encoding (it runs stock Dream-7B and LLaDA-8B checkpoints, Sec. 4); both use the
 * rotary embedding of Su et al. (RoFormer) in the half-split layout of their public implementations.  READING taken:
 * within a head of D features, feature d < D/2 is paired with feature d + D/2, and for the row's angle table
 * (cos, sin fp32 [B][q_cap][D/2], supplied by the caller for the rows' positions):
 *     out[d]       = y[d] * cos[d] - y[d + D/2] * sin[d]
 *     out[d + D/2] = y[d + D/2] * cos[d] + y[d] * sin[d]            (d < D/2; y includes the bias)
 * applied to the Hq query heads and the Hkv key heads; the value heads are left as they are.  The rotation runs on
 * the fp64 sums, one rounding to fp32 at the end.
 */
int oracle_qkv_project_rope(int B, int q_cap, int d_model, int Hq, int Hkv, int D, const float* x, const float* w,
                            const float* bias, const float* rope_cos, const float* rope_sin, float* q_out, float* k_out,
                            float* v_out) {
  if (D % 2 != 0 || D > 1024) return -1;   /* not a head size this checker handles */
  const int half = D / 2;
  const int n_heads = Hq + 2 * Hkv;
#pragma omp parallel for collapse(2) schedule(static)
  for (int b = 0; b < B; ++b) {
    for (int head = 0; head < n_heads; ++head) {
      float* dst;
      int heads, h;
      if (head < Hq) { dst = q_out; heads = Hq; h = head; }
      else if (head < Hq + Hkv) { dst = k_out; heads = Hkv; h = head - Hq; }
      else { dst = v_out; heads = Hkv; h = head - Hq - Hkv; }
      const int rotate = head < Hq + Hkv;
      double y[1024];
      for (int i = 0; i < q_cap; ++i) {
        const float* xr = x + ((size_t)b * q_cap + i) * d_model;
        for (int d = 0; d < D; ++d) {
          const int n = head * D + d;
          const float* wr = w + (size_t)n * d_model;
          double acc = bias ? (double)bias[n] : 0.0;
          for (int c = 0; c < d_model; ++c) acc += (double)xr[c] * (double)wr[c];
          y[d] = acc;
        }
        float* out = dst + (((size_t)b * heads + h) * q_cap + i) * D;
        if (rotate) {
          const float* cs = rope_cos + ((size_t)b * q_cap + i) * half;
          const float* sn = rope_sin + ((size_t)b * q_cap + i) * half;
          for (int d = 0; d < half; ++d) {
            out[d] = (float)(y[d] * (double)cs[d] - y[d + half] * (double)sn[d]);
            out[d + half] = (float)(y[d + half] * (double)cs[d] + y[d] * (double)sn[d]);
          }
        } else {
          for (int d = 0; d < D; ++d) out[d] = (float)y[d];
        }
      }
    }
  }
  return ORACLE_OK;
}

/*
 * Output projection (Table 1 row "output projection"): the attention output [B][Hq][q_cap][D], read with features
 * ordered (head, d), times wo [d_model][Hq * D]:
 *     y[b][i][m] = bias[m] + sum_{h,d} o[b][h][i][d] * wo[m][h * D + d]       -> y [B][q_cap][d_model]
 */
int oracle_out_project(int B, int q_cap, int d_model, int Hq, int D, const float* o, const float* wo,
                       const float* bias, float* y) {
#pragma omp parallel for collapse(2) schedule(static)
  for (int b = 0; b < B; ++b) {
    for (int m = 0; m < d_model; ++m) {
      for (int i = 0; i < q_cap; ++i) {
        double acc = bias ? (double)bias[m] : 0.0;
        for (int h = 0; h < Hq; ++h) {
          const float* orow = o + (((size_t)b * Hq + h) * q_cap + i) * D;
          const float* wr = wo + (size_t)m * Hq * D + (size_t)h * D;
          for (int d = 0; d < D; ++d) acc += (double)orow[d] * (double)wr[d];
        }
        y[((size_t)b * q_cap + i) * d_model + m] = (float)acc;
      }
    }
  }
  return ORACLE_OK;
}
