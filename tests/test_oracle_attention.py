"""Pins for the attention oracle: fp64 brute force over the whole sequence, the FreeCache
invariant, split/permutation invariance, a library SDPA, closed forms and poison rows.
None of these re-types the oracle's loop: each compares it with an independent definition."""
import numpy as np
import pytest
import torch

from workloads import make_kv_rows, widen


def _rand(shape, seed):
    return widen(make_kv_rows(shape, seed))


def full_bidirectional_attention_fp64(Q, K, V, scale, group):
    """Textbook softmax(Q K^T * scale) V over one whole sequence, fp64, matrices only.
    Q [Hq, L, D]; K, V [Hkv, L, D]; query head h reads KV head h // group."""
    Q, K, V = (x.astype(np.float64) for x in (Q, K, V))
    Kr = np.repeat(K, group, axis=0)
    Vr = np.repeat(V, group, axis=0)
    S = np.einsum("hid,hjd->hij", Q, Kr) * scale
    S = S - S.max(axis=-1, keepdims=True)
    P = np.exp(S)
    P = P / P.sum(axis=-1, keepdims=True)
    return np.einsum("hij,hjd->hid", P, Vr)


@pytest.mark.parametrize("Hq,Hkv,D,Lc,Lq", [
    (4, 2, 64, 256, 32),     # the tiny workload's shape
    (7, 1, 16, 37, 5),       # group of 7, ragged sizes
    (2, 2, 8, 0, 9),         # empty cache
    (1, 1, 128, 70, 64),
    (6, 3, 32, 19, 1),
])
def test_freecache_step_equals_rows_of_uncached_full_attention(oracle, Hq, Hkv, D, Lc, Lq):
    """If the cache holds this step's K/V of the context, the step equals rows [Lc, Lc+Lq) of
    full bidirectional attention over the concatenated sequence (Sec. 3.2.1)."""
    B, L, g = 2, Lc + Lq, Hq // Hkv
    scale = 1.0 / np.sqrt(D)
    Lcap = Lc + 3                                  # extra never-visible rows
    cache_k = _rand((B, Hkv, Lcap, D), 11)
    cache_v = _rand((B, Hkv, Lcap, D), 12)
    q = _rand((B, Hq, Lq, D), 13)
    k_new = _rand((B, Hkv, Lq, D), 14)
    v_new = _rand((B, Hkv, Lq, D), 15)
    cache_len = np.full((B,), Lc, np.int32)
    out, lse = oracle.attn_step(cache_k, cache_v, cache_len, q, k_new, v_new)
    for b in range(B):
        Kfull = np.concatenate([cache_k[b, :, :Lc], k_new[b]], axis=1)
        Vfull = np.concatenate([cache_v[b, :, :Lc], v_new[b]], axis=1)
        # queries of the context rows are irrelevant to the active rows: fill them with noise
        Qfull = np.concatenate([_rand((Hq, Lc, D), 16 + b), q[b]], axis=1)
        ref = full_bidirectional_attention_fp64(Qfull, Kfull, Vfull, scale, g)[:, Lc:]
        assert ref.shape == (Hq, Lq, D)
        np.testing.assert_allclose(out[b], ref, rtol=0, atol=2e-6)
        S = np.einsum("hid,hjd->hij", q[b].astype(np.float64), np.repeat(Kfull, g, 0).astype(np.float64)) * scale
        ref_lse = np.log(np.exp(S - S.max(-1, keepdims=True)).sum(-1)) + S.max(-1)
        np.testing.assert_allclose(lse[b], ref_lse, rtol=1e-6, atol=1e-6)


def test_matches_library_sdpa_with_repeated_kv_heads(oracle):
    """cache_len = 0 reduces to plain SDPA; GQA = MHA with each KV head repeated g times."""
    B, Hq, Hkv, D, Lq = 2, 8, 2, 64, 48
    q = make_kv_rows((B, Hq, Lq, D), 21)
    k = make_kv_rows((B, Hkv, Lq, D), 22)
    v = make_kv_rows((B, Hkv, Lq, D), 23)
    ref = torch.nn.functional.scaled_dot_product_attention(
        q.float(), k.float().repeat_interleave(Hq // Hkv, dim=1),
        v.float().repeat_interleave(Hq // Hkv, dim=1)).numpy()
    empty = np.zeros((B, Hkv, 4, D), np.float32)
    out, _ = oracle.attn_step(empty, empty, np.zeros(B, np.int32), widen(q), widen(k), widen(v))
    np.testing.assert_allclose(out, ref, rtol=0, atol=3e-6)


def test_split_and_permutation_invariance(oracle):
    """Which part (cache or fresh) a key row sits in, and the order of cached rows, do not matter."""
    B, Hq, Hkv, D, Lc, Lq = 1, 4, 2, 32, 40, 8
    ck, cv = _rand((B, Hkv, Lc, D), 31), _rand((B, Hkv, Lc, D), 32)
    q, kn, vn = _rand((B, Hq, Lq, D), 33), _rand((B, Hkv, Lq, D), 34), _rand((B, Hkv, Lq, D), 35)
    base, base_lse = oracle.attn_step(ck, cv, np.array([Lc], np.int32), q, kn, vn)
    perm = np.random.default_rng(3).permutation(Lc)
    out, lse = oracle.attn_step(np.ascontiguousarray(ck[:, :, perm]), np.ascontiguousarray(cv[:, :, perm]),
                                np.array([Lc], np.int32), q, kn, vn)
    np.testing.assert_allclose(out, base, atol=1e-6)
    np.testing.assert_allclose(lse, base_lse, atol=1e-6)
    # move the last 5 cached rows to the front of a wider fresh part; the first 5 queries are
    # new rows, the remaining Lq must reproduce the base result
    kn2 = np.ascontiguousarray(np.concatenate([ck[:, :, Lc - 5:], kn], axis=2))
    vn2 = np.ascontiguousarray(np.concatenate([cv[:, :, Lc - 5:], vn], axis=2))
    q2 = np.ascontiguousarray(np.concatenate([_rand((B, Hq, 5, D), 36), q], axis=2))
    out2, _ = oracle.attn_step(ck, cv, np.array([Lc - 5], np.int32), q2, kn2, vn2)
    np.testing.assert_allclose(out2[:, :, 5:], base, atol=1e-6)


def test_closed_forms(oracle):
    B, Hq, Hkv, D, Lc, Lq = 1, 2, 1, 16, 12, 4
    q = _rand((B, Hq, Lq, D), 41)
    one_key = _rand((1, 1, 1, D), 42)
    # all keys equal -> uniform weights -> output is the mean of the V rows
    ck = np.ascontiguousarray(np.broadcast_to(one_key, (B, Hkv, Lc, D)))
    kn = np.ascontiguousarray(np.broadcast_to(one_key, (B, Hkv, Lq, D)))
    cv, vn = _rand((B, Hkv, Lc, D), 43), _rand((B, Hkv, Lq, D), 44)
    out, _ = oracle.attn_step(ck, cv, np.array([Lc], np.int32), q, kn, vn)
    mean_v = np.concatenate([cv, vn], axis=2).astype(np.float64).mean(axis=2)   # [B,Hkv,D]
    np.testing.assert_allclose(out, np.broadcast_to(mean_v[:, :, None, :], out.shape), atol=1e-6)
    # all V rows equal to v -> output v whatever the scores
    v = _rand((1, 1, 1, D), 45)
    cv2 = np.ascontiguousarray(np.broadcast_to(v, (B, Hkv, Lc, D)))
    vn2 = np.ascontiguousarray(np.broadcast_to(v, (B, Hkv, Lq, D)))
    out, _ = oracle.attn_step(_rand((B, Hkv, Lc, D), 46), cv2, np.array([Lc], np.int32), q,
                              _rand((B, Hkv, Lq, D), 47), vn2)
    np.testing.assert_allclose(out, np.broadcast_to(v, out.shape), atol=1e-6)
    # zero queries -> all scores zero -> lse = log(number of keys)
    _, lse = oracle.attn_step(ck, cv, np.array([Lc], np.int32), np.zeros_like(q), kn, vn)
    np.testing.assert_allclose(lse, np.log(Lc + Lq), rtol=1e-6)


def test_scale_is_applied_to_scores_only(oracle):
    """Doubling the scale equals doubling q; a sign error or a scale on V would break this."""
    B, Hq, Hkv, D, Lc, Lq = 1, 2, 2, 16, 9, 3
    ck, cv = _rand((B, Hkv, Lc, D), 51), _rand((B, Hkv, Lc, D), 52)
    q, kn, vn = _rand((B, Hq, Lq, D), 53), _rand((B, Hkv, Lq, D), 54), _rand((B, Hkv, Lq, D), 55)
    cl = np.array([Lc], np.int32)
    a, _ = oracle.attn_step(ck, cv, cl, q, kn, vn, scale=0.5)
    b, _ = oracle.attn_step(ck, cv, cl, (2 * q).astype(np.float32), kn, vn, scale=0.25)
    np.testing.assert_allclose(a, b, atol=1e-6)
    # default scale is 1/sqrt(D)
    c, _ = oracle.attn_step(ck, cv, cl, q, kn, vn)
    d, _ = oracle.attn_step(ck, cv, cl, q, kn, vn, scale=0.25)
    np.testing.assert_allclose(c, d, atol=0)


def test_rows_beyond_cache_len_and_q_len_never_leak(oracle):
    B, Hq, Hkv, D, Lcap, q_cap = 2, 4, 2, 16, 24, 6
    ck, cv = _rand((B, Hkv, Lcap, D), 61), _rand((B, Hkv, Lcap, D), 62)
    q, kn, vn = _rand((B, Hq, q_cap, D), 63), _rand((B, Hkv, q_cap, D), 64), _rand((B, Hkv, q_cap, D), 65)
    cache_len = np.array([10, 17], np.int32)
    q_len = np.array([6, 4], np.int32)
    base, base_lse = oracle.attn_step(ck, cv, cache_len, q, kn, vn, q_len)
    ckp, cvp, knp, vnp, qp = (x.copy() for x in (ck, cv, kn, vn, q))
    for b in range(B):
        ckp[b, :, cache_len[b]:] = np.nan
        cvp[b, :, cache_len[b]:] = np.nan
        knp[b, :, q_len[b]:] = np.nan
        vnp[b, :, q_len[b]:] = np.nan
        qp[b, :, q_len[b]:] = np.nan
    out, lse = oracle.attn_step(ckp, cvp, cache_len, qp, knp, vnp, q_len)
    np.testing.assert_array_equal(out, base)
    np.testing.assert_array_equal(lse, base_lse)
    assert np.all(out[1, :, 4:] == 0) and np.all(np.isneginf(lse[1, :, 4:]))
    # ragged batch element == the same element run alone with trimmed tensors
    solo, _ = oracle.attn_step(np.ascontiguousarray(ck[1:2, :, :17]), np.ascontiguousarray(cv[1:2, :, :17]),
                               np.array([17], np.int32), np.ascontiguousarray(q[1:2, :, :4]),
                               np.ascontiguousarray(kn[1:2, :, :4]), np.ascontiguousarray(vn[1:2, :, :4]))
    np.testing.assert_allclose(out[1:2, :, :4], solo, atol=1e-6)
