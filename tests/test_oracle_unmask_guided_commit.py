"""Pins for the integer parts of the oracle: cache commit, confidence / top-k unmasking and the
guided accept rule, against hand-worked fixtures, closed forms, sorting and exhaustive enumeration."""
import itertools
import math
import os

import numpy as np
import pytest

from workloads import make_kv_rows, make_logits, make_mask, bf16_bits

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------- commit
def _commit_case(seed, NL=3, B=2, Hkv=2, Lcap=20, D=8, src_len=6):
    ck = bf16_bits(make_kv_rows((NL, B, Hkv, Lcap, D), seed)).copy()
    cv = bf16_bits(make_kv_rows((NL, B, Hkv, Lcap, D), seed + 1)).copy()
    kn = bf16_bits(make_kv_rows((NL, B, Hkv, src_len, D), seed + 2)).copy()
    vn = bf16_bits(make_kv_rows((NL, B, Hkv, src_len, D), seed + 3)).copy()
    return ck, cv, kn, vn


def test_commit_scatter_moves_exactly_the_named_rows(oracle):
    ck, cv, kn, vn = _commit_case(100)
    ck0, cv0 = ck.copy(), cv.copy()
    cache_len = np.array([5, 9], np.int32)
    src_idx = np.array([[4, 0, 2], [1, 5, 0]], np.int32)
    dst_pos = np.array([[7, 19, 0], [3, 4, 0]], np.int32)
    n_rows = np.array([3, 2], np.int32)
    rc = oracle.kv_cache_commit(ck, cv, cache_len, kn, vn, src_idx, dst_pos, n_rows)
    assert rc == 0
    touched = np.zeros(ck.shape[:4], bool)
    for b in range(2):
        for r in range(n_rows[b]):
            np.testing.assert_array_equal(ck[:, b, :, dst_pos[b, r]], kn[:, b, :, src_idx[b, r]])
            np.testing.assert_array_equal(cv[:, b, :, dst_pos[b, r]], vn[:, b, :, src_idx[b, r]])
            touched[:, b, :, dst_pos[b, r]] = True
    np.testing.assert_array_equal(ck[~touched], ck0[~touched])
    np.testing.assert_array_equal(cv[~touched], cv0[~touched])
    np.testing.assert_array_equal(cache_len, [5, 9])          # staged: visibility unchanged


def test_commit_append_and_layer_range(oracle):
    ck, cv, kn, vn = _commit_case(200)
    ck0 = ck.copy()
    cache_len = np.array([5, 9], np.int32)
    n_rows = np.array([6, 2], np.int32)
    rc = oracle.kv_cache_commit(ck, cv, cache_len, kn[1:3].copy(), vn[1:3].copy(), n_rows=n_rows,
                                advance_len=True, layer_begin=1, layer_end=3)
    assert rc == 0
    np.testing.assert_array_equal(cache_len, [11, 11])
    np.testing.assert_array_equal(ck[0], ck0[0])              # layer 0 not in range
    np.testing.assert_array_equal(ck[1:3, 0, :, 5:11], kn[1:3, 0, :, 0:6])
    np.testing.assert_array_equal(ck[1:3, 1, :, 9:11], kn[1:3, 1, :, 0:2])
    np.testing.assert_array_equal(ck[1:3, 1, :, 11:], ck0[1:3, 1, :, 11:])
    np.testing.assert_array_equal(ck[1:3, :, :, :5], ck0[1:3, :, :, :5])


def test_commit_refresh_from_empty_is_a_plain_copy(oracle):
    ck, cv, kn, vn = _commit_case(300, Lcap=6, src_len=6)
    cache_len = np.zeros(2, np.int32)
    assert oracle.kv_cache_commit(ck, cv, cache_len, kn, vn, advance_len=True) == 0
    np.testing.assert_array_equal(ck, kn)
    np.testing.assert_array_equal(cv, vn)
    np.testing.assert_array_equal(cache_len, [6, 6])


def test_commit_errors_leave_memory_alone(oracle):
    ck, cv, kn, vn = _commit_case(400)
    ck0, cv0 = ck.copy(), cv.copy()
    cache_len = np.array([18, 2], np.int32)                    # 18 + 6 > 20: capacity error for b = 0
    rc = oracle.kv_cache_commit(ck, cv, cache_len, kn, vn, advance_len=True)
    assert rc == oracle.ERR_CAPACITY
    np.testing.assert_array_equal(ck[:, 0], ck0[:, 0])
    np.testing.assert_array_equal(cache_len, [18, 8])
    np.testing.assert_array_equal(ck[:, 1, :, 2:8], kn[:, 1])
    ck, cv = ck0.copy(), cv0.copy()
    src_idx = np.array([[0, 6], [-1, 1]], np.int32)            # 6 and -1 are out of range
    dst_pos = np.array([[1, 2], [3, 20]], np.int32)            # 20 is out of range
    rc = oracle.kv_cache_commit(ck, cv, np.array([0, 0], np.int32), kn, vn, src_idx, dst_pos)
    assert rc == oracle.ERR_INDEX
    np.testing.assert_array_equal(ck[:, 0, :, 1], kn[:, 0, :, 0])
    ck[:, 0, :, 1] = ck0[:, 0, :, 1]
    np.testing.assert_array_equal(ck, ck0)


# ------------------------------------------------------------------- confidence / top-k
def _parse_topk_fixture():
    ln = {"ln9": np.float32(math.log(9.0)), "ln3": np.float32(math.log(3.0))}
    rows, select = {}, {}
    masked = tok = conf = None
    for line in open(os.path.join(GOLDEN, "unmask_topk_handworked.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, val = line.split(":")
        vals = val.split()
        if key == "masked":
            masked = np.array(vals, np.uint8)
        elif key.startswith("row"):
            rows[int(key.split()[1])] = [ln[v] if v in ln else np.float32(float(v)) for v in vals]
        elif key == "tok":
            tok = np.array(vals, np.int32)
        elif key == "conf":
            conf = np.array(vals, np.float32)
        elif key.startswith("select"):
            select[int(key.split()[1])] = np.array(vals, np.int32)
    logits = np.array([rows[i] for i in range(len(rows))], np.float32)[None]
    return logits, masked[None], tok, conf, select


def test_topk_handworked_fixture(oracle):
    logits, masked0, tok_ref, conf_ref, select = _parse_topk_fixture()
    for k, want in select.items():
        masked = masked0.copy()
        tokens = np.full(masked.shape, 99, np.int32)
        tok, conf, sel_idx, n_sel = oracle.unmask_select(logits, masked, tokens, k)
        np.testing.assert_array_equal(tok[0], tok_ref)
        np.testing.assert_allclose(conf[0], conf_ref, rtol=2e-7)
        assert n_sel[0] == len(want)
        np.testing.assert_array_equal(sel_idx[0, :len(want)], want)
        assert np.all(sel_idx[0, len(want):] == -1)
        expect_mask = masked0[0].copy()
        expect_mask[want] = 0
        np.testing.assert_array_equal(masked[0], expect_mask)
        expect_tokens = np.full(6, 99, np.int32)
        expect_tokens[want] = tok_ref[want]
        np.testing.assert_array_equal(tokens[0], expect_tokens)
    # propose only: nothing but tok / conf is produced
    masked, tokens = masked0.copy(), np.full(masked0.shape, 99, np.int32)
    tok, conf, sel_idx, n_sel = oracle.unmask_select(logits, masked, tokens, 0)
    np.testing.assert_array_equal(masked, masked0)
    assert np.all(tokens == 99) and sel_idx is None and n_sel is None
    np.testing.assert_array_equal(tok[0], tok_ref)


def test_confidence_closed_forms(oracle):
    V = 1024
    ones = np.ones((1, 3), np.uint8)
    z = np.zeros((1, 3, V), np.float32)
    z[0, 0, :] = -2.5                       # constant row: conf = 1/V exactly, tok = 0
    a = np.float32(1.75)
    z[0, 1, 700] = a                        # one logit a, rest 0: e^a / (e^a + V - 1)
    z[0, 2, 5] = z[0, 2, 900] = 3.0         # duplicate maxima: lowest index
    tok, conf, _, _ = oracle.unmask_select(z, ones.copy(), np.zeros((1, 3), np.int32), 0)
    assert tok[0, 0] == 0 and conf[0, 0] == np.float32(2.0 ** -10)
    assert tok[0, 1] == 700
    np.testing.assert_allclose(conf[0, 1], math.exp(float(a)) / (math.exp(float(a)) + V - 1), rtol=2e-7)
    assert tok[0, 2] == 5
    np.testing.assert_allclose(conf[0, 2], 1.0 / (2.0 + (V - 2) * math.exp(-3.0)), rtol=2e-7)
    # -inf logits contribute nothing
    z2 = np.full((1, 1, 8), -np.inf, np.float32)
    z2[0, 0, 3] = 0.0
    z2[0, 0, 6] = 0.0
    tok, conf, _, _ = oracle.unmask_select(z2, np.ones((1, 1), np.uint8), np.zeros((1, 1), np.int32), 0)
    assert tok[0, 0] == 3 and conf[0, 0] == np.float32(0.5)


@pytest.mark.parametrize("seed", range(6))
def test_topk_matches_softmax_and_stable_sort(oracle, seed):
    """Random tiny cases: tok/conf against a numpy fp64 softmax, the selection against a
    lexicographic sort on (-conf, position)."""
    B, Lblk, V, k = 3, 11, 37, 1 + seed % 4
    logits = make_logits(B, Lblk, V, (0.5, 4.0), 500 + seed).numpy()
    if seed % 2:
        logits[:, 7] = logits[:, 2]                         # exact ties between positions
    masked0 = make_mask(B, Lblk, 3 + seed, 600 + seed).numpy()
    masked, tokens = masked0.copy(), np.full((B, Lblk), -7, np.int32)
    tok, conf, sel_idx, n_sel = oracle.unmask_select(logits, masked, tokens, k)
    z = logits.astype(np.float64)
    prob = np.exp(z - z.max(-1, keepdims=True))
    prob /= prob.sum(-1, keepdims=True)
    for b in range(B):
        for i in range(Lblk):
            if masked0[b, i]:
                assert tok[b, i] == int(np.argmax(prob[b, i]))      # numpy argmax: first maximum
                np.testing.assert_allclose(conf[b, i], prob[b, i].max(), rtol=3e-7)
                assert 1.0 / V <= conf[b, i] <= 1.0
            else:
                assert tok[b, i] == -1 and conf[b, i] == -1
        cand = [i for i in range(Lblk) if masked0[b, i]]
        order = sorted(cand, key=lambda i: (-float(conf[b, i]), i))
        want = sorted(order[:k])
        assert n_sel[b] == len(want) == min(k, len(cand))
        assert list(sel_idx[b, :len(want)]) == want
        assert [i for i in range(Lblk) if masked0[b, i] and not masked[b, i]] == want


def test_block_empties_in_ceil_m_over_k_steps(oracle):
    B, Lblk, V, k, m = 2, 16, 50, 3, 10
    logits = make_logits(B, Lblk, V, (1.0, 3.0), 700).numpy()
    masked = make_mask(B, Lblk, m, 701).numpy()
    tokens = np.full((B, Lblk), -1, np.int32)
    steps = 0
    while masked.any():
        before = masked.sum(1)
        _, _, _, n_sel = oracle.unmask_select(logits, masked, tokens, k)
        np.testing.assert_array_equal(before - masked.sum(1), n_sel)
        steps += 1
    assert steps == math.ceil(m / k)
    _, _, _, n_sel = oracle.unmask_select(logits, masked, tokens, k)   # nothing left: no-op
    assert np.all(n_sel == 0)


# ------------------------------------------------------------------------ guided accept
def test_guided_handworked_fixture(oracle):
    for line in open(os.path.join(GOLDEN, "guided_accept_handworked.txt")):
        if not line.strip() or line.startswith("#"):
            continue
        f = [np.array(x.split(), np.int64) for x in line.rstrip("\n").split("|")]
        masked0, dlm, ar, want, w0, w1 = f
        for source, written in ((0, w0), (1, w1)):
            masked = masked0.astype(np.uint8)[None].copy()
            tokens = np.full(masked.shape, -5, np.int32)
            accept, acc_idx, n_acc = oracle.guided_accept(
                dlm.astype(np.int32)[None], ar.astype(np.int32)[None], masked, tokens, source)
            assert n_acc[0] == len(want)
            np.testing.assert_array_equal(acc_idx[0, :len(want)], want)
            assert np.all(acc_idx[0, len(want):] == -1)
            exp_accept = np.zeros(len(masked0), np.uint8)
            exp_accept[want] = 1
            np.testing.assert_array_equal(accept[0], exp_accept)
            exp_tokens = np.full(len(masked0), -5, np.int32)
            exp_tokens[want] = written
            np.testing.assert_array_equal(tokens[0], exp_tokens)
            np.testing.assert_array_equal(masked[0], masked0.astype(np.uint8) & (1 - exp_accept))


@pytest.mark.parametrize("m", [1, 2, 5, 10])
def test_guided_exhaustive_agreement_patterns(oracle, m):
    """All 2^m agreement patterns over m masked positions interleaved with unmasked ones:
    n_acc = max(1, number of leading agreements), accepted = the first n_acc masked positions."""
    Lblk = 2 * m + 1
    pos = np.arange(1, Lblk, 2)[:m]                          # masked positions 1, 3, 5, ...
    pats = np.array(list(itertools.product([0, 1], repeat=m)), np.int32)
    B = len(pats)
    masked = np.zeros((B, Lblk), np.uint8)
    masked[:, pos] = 1
    dlm = np.tile(np.arange(100, 100 + Lblk, dtype=np.int32), (B, 1))
    ar = dlm.copy()
    ar[:, ::2] += 50                                         # disagreement at unmasked slots is ignored
    for j, p in enumerate(pos):
        ar[:, p] = np.where(pats[:, j] == 1, dlm[:, p], dlm[:, p] + 1)
    tokens = np.full((B, Lblk), -1, np.int32)
    accept, acc_idx, n_acc = oracle.guided_accept(dlm, ar, masked, tokens)
    for b in range(B):
        lead = 0
        while lead < m and pats[b, lead]:
            lead += 1
        want = max(1, lead)
        assert n_acc[b] == want
        np.testing.assert_array_equal(acc_idx[b, :want], pos[:want])
        assert accept[b].sum() == want and masked[b].sum() == m - want
        np.testing.assert_array_equal(tokens[b, pos[:want]], dlm[b, pos[:want]])


def test_guided_topk_handworked_fixture(oracle):
    for line in open(os.path.join(GOLDEN, "guided_accept_topk_handworked.txt")):
        if not line.strip() or line.startswith("#"):
            continue
        f = line.rstrip("\n").split("|")
        masked0 = np.array(f[0].split(), np.int64)
        dlm = np.array(f[1].split(), np.int32)
        ar = np.array([[int(t) for t in pair.split(",")] for pair in f[2].split()], np.int32)
        want, w0, w1 = (np.array(x.split(), np.int64) for x in f[3:6])
        for source, written in ((0, w0), (1, w1)):
            masked = masked0.astype(np.uint8)[None].copy()
            tokens = np.full(masked.shape, -5, np.int32)
            accept, acc_idx, n_acc = oracle.guided_accept_topk(dlm[None], ar[None], masked, tokens, source)
            assert n_acc[0] == len(want)
            np.testing.assert_array_equal(acc_idx[0, :len(want)], want)
            assert np.all(acc_idx[0, len(want):] == -1)
            exp_tokens = np.full(len(masked0), -5, np.int32)
            exp_tokens[want] = written
            np.testing.assert_array_equal(tokens[0], exp_tokens)
            exp_accept = np.zeros(len(masked0), np.uint8)
            exp_accept[want] = 1
            np.testing.assert_array_equal(accept[0], exp_accept)
            np.testing.assert_array_equal(masked[0], masked0.astype(np.uint8) & (1 - exp_accept))


@pytest.mark.parametrize("K", [1, 2, 5])
def test_guided_topk_against_set_membership_brute_force(oracle, K):
    """Random small blocks against a plain Python statement of the rule with sets; K = 1 must also equal the
    Top-1 rule (itself pinned by the exhaustive test above)."""
    rng = np.random.default_rng(100 + K)
    B, Lblk, V = 300, 9, 6                                  # tiny vocabulary: agreements at every rank are common
    dlm = rng.integers(0, V, (B, Lblk)).astype(np.int32)
    ar = np.stack([rng.permutation(V)[:K] for _ in range(B * Lblk)]).reshape(B, Lblk, K).astype(np.int32)
    masked0 = (rng.random((B, Lblk)) < 0.7).astype(np.uint8)
    for source in (0, 1):
        masked, tokens = masked0.copy(), np.full((B, Lblk), -1, np.int32)
        accept, acc_idx, n_acc = oracle.guided_accept_topk(dlm, ar, masked, tokens, source)
        for b in range(B):
            M = [i for i in range(Lblk) if masked0[b, i]]
            lead = 0
            while lead < len(M) and int(dlm[b, M[lead]]) in set(ar[b, M[lead]].tolist()):
                lead += 1
            want = M[:max(lead, 1)] if M else []
            assert n_acc[b] == len(want) and list(acc_idx[b, :len(want)]) == want
            for i in range(Lblk):
                if i in want:
                    exp = ar[b, i, 0] if (lead == 0 and source == 1) else dlm[b, i]
                    assert tokens[b, i] == exp and masked[b, i] == 0 and accept[b, i] == 1
                else:
                    assert tokens[b, i] == -1 and masked[b, i] == masked0[b, i] and accept[b, i] == 0
        if K == 1:
            m1, t1 = masked0.copy(), np.full((B, Lblk), -1, np.int32)
            a1, i1, n1 = oracle.guided_accept(dlm, ar[:, :, 0].copy(), m1, t1, source)
            np.testing.assert_array_equal(a1, accept)
            np.testing.assert_array_equal(i1, acc_idx)
            np.testing.assert_array_equal(t1, tokens)


def test_commit_window_mode_stages_rows_at_their_own_slots(oracle):
    """dst_mode 1: fresh row p goes to slot cache_len + p, whatever its place in the index list."""
    ck, cv, kn, vn = _commit_case(500)
    ck0 = ck.copy()
    cache_len = np.array([5, 14], np.int32)
    src_idx = np.array([[4, 1], [5, 0]], np.int32)
    rc = oracle.kv_cache_commit(ck, cv, cache_len, kn, vn, src_idx, None, np.array([2, 2], np.int32), dst_mode=1)
    assert rc == 0
    np.testing.assert_array_equal(ck[:, 0, :, 9], kn[:, 0, :, 4])
    np.testing.assert_array_equal(ck[:, 0, :, 6], kn[:, 0, :, 1])
    np.testing.assert_array_equal(ck[:, 1, :, 19], kn[:, 1, :, 5])
    np.testing.assert_array_equal(cv[:, 1, :, 14], vn[:, 1, :, 0])
    ck[:, 0, :, [9, 6]] = ck0[:, 0, :, [9, 6]]
    ck[:, 1, :, [19, 14]] = ck0[:, 1, :, [19, 14]]
    np.testing.assert_array_equal(ck, ck0)
    np.testing.assert_array_equal(cache_len, [5, 14])
    cache_len = np.array([5, 15], np.int32)                     # 15 + 5 = 20 is past the last slot
    assert oracle.kv_cache_commit(ck, cv, cache_len, kn, vn, src_idx, None, np.array([2, 2], np.int32),
                                  dst_mode=1) == oracle.ERR_INDEX
