"""Pins for the oracle's other unmask scores (entropy, top-2 margin, noisy confidence) and for the guided accept
with the confidence threshold: hand-worked fixtures, closed forms, library routines and brute force."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

from workloads import make_logits, make_mask

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
LN = {"ln3": math.log(3.0), "ln4": math.log(4.0), "ln5": math.log(5.0), "ln9": math.log(9.0)}


def _parse_scores_fixture():
    out, rows, order = {}, {}, {}
    for line in open(os.path.join(GOLDEN, "unmask_scores_handworked.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, val = line.split(":")
        vals = [LN[v] if v in LN else float(v) for v in val.split()]
        if key.startswith("row"):
            rows[int(key.split()[1])] = vals
        elif key.startswith("order"):
            order[key.split()[1]] = [int(v) for v in vals]
        else:
            out[key] = vals
    logits = np.array([rows[i] for i in range(len(rows))], np.float32)[None]
    return logits, out, order


KINDS = {"conf": 0, "neg_entropy": 1, "margin": 2, "noisy": 3}


def test_scores_handworked_fixture(oracle):
    logits, want, order = _parse_scores_fixture()
    masked = np.array(want["masked"], np.uint8)[None]
    tok, conf, zmax, ne, mg = oracle.unmask_scores(logits, masked)
    np.testing.assert_array_equal(tok[0], np.array(want["tok"], np.int32))
    for got, key in ((conf, "conf"), (zmax, "zmax"), (ne, "neg_entropy"), (mg, "margin")):
        np.testing.assert_allclose(got[0], np.array(want[key], np.float32), rtol=3e-7, atol=1e-7, err_msg=key)
    noise = np.array(want["noise"], np.float32)[None]
    m_pos = [i for i in range(masked.shape[1]) if masked[0, i]]
    for name, kind in KINDS.items():
        for k in range(1, len(m_pos) + 2):
            mk, tokens = masked.copy(), np.full(masked.shape, 77, np.int32)
            tok2, conf2, score, zmax2, sel, n = oracle.unmask_select_scored(logits, mk, tokens, k, kind, noise if kind == 3 else None)
            k_eff = min(k, len(m_pos))
            chosen = sorted(order[name][:k_eff])
            assert n[0] == k_eff
            np.testing.assert_array_equal(sel[0, :k_eff], chosen)
            assert np.all(sel[0, k_eff:] == -1)
            exp_mask = masked[0].copy(); exp_mask[chosen] = 0
            np.testing.assert_array_equal(mk[0], exp_mask)
            exp_tok = np.full(masked.shape[1], 77, np.int32); exp_tok[chosen] = tok[0, chosen]
            np.testing.assert_array_equal(tokens[0], exp_tok)
            if kind == 3:
                np.testing.assert_allclose(score[0, m_pos], np.array(want["noisy"], np.float32)[m_pos], rtol=3e-7, atol=1e-7)
    # kind 0 is the plain confidence rule
    mk, tokens = masked.copy(), np.full(masked.shape, 77, np.int32)
    a = oracle.unmask_select_scored(logits, mk, tokens, 2, 0)
    mk2, tokens2 = masked.copy(), np.full(masked.shape, 77, np.int32)
    b = oracle.unmask_select(logits, mk2, tokens2, 2)
    np.testing.assert_array_equal(a[4], b[2]); np.testing.assert_array_equal(mk, mk2); np.testing.assert_array_equal(tokens, tokens2)
    np.testing.assert_array_equal(a[1], b[1])


def test_scores_closed_forms(oracle):
    V = 1024
    z = np.zeros((1, 3, V), np.float32)
    z[0, 0, :] = 1.25                      # uniform: entropy ln V, margin 0
    a = np.float32(2.5)
    z[0, 1, 17] = a                         # one raised logit: p1 = e^a / (e^a + V - 1), the rest equal
    z[0, 2, 5] = z[0, 2, 900] = a           # the maximum twice: margin 0, tok the lower index
    tok, conf, zmax, ne, mg = oracle.unmask_scores(z, np.ones((1, 3), np.uint8))
    assert tok[0].tolist() == [0, 17, 5]
    assert ne[0, 0] == np.float32(-math.log(V)) and mg[0, 0] == 0 and conf[0, 0] == np.float32(2.0 ** -10)
    ea = math.exp(float(a))
    p1, pr = ea / (ea + V - 1), 1.0 / (ea + V - 1)
    np.testing.assert_allclose(conf[0, 1], p1, rtol=2e-7)
    np.testing.assert_allclose(mg[0, 1], p1 - pr, rtol=2e-7)
    np.testing.assert_allclose(ne[0, 1], p1 * math.log(p1) + (V - 1) * pr * math.log(pr), rtol=2e-7)
    assert mg[0, 2] == 0 and zmax[0].tolist() == [1.25, 2.5, 2.5]
    # a single-entry vocabulary: certainty
    tok, conf, zmax, ne, mg = oracle.unmask_scores(np.full((1, 1, 1), -3.0, np.float32), np.ones((1, 1), np.uint8))
    assert (tok[0, 0], conf[0, 0], ne[0, 0], mg[0, 0], zmax[0, 0]) == (0, 1.0, 0.0, 1.0, -3.0)
    # -inf entries contribute nothing
    zi = np.array([[[0.0, -np.inf, math.log(3.0), -np.inf]]], np.float32)
    tok, conf, zmax, ne, mg = oracle.unmask_scores(zi, np.ones((1, 1), np.uint8))
    np.testing.assert_allclose([conf[0, 0], mg[0, 0], ne[0, 0]], [0.75, 0.5, 0.75 * math.log(0.75) + 0.25 * math.log(0.25)], rtol=3e-7)


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_scores_against_library_softmax_and_sort(oracle, seed):
    """torch's float64 softmax / entropy and a plain sort as independent routines; ranking by lexicographic sort."""
    B, L, V, k = 2, 9, 257, 3
    logits = make_logits(B, L, V, (1.0, 6.0), 500 + seed).numpy()
    masked0 = make_mask(B, L, 6, 600 + seed).numpy()
    noise = np.random.default_rng(seed).gumbel(size=(B, L)).astype(np.float32)
    p = torch.softmax(torch.from_numpy(logits).double(), -1)
    ent = torch.distributions.Categorical(probs=p).entropy().numpy()
    ps = np.sort(p.numpy(), -1)[..., ::-1]
    ref = {0: ps[..., 0], 1: -ent, 2: ps[..., 0] - ps[..., 1], 3: np.log(ps[..., 0].astype(np.float32).astype(np.float64)) + noise}
    tok, conf, zmax, ne, mg = oracle.unmask_scores(logits, masked0)
    m = masked0.astype(bool)
    np.testing.assert_allclose(conf[m], ref[0][m], rtol=3e-7)
    np.testing.assert_allclose(ne[m], ref[1][m], rtol=3e-6)
    np.testing.assert_allclose(mg[m], ref[2][m], rtol=3e-6, atol=1e-9)
    np.testing.assert_array_equal(zmax[m], logits.max(-1)[m])
    for kind in range(4):
        mk, tokens = masked0.copy(), np.zeros((B, L), np.int32)
        _, _, score, _, sel, n = oracle.unmask_select_scored(logits, mk, tokens, k, kind, noise if kind == 3 else None)
        for b in range(B):
            pos = [i for i in range(L) if masked0[b, i]]
            ranked = sorted(pos, key=lambda i: (-float(score[b, i]), i))[:k]
            assert n[b] == len(ranked) and sel[b, :len(ranked)].tolist() == sorted(ranked)
            np.testing.assert_allclose(score[b, pos], ref[kind][b, pos], rtol=5e-6, atol=1e-7)


# ------------------------------------------------------------------------ threshold accept
def _parse_threshold_fixture():
    for line in open(os.path.join(GOLDEN, "guided_accept_threshold_handworked.txt")):
        if not line.strip() or line.startswith("#"):
            continue
        f = [x.strip() for x in line.rstrip("\n").split("|")]
        pairs = lambda s, t: np.array([[t(v) for v in pr.split(",")] for pr in s.split()], np.float32 if t is float else np.int32)  # noqa: E731
        yield (float(f[0]), np.array(f[1].split(), np.uint8), np.array(f[2].split(), np.int32), np.array(f[3].split(), np.float32),
               pairs(f[4], int), pairs(f[5], float), np.array(f[6].split(), np.int64), np.array(f[7].split(), np.int32),
               np.array(f[8].split(), np.int32))


def test_threshold_handworked_fixture(oracle):
    n_cases = 0
    for tau, masked0, dlm, zmax, ar_tok, ar_logit, want, w0, w1 in _parse_threshold_fixture():
        n_cases += 1
        for source, written in ((0, w0), (1, w1)):
            masked = masked0[None].copy()
            tokens = np.full(masked.shape, -5, np.int32)
            accept, acc_idx, n_acc = oracle.guided_accept_threshold(dlm[None], zmax[None], ar_tok[None], ar_logit[None], tau,
                                                                    masked, tokens, source)
            assert n_acc[0] == len(want)
            np.testing.assert_array_equal(acc_idx[0, :len(want)], want)
            assert np.all(acc_idx[0, len(want):] == -1)
            exp_tokens = np.full(len(masked0), -5, np.int32); exp_tokens[want] = written
            np.testing.assert_array_equal(tokens[0], exp_tokens)
            exp_accept = np.zeros(len(masked0), np.uint8); exp_accept[want] = 1
            np.testing.assert_array_equal(accept[0], exp_accept)
            exp_mask = masked0.copy(); exp_mask[want] = 0
            np.testing.assert_array_equal(masked[0], exp_mask)
    assert n_cases == 7


def _threshold_bruteforce(dlm, zmax, ar_tok, ar_logit, tau, masked, source):
    """The reading written with sets: deterministic accept (with fallback) united with the threshold passes."""
    pos = [i for i in range(len(masked)) if masked[i]]
    prefix = list(itertools.takewhile(lambda i: dlm[i] in set(ar_tok[i].tolist()), pos))
    fallback = pos[0] if pos and not prefix else None
    passes = {i for i in pos if np.float32(zmax[i]) > np.float32(tau) * np.float32(ar_logit[i].max())}
    acc = sorted(set(prefix) | passes | ({fallback} if fallback is not None else set()))
    toks = {i: (ar_tok[i, 0] if (i == fallback and i not in passes and source == 1) else dlm[i]) for i in acc}
    return acc, toks


@pytest.mark.parametrize("K", [1, 2, 5])
def test_threshold_bruteforce_random(oracle, K):
    rng = np.random.default_rng(40 + K)
    B, L, V = 16, 12, 9
    dlm = rng.integers(0, V, (B, L)).astype(np.int32)
    ar_tok = rng.integers(0, V, (B, L, K)).astype(np.int32)
    ar_tok[rng.random((B, L)) < 0.6, 0] = 0
    ar_tok[..., 0] = np.where(ar_tok[..., 0] == 0, dlm, ar_tok[..., 0])     # a good share of agreement
    zmax = rng.normal(4, 3, (B, L)).astype(np.float32)
    ar_logit = rng.normal(8, 4, (B, L, K)).astype(np.float32)
    masked0 = (rng.random((B, L)) < 0.7).astype(np.uint8)
    masked0[0] = 0
    for tau, source in itertools.product([0.5, 1.0, -0.25], [0, 1]):
        masked, tokens = masked0.copy(), np.full((B, L), -9, np.int32)
        accept, acc_idx, n_acc = oracle.guided_accept_threshold(dlm, zmax, ar_tok, ar_logit, tau, masked, tokens, source)
        for b in range(B):
            acc, toks = _threshold_bruteforce(dlm[b], zmax[b], ar_tok[b], ar_logit[b], tau, masked0[b], source)
            assert n_acc[b] == len(acc) and acc_idx[b, :len(acc)].tolist() == acc
            for i in range(L):
                assert accept[b, i] == (i in acc) and masked[b, i] == (masked0[b, i] and i not in acc)
                assert tokens[b, i] == (toks[i] if i in acc else -9)


def test_threshold_that_nothing_passes_is_the_topk_match_rule(oracle):
    """With a bound no DLM logit can exceed, the rule is the Top-K match accept; with K = 1 it is Algorithm 1."""
    rng = np.random.default_rng(7)
    B, L, K = 8, 16, 2
    dlm = rng.integers(0, 5, (B, L)).astype(np.int32)
    ar_tok = rng.integers(0, 5, (B, L, K)).astype(np.int32)
    zmax = rng.normal(0, 1, (B, L)).astype(np.float32)
    big = np.full((B, L, K), 1e30, np.float32)
    masked0 = (rng.random((B, L)) < 0.8).astype(np.uint8)
    for source in (0, 1):
        m1, t1 = masked0.copy(), np.zeros((B, L), np.int32)
        r1 = oracle.guided_accept_threshold(dlm, zmax, ar_tok, big, 1.0, m1, t1, source)
        m2, t2 = masked0.copy(), np.zeros((B, L), np.int32)
        r2 = oracle.guided_accept_topk(dlm, ar_tok, m2, t2, source)
        for a, b in zip(r1 + (m1, t1), r2 + (m2, t2)):
            np.testing.assert_array_equal(a, b)
        m3, t3 = masked0.copy(), np.zeros((B, L), np.int32)
        r3 = oracle.guided_accept_threshold(dlm, zmax, ar_tok[..., :1].copy(), big[..., :1].copy(), 1.0, m3, t3, source)
        m4, t4 = masked0.copy(), np.zeros((B, L), np.int32)
        r4 = oracle.guided_accept(dlm, ar_tok[..., 0].copy(), m4, t4, source)
        for a, b in zip(r3 + (m3, t3), r4 + (m4, t4)):
            np.testing.assert_array_equal(a, b)
    # and a bound everything exceeds accepts every masked position
    m5, t5 = masked0.copy(), np.zeros((B, L), np.int32)
    _, _, n = oracle.guided_accept_threshold(dlm, zmax, ar_tok, -big, 1.0, m5, t5, 0)
    np.testing.assert_array_equal(n, masked0.sum(1)); assert not m5.any()
