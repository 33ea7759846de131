"""GPU parity of dlm_unmask_select_scored and dlm_guided_accept_threshold against the oracle, through the C-ABI:
token ids, selected positions, masks and accepted sets bit-exact; scores within the tolerance of fp32 sums."""
import itertools
import os

import numpy as np
import pytest
import torch

import paper_2505_21467_b200 as dlm
from helpers import Dev
from workloads import get_config, make_logits, make_mask, seed_for

pytestmark = pytest.mark.gpu

SCORE_RTOL = 3e-5   # fp32 sums of up to 152064 terms in another order than the oracle's fp64 ones; entropy loses a
SCORE_ATOL = 3e-6   # little more where t/s and ln s nearly cancel (near-uniform rows), hence the absolute term


@pytest.fixture(scope="module")
def dev():
    return Dev()


def _gpu_scored(dev, logits, masked, tokens, k, kind, noise):
    B, L, V = logits.shape
    tok = torch.full((B, L), -9, dtype=torch.int32, device="cuda")
    conf, score, zmax = (torch.full((B, L), float("nan"), device="cuda") for _ in range(3))
    sel = torch.full((B, max(k, 1)), -9, dtype=torch.int32, device="cuda") if k > 0 else None
    n = torch.full((B,), -9, dtype=torch.int32, device="cuda") if k > 0 else None
    ws = dev.workspace(dlm.dlm_unmask_scored_workspace_bytes(dev.ctx, B, L, V))
    dlm.dlm_unmask_select_scored(dev.ctx, logits, B, L, V, masked, tokens, k, kind, noise, tok, conf, score, zmax, sel, n, ws)
    return tok, conf, score, zmax, sel, n


def _score_gap(score, masked0, k):
    """Smallest gap between the k_eff-th and (k_eff+1)-th largest oracle scores, ignoring exact ties."""
    worst = np.inf
    for b in range(score.shape[0]):
        s = np.sort(score[b][masked0[b] != 0].astype(np.float64))[::-1]
        if k < len(s) and s[k - 1] != s[k]:
            worst = min(worst, (s[k - 1] - s[k]) / max(abs(s[k - 1]), abs(s[k]), 1e-30))
    return worst


def _compare_scored(dev, oracle, logits, masked0, k, kind, noise=None, tokens0=None):
    B, L, V = logits.shape
    o_masked = masked0.copy()
    o_tokens = np.full((B, L), -3, np.int32) if tokens0 is None else tokens0.copy()
    o = oracle.unmask_select_scored(logits.numpy(), o_masked, o_tokens, k, kind, None if noise is None else noise.numpy())
    if k > 0 and _score_gap(o[2], masked0, k) < 1e-3:
        return False                                  # several top-k sets are acceptable: not a parity input
    g_masked = torch.from_numpy(masked0.copy()).cuda()
    g_tokens = torch.from_numpy(np.full((B, L), -3, np.int32) if tokens0 is None else tokens0.copy()).cuda()
    tok, conf, score, zmax, sel, n = _gpu_scored(dev, logits.cuda(), g_masked, g_tokens, k, kind, None if noise is None else noise.cuda())
    torch.cuda.synchronize()
    assert dev.status() == 0
    m = masked0.astype(bool)
    np.testing.assert_array_equal(tok.cpu().numpy(), o[0])                       # argmax ids: bit-exact
    np.testing.assert_allclose(conf.cpu().numpy()[m], o[1][m], rtol=SCORE_RTOL)
    np.testing.assert_allclose(score.cpu().numpy()[m], o[2][m], rtol=SCORE_RTOL, atol=SCORE_ATOL)
    np.testing.assert_array_equal(zmax.cpu().numpy(), o[3])                      # a maximum of inputs: exact
    assert np.all(score.cpu().numpy()[~m] == 0) and np.all(conf.cpu().numpy()[~m] == -1)
    np.testing.assert_array_equal(g_masked.cpu().numpy(), o_masked)
    np.testing.assert_array_equal(g_tokens.cpu().numpy(), o_tokens)
    if k > 0:
        np.testing.assert_array_equal(sel.cpu().numpy(), o[4])                   # committed positions: bit-exact
        np.testing.assert_array_equal(n.cpu().numpy(), o[5])
    return True


@pytest.mark.parametrize("kind", [0, 1, 2, 3])
def test_scored_unmask_small_and_ragged_vocabularies(dev, oracle, kind):
    checked = 0
    for V, seed in ((1, 1), (7, 2), (1023, 3), (4096, 4), (4097, 5), (16385, 6), (40000, 7)):
        B, L, k = 3, 21, 4
        masked0 = make_mask(B, L, 13, 100 + V).numpy()
        logits = make_logits(B, L, V, (0.5, 6.0), 200 + seed)
        rows = np.flatnonzero(masked0[0])
        logits[0, rows[1]] = logits[0, rows[0]]                 # bit-identical rows: an exact tie, lowest position wins
        if V > 8:
            logits[1, np.flatnonzero(masked0[1])[0], V // 3:] = -float("inf")
            r = np.flatnonzero(masked0[2])[0]
            logits[2, r, V - 2] = logits[2, r, 3] = logits[2].max() + 2.0    # the maximum twice: margin 0, lowest index
        noise = torch.from_numpy(np.random.default_rng(seed).gumbel(size=(B, L)).astype(np.float32)) if kind == 3 else None
        checked += _compare_scored(dev, oracle, logits, masked0, k, kind, noise)
        checked += _compare_scored(dev, oracle, logits, masked0, 0, kind, noise)
    assert checked >= 10


@pytest.mark.parametrize("kind", [0, 1, 2, 3])
def test_scored_unmask_dream7b_vocab_every_mask_count(dev, oracle, kind):
    """The Dream vocabulary (152064) and block (32), emptied 4 positions at a time by each score."""
    cfg = get_config(1)
    masked = np.ones((cfg.batch, cfg.block_len), np.uint8)
    tokens = np.full((cfg.batch, cfg.block_len), -1, np.int32)
    rng = np.random.default_rng(9)
    done = 0
    for step in range(cfg.steps_per_block):
        for attempt in range(6):
            logits = make_logits(cfg.batch, cfg.block_len, cfg.vocab, cfg.logit_sigma, seed_for(1, 300 + 10 * step + attempt))
            noise = torch.from_numpy(rng.gumbel(size=masked.shape).astype(np.float32)) if kind == 3 else None
            if _compare_scored(dev, oracle, logits, masked.copy(), cfg.top_k, kind, noise, tokens):
                done += 1
                break
        oracle.unmask_select_scored(logits.numpy(), masked, tokens, cfg.top_k, kind, None if noise is None else noise.numpy())
    assert masked.sum() == 0 and done == cfg.steps_per_block


def test_scored_unmask_kind_confidence_equals_the_plain_call(dev):
    from helpers import gpu_unmask
    B, L, V, k = 2, 32, 50000, 4
    logits = make_logits(B, L, V, (1.0, 8.0), 55, device="cuda")
    m1, t1 = torch.ones(B, L, dtype=torch.uint8, device="cuda"), torch.zeros(B, L, dtype=torch.int32, device="cuda")
    m2, t2 = m1.clone(), t1.clone()
    a = gpu_unmask(dev, logits, m1, t1, k)
    b = _gpu_scored(dev, logits, m2, t2, k, 0, None)
    assert torch.equal(a[0], b[0]) and torch.equal(a[2], b[4]) and torch.equal(a[3], b[5]) and torch.equal(m1, m2) and torch.equal(t1, t2)
    torch.testing.assert_close(a[1], b[1], rtol=1e-5, atol=0)


def test_scored_unmask_argument_errors(dev):
    z = torch.zeros(8, device="cuda"); m = torch.ones(2, dtype=torch.uint8, device="cuda"); i = torch.zeros(2, dtype=torch.int32, device="cuda")
    ws = dev.workspace(1024)
    for kind, noise, code in ((4, None, dlm.DLM_ERR_SHAPE), (-1, None, dlm.DLM_ERR_SHAPE), (3, None, dlm.DLM_ERR_NULL)):
        with pytest.raises(dlm.DlmError) as e:
            dlm.dlm_unmask_select_scored(dev.ctx, z, 1, 2, 4, m, i, 1, kind, noise, i, z, z, z, i, i, ws)
        assert e.value.code == code
    assert dev.status() == 0


# ---------------------------------------------------------------------------------- threshold accept
def _compare_threshold(dev, oracle, dlm_tok, zmax, ar_tok, ar_logit, tau, masked0, source):
    B, L = dlm_tok.shape
    K = ar_tok.shape[2]
    o_masked, o_tokens = masked0.copy(), np.full((B, L), -4, np.int32)
    o_acc, o_idx, o_n = oracle.guided_accept_threshold(dlm_tok, zmax, ar_tok, ar_logit, tau, o_masked, o_tokens, source)
    g_masked = torch.from_numpy(masked0.copy()).cuda()
    g_tokens = torch.full((B, L), -4, dtype=torch.int32, device="cuda")
    accept = torch.full((B, L), 9, dtype=torch.uint8, device="cuda")
    acc_idx = torch.full((B, L), -9, dtype=torch.int32, device="cuda")
    n_acc = torch.full((B,), -9, dtype=torch.int32, device="cuda")
    dlm.dlm_guided_accept_threshold(dev.ctx, torch.from_numpy(dlm_tok).cuda(), torch.from_numpy(zmax).cuda(),
                                    torch.from_numpy(ar_tok).cuda(), torch.from_numpy(ar_logit).cuda(), K, tau, B, L, g_masked,
                                    g_tokens, source, accept, acc_idx, n_acc)
    torch.cuda.synchronize()
    assert dev.status() == 0
    np.testing.assert_array_equal(accept.cpu().numpy(), o_acc)
    np.testing.assert_array_equal(acc_idx.cpu().numpy(), o_idx)
    np.testing.assert_array_equal(n_acc.cpu().numpy(), o_n)
    np.testing.assert_array_equal(g_masked.cpu().numpy(), o_masked)
    np.testing.assert_array_equal(g_tokens.cpu().numpy(), o_tokens)
    return o_n


def test_threshold_handworked_fixture_on_gpu(dev, oracle):
    from test_oracle_scores_threshold import _parse_threshold_fixture
    for tau, masked0, d, zmax, ar_tok, ar_logit, want, w0, w1 in _parse_threshold_fixture():
        for source in (0, 1):
            n = _compare_threshold(dev, oracle, d[None].copy(), zmax[None].copy(), ar_tok[None].copy(), ar_logit[None].copy(), tau,
                                   masked0[None].copy(), source)
            assert n[0] == len(want)


@pytest.mark.parametrize("K,L", [(1, 1), (1, 32), (2, 32), (2, 33), (5, 64), (2, 1024), (64, 40)])
def test_threshold_random_blocks(dev, oracle, K, L):
    rng = np.random.default_rng(1000 * K + L)
    B, V = 24, 11
    d = rng.integers(0, V, (B, L)).astype(np.int32)
    ar_tok = rng.integers(0, V, (B, L, K)).astype(np.int32)
    agree = rng.random((B, L)) < 0.75
    ar_tok[..., K - 1] = np.where(agree, d, ar_tok[..., K - 1])
    zmax = rng.normal(5, 3, (B, L)).astype(np.float32)
    ar_logit = rng.normal(9, 4, (B, L, K)).astype(np.float32)
    masked0 = (rng.random((B, L)) < 0.7).astype(np.uint8)
    masked0[0] = 0
    masked0[1] = 1
    for tau, source in itertools.product([0.5, 1.5, -1.0], [0, 1]):
        _compare_threshold(dev, oracle, d, zmax, ar_tok, ar_logit, tau, masked0, source)


def test_threshold_guided_config_shape_with_the_scored_pass(dev, oracle):
    """Guided config's shape (batch 8, block 32, vocab 152064): zmax from the scored pass feeds the accept rule;
    the guider's Top-2 logits are drawn so that a share of the positions passes tau = 0.5."""
    cfg = get_config(4)
    B, L, V, K = cfg.batch, cfg.block_len, cfg.vocab, 2
    logits = make_logits(B, L, V, cfg.logit_sigma, seed_for(4, 77))
    masked0 = np.ones((B, L), np.uint8)
    tok, conf, score, zmax, _, _ = _gpu_scored(dev, logits.cuda(), torch.from_numpy(masked0).cuda(),
                                               torch.zeros(B, L, dtype=torch.int32, device="cuda"), 0, 0, None)
    o = oracle.unmask_select_scored(logits.numpy(), masked0.copy(), np.zeros((B, L), np.int32), 0, 0)
    np.testing.assert_array_equal(tok.cpu().numpy(), o[0])
    np.testing.assert_array_equal(zmax.cpu().numpy(), o[3])
    rng = np.random.default_rng(5)
    d = o[0]
    ar_tok = np.stack([np.where(rng.random((B, L)) < 0.8, d, (d + 1) % V), (d + 7) % V], -1).astype(np.int32)
    ar_logit = (o[3][..., None] * rng.uniform(1.2, 3.0, (B, L, K))).astype(np.float32)
    n = _compare_threshold(dev, oracle, d, o[3], ar_tok, ar_logit, 0.5, masked0, 0)
    assert n.min() >= 1
