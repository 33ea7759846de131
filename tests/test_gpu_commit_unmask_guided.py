"""GPU parity (bit-exact) of cache commit, confidence/top-k unmasking and guided accept against the
CPU oracle, through the C-ABI."""
import itertools

import numpy as np
import pytest
import torch

import paper_2505_21467_b200 as dlm
from workloads import (bf16_bits, get_config, make_cache, make_kv_rows, make_logits, make_mask, make_tok_ar,
                       seed_for)
from helpers import CONF_RTOL, Dev, gpu_unmask, topk_margin

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev():
    return Dev()


def _i32(a):
    return None if a is None else torch.tensor(np.asarray(a), dtype=torch.int32, device="cuda")


def _run_commit(dev, oracle, ck, cv, cache_len, kn, vn, src_idx=None, dst_pos=None, n_rows=None, n_max=None,
                advance=False, layer_begin=0, layer_end=None, expect_status=0, dst_mode=0):
    """ck.. are CPU bf16 tensors; runs both sides and compares every byte."""
    NL = ck.shape[0]
    layer_end = NL if layer_end is None else layer_end
    src_len = kn.shape[3]
    if n_max is None:
        n_max = (np.asarray(src_idx).shape[1] if src_idx is not None else
                 np.asarray(dst_pos).shape[1] if dst_pos is not None else src_len)
    o_ck, o_cv = bf16_bits(ck).copy(), bf16_bits(cv).copy()
    o_len = np.asarray(cache_len, np.int32).copy()
    rc = oracle.kv_cache_commit(o_ck, o_cv, o_len, bf16_bits(kn), bf16_bits(vn),
                                None if src_idx is None else np.asarray(src_idx, np.int32),
                                None if dst_pos is None else np.asarray(dst_pos, np.int32),
                                None if n_rows is None else np.asarray(n_rows, np.int32), n_max, advance,
                                layer_begin, layer_end, dst_mode)
    g_ck = dev.guarded(tuple(ck.shape), torch.bfloat16, 0).copy_(ck)
    g_cv = dev.guarded(tuple(cv.shape), torch.bfloat16, 0).copy_(cv)
    g_len = dev.guarded((len(cache_len),), torch.int32, 0).copy_(_i32(cache_len))
    cache = dlm.make_kv_cache(g_ck, g_cv, g_len)
    dlm.dlm_kv_cache_commit(dev.ctx, cache, kn.cuda(), vn.cuda(), src_len, _i32(src_idx), _i32(dst_pos), dst_mode,
                            _i32(n_rows), n_max, advance, layer_begin, layer_end)
    st = dev.status()
    np.testing.assert_array_equal(bf16_bits(g_ck), o_ck)
    np.testing.assert_array_equal(bf16_bits(g_cv), o_cv)
    np.testing.assert_array_equal(g_len.cpu().numpy(), o_len)
    want = {0: 0, 1: dlm.DLM_ERR_CAPACITY, 2: dlm.DLM_ERR_INDEX}.get(rc, None)
    if want is not None:
        assert st == want
    else:
        assert st in (dlm.DLM_ERR_CAPACITY, dlm.DLM_ERR_INDEX)
    assert (rc != 0) == (expect_status != 0)


def test_commit_tiny_config_scatter_of_unmasked_rows(dev, oracle):
    cfg = get_config(0)
    s = seed_for(0)
    ck, cv = make_cache(cfg.n_layers, cfg.batch, cfg.n_kv_heads, cfg.capacity, cfg.head_dim, s)
    kn = make_kv_rows((cfg.n_layers, cfg.batch, cfg.n_kv_heads, cfg.block_len, cfg.head_dim), s + 1)
    vn = make_kv_rows((cfg.n_layers, cfg.batch, cfg.n_kv_heads, cfg.block_len, cfg.head_dim), s + 2)
    src = [[3, 9, 17, 30]]
    dst = [[cfg.prompt_len + p for p in src[0]]]
    _run_commit(dev, oracle, ck, cv, [cfg.prompt_len], kn, vn, src, dst, [4])


@pytest.mark.parametrize("D", [64, 128, 24])
def test_commit_ragged_scatter_append_and_layer_range(dev, oracle, D):
    NL, B, Hkv, Lcap, src_len = 5, 3, 2, 301, 70
    ck, cv = make_cache(NL, B, Hkv, Lcap, D, 900 + D)
    kn = make_kv_rows((3, B, Hkv, src_len, D), 901 + D)
    vn = make_kv_rows((3, B, Hkv, src_len, D), 902 + D)
    rng = np.random.default_rng(D)
    n_max = 37
    src = np.stack([rng.permutation(src_len)[:n_max] for _ in range(B)])
    dst = np.stack([rng.permutation(Lcap)[:n_max] for _ in range(B)])
    _run_commit(dev, oracle, ck, cv, [10, 200, 0], kn, vn, src, dst, [37, 0, 5], layer_begin=1, layer_end=4)
    # append with a source gather, advancing the visible length
    _run_commit(dev, oracle, ck, cv, [10, 200, 0], kn, vn, src, None, [37, 20, 1], advance=True, layer_begin=2,
                layer_end=5)
    # window staging: row p of the fresh block lands at cache_len + p; the last slot may overflow
    _run_commit(dev, oracle, ck, cv, [10, 231, 0], kn, vn, src, None, [37, 20, 1], dst_mode=1, layer_begin=0,
                layer_end=3)
    _run_commit(dev, oracle, ck, cv, [10, 240, 0], kn, vn, src, None, [37, 37, 1], dst_mode=1, layer_begin=0,
                layer_end=3, expect_status=1)
    # plain contiguous append of every source row
    _run_commit(dev, oracle, ck, cv, [10, 231, 0], kn, vn, advance=True, layer_begin=0, layer_end=3)


def test_commit_errors_are_reported_and_suppressed(dev, oracle):
    NL, B, Hkv, Lcap, D, src_len = 2, 2, 2, 40, 64, 8
    ck, cv = make_cache(NL, B, Hkv, Lcap, D, 950)
    kn, vn = make_kv_rows((NL, B, Hkv, src_len, D), 951), make_kv_rows((NL, B, Hkv, src_len, D), 952)
    _run_commit(dev, oracle, ck, cv, [36, 3], kn, vn, advance=True, expect_status=1)            # 36 + 8 > 40
    _run_commit(dev, oracle, ck, cv, [0, 0], kn, vn, [[0, 8], [-1, 1]], [[1, 2], [3, 40]], expect_status=1)
    _run_commit(dev, oracle, ck, cv, [0, 0], kn, vn, None, [[1, 2], [3, 4]], [3, 1], expect_status=1)  # n > n_max
    assert dev.status() == 0                                                                  # cleared


def test_commit_argument_errors_launch_nothing(dev):
    ck, cv = make_cache(1, 1, 1, 8, 64, 1, device="cuda")
    cl = _i32([0])
    cache = dlm.make_kv_cache(ck, cv, cl)
    kn = make_kv_rows((1, 1, 1, 4, 64), 2, device="cuda")
    before = dlm.dlm_launch_count(dev.ctx)
    for kwargs, code in ((dict(src_len=0), dlm.DLM_ERR_SHAPE), (dict(n_max=0), dlm.DLM_ERR_SHAPE),
                         (dict(layer_end=2), dlm.DLM_ERR_SHAPE), (dict(layer_begin=1), dlm.DLM_ERR_SHAPE),
                         (dict(dst_mode=2), dlm.DLM_ERR_SHAPE)):
        a = dict(src_len=4, n_max=4, layer_begin=0, layer_end=1, dst_mode=0)
        a.update(kwargs)
        with pytest.raises(dlm.DlmError) as e:
            dlm.dlm_kv_cache_commit(dev.ctx, cache, kn, kn, a["src_len"], None, None, a["dst_mode"], None,
                                    a["n_max"], 0, a["layer_begin"], a["layer_end"])
        assert e.value.code == code
    assert dlm.dlm_launch_count(dev.ctx) == before


def test_commit_dream7b_prompt_refresh_and_block_freeze_full_size(dev, oracle):
    """The benchmark's own commit shapes: refresh of the 1024-row prompt, then staged 4-row commits
    and the block-end advance, all 28 layers in one launch."""
    cfg = get_config(1)
    s = seed_for(1)
    ck, cv = make_cache(cfg.n_layers, cfg.batch, cfg.n_kv_heads, cfg.capacity, cfg.head_dim, s)
    pk = make_kv_rows((cfg.n_layers, cfg.batch, cfg.n_kv_heads, cfg.prompt_len, cfg.head_dim), s + 1)
    pv = make_kv_rows((cfg.n_layers, cfg.batch, cfg.n_kv_heads, cfg.prompt_len, cfg.head_dim), s + 2)
    _run_commit(dev, oracle, ck, cv, [0], pk, pv, advance=True)
    kn = make_kv_rows((cfg.n_layers, cfg.batch, cfg.n_kv_heads, cfg.block_len, cfg.head_dim), s + 3)
    vn = make_kv_rows((cfg.n_layers, cfg.batch, cfg.n_kv_heads, cfg.block_len, cfg.head_dim), s + 4)
    sel = [[2, 11, 12, 31]]
    _run_commit(dev, oracle, ck, cv, [1024], kn, vn, sel, [[1024 + p for p in sel[0]]], [4])
    _run_commit(dev, oracle, ck, cv, [1056], kn, vn, sel, None, [3], dst_mode=1)   # staged in the window
    _run_commit(dev, oracle, ck, cv, [1024], kn, vn, advance=True)            # whole block frozen


# ----------------------------------------------------------------------------- unmasking
def _compare_unmask(dev, oracle, logits, masked0, k, tokens0=None):
    B, Lblk, V = logits.shape
    tokens0 = np.full((B, Lblk), -3, np.int32) if tokens0 is None else tokens0
    o_masked, o_tokens = masked0.copy(), tokens0.copy()
    o_tok, o_conf, o_sel, o_n = oracle.unmask_select(logits.numpy(), o_masked, o_tokens, k)
    g_masked = torch.from_numpy(masked0.copy()).cuda()
    g_tokens = torch.from_numpy(tokens0.copy()).cuda()
    tok, conf, sel_idx, n_sel = gpu_unmask(dev, logits.cuda(), g_masked, g_tokens, k)
    assert dev.status() == 0
    np.testing.assert_array_equal(tok.cpu().numpy(), o_tok)                    # argmax ids: bit-exact
    m = masked0 != 0
    np.testing.assert_allclose(conf.cpu().numpy()[m], o_conf[m], rtol=CONF_RTOL)
    assert np.all(conf.cpu().numpy()[~m] == -1)
    np.testing.assert_array_equal(g_masked.cpu().numpy(), o_masked)
    np.testing.assert_array_equal(g_tokens.cpu().numpy(), o_tokens)
    if k > 0:
        np.testing.assert_array_equal(sel_idx.cpu().numpy(), o_sel)            # committed positions: bit-exact
        np.testing.assert_array_equal(n_sel.cpu().numpy(), o_n)
    return o_conf


def _logits_with_margin(oracle, B, Lblk, V, sigma, masked0, k, seed):
    """Draws logits; re-draws (seed + 1) while the k-th / (k+1)-th oracle confidences are closer than
    1e-4 relative, so that exactly one top-k set is correct."""
    for attempt in range(8):
        logits = make_logits(B, Lblk, V, sigma, seed + attempt)
        if k == 0:
            return logits
        _, conf, _, _ = oracle.unmask_select(logits.numpy(), masked0.copy(), np.zeros((B, Lblk), np.int32), 0)
        if topk_margin(conf, masked0, k) > 1e-4:
            return logits
    raise AssertionError("no seed with a clear top-k margin")


def test_unmask_tiny_config(dev, oracle):
    cfg = get_config(0)
    masked0 = make_mask(cfg.batch, cfg.block_len, 12, seed_for(0)).numpy()
    logits = _logits_with_margin(oracle, cfg.batch, cfg.block_len, cfg.vocab, cfg.logit_sigma, masked0, cfg.top_k,
                                 seed_for(0))
    _compare_unmask(dev, oracle, logits, masked0, cfg.top_k)
    _compare_unmask(dev, oracle, logits, masked0, 0)


@pytest.mark.parametrize("V", [1, 7, 4095, 4096, 4097, 10007, 12290])
def test_unmask_ragged_vocab_and_ties(dev, oracle, V):
    B, Lblk, k = 3, 19, 3
    masked0 = make_mask(B, Lblk, 11, V).numpy()
    logits = make_logits(B, Lblk, V, (0.5, 5.0), 40 + V)
    rows = np.flatnonzero(masked0[0])
    logits[0, rows[1]] = logits[0, rows[0]]          # bit-identical rows: exact confidence tie
    if V > 8:
        logits[1, np.flatnonzero(masked0[1])[0], V // 2:] = -float("inf")
        r2 = np.flatnonzero(masked0[2])[:2]
        logits[2, r2, V - 3] = logits[2].max() + 1.0  # maximum near the ragged tail ...
        logits[2, r2[0], 5] = logits[2, r2[0], V - 3]  # ... and a duplicate of it: lowest index wins
    _, conf, _, _ = oracle.unmask_select(logits.numpy(), masked0.copy(), np.zeros((B, Lblk), np.int32), 0)
    if V > 1 and topk_margin(conf, masked0, k) < 1e-4:
        pytest.skip("near-tie between distinct rows: several top-k sets are acceptable")
    if V == 1:
        k = 30                                        # all confidences equal 1: ties by position, k > n_masked
    _compare_unmask(dev, oracle, logits, masked0, k)


def test_unmask_dream7b_full_vocab_every_mask_count(dev, oracle):
    """The benchmark's shape (vocab 152064, block 32): a whole block emptied 4 positions at a time."""
    cfg = get_config(1)
    masked = np.ones((cfg.batch, cfg.block_len), np.uint8)
    tokens = np.full((cfg.batch, cfg.block_len), -1, np.int32)
    for step in range(cfg.steps_per_block):
        logits = _logits_with_margin(oracle, cfg.batch, cfg.block_len, cfg.vocab, cfg.logit_sigma, masked,
                                     cfg.top_k, seed_for(1, 10 * step))
        before = masked.copy()
        _compare_unmask(dev, oracle, logits, before, cfg.top_k, tokens)
        oracle.unmask_select(logits.numpy(), masked, tokens, cfg.top_k)
    assert masked.sum() == 0


def test_unmask_llada_shape_batch4_block64(dev, oracle):
    cfg = get_config(2)
    masked0 = make_mask(cfg.batch, cfg.block_len, 40, seed_for(2)).numpy()
    logits = _logits_with_margin(oracle, cfg.batch, cfg.block_len, cfg.vocab, cfg.logit_sigma, masked0, cfg.top_k,
                                 seed_for(2))
    _compare_unmask(dev, oracle, logits, masked0, cfg.top_k)


def test_unmask_nothing_masked_and_large_block(dev, oracle):
    logits = make_logits(2, 1024, 33, (1.0, 2.0), 77)
    masked0 = np.zeros((2, 1024), np.uint8)
    _compare_unmask(dev, oracle, logits, masked0, 4)
    masked0 = make_mask(2, 1024, 700, 78).numpy()
    _, conf, _, _ = oracle.unmask_select(logits.numpy(), masked0.copy(), np.zeros((2, 1024), np.int32), 0)
    if topk_margin(conf, masked0, 100) > 1e-4:
        _compare_unmask(dev, oracle, logits, masked0, 100)


def test_unmask_is_deterministic(dev):
    logits = make_logits(2, 32, 152064, (1.0, 8.0), 5).cuda()
    outs = []
    for _ in range(2):
        masked = torch.ones(2, 32, dtype=torch.uint8, device="cuda")
        tokens = torch.zeros(2, 32, dtype=torch.int32, device="cuda")
        tok, conf, sel, n = gpu_unmask(dev, logits, masked, tokens, 4)
        outs.append((tok.clone(), conf.clone(), sel.clone()))
    for a, b in zip(outs[0], outs[1]):
        assert torch.equal(a, b)


# ------------------------------------------------------------------------------- guided
def _compare_guided(dev, oracle, dlm_tok, ar_tok, masked0, source=0):
    B, Lblk = dlm_tok.shape
    o_masked, o_tokens = masked0.copy(), np.full((B, Lblk), -4, np.int32)
    o_acc, o_idx, o_n = oracle.guided_accept(dlm_tok, ar_tok, o_masked, o_tokens, source)
    g_masked = torch.from_numpy(masked0.copy()).cuda()
    g_tokens = torch.full((B, Lblk), -4, dtype=torch.int32, device="cuda")
    accept = dev.guarded((B, Lblk), torch.uint8, 9)
    acc_idx = dev.guarded((B, Lblk), torch.int32, -9)
    n_acc = dev.guarded((B,), torch.int32, -9)
    dlm.dlm_guided_accept(dev.ctx, torch.from_numpy(dlm_tok).cuda(), torch.from_numpy(ar_tok).cuda(), B, Lblk,
                          g_masked, g_tokens, source, accept, acc_idx, n_acc)
    assert dev.status() == 0
    np.testing.assert_array_equal(accept.cpu().numpy(), o_acc)
    np.testing.assert_array_equal(acc_idx.cpu().numpy(), o_idx)
    np.testing.assert_array_equal(n_acc.cpu().numpy(), o_n)
    np.testing.assert_array_equal(g_masked.cpu().numpy(), o_masked)
    np.testing.assert_array_equal(g_tokens.cpu().numpy(), o_tokens)
    return o_n


@pytest.mark.parametrize("source", [0, 1])
def test_guided_exhaustive_patterns(dev, oracle, source):
    m = 9
    Lblk = 2 * m + 1
    pats = np.array(list(itertools.product([0, 1], repeat=m)), np.int32)
    B = len(pats)
    masked0 = np.zeros((B, Lblk), np.uint8)
    pos = np.arange(1, Lblk, 2)
    masked0[:, pos] = 1
    d = np.tile(np.arange(100, 100 + Lblk, dtype=np.int32), (B, 1))
    a = d.copy()
    a[:, ::2] += 7
    a[:, pos] = np.where(pats == 1, d[:, pos], d[:, pos] + 1)
    _compare_guided(dev, oracle, d, a, masked0, source)


@pytest.mark.parametrize("Lblk", [1, 31, 32, 33, 100, 1024])
def test_guided_random_blocks(dev, oracle, Lblk):
    B = 8
    rng = np.random.default_rng(Lblk)
    masked0 = (rng.random((B, Lblk)) < 0.6).astype(np.uint8)
    masked0[0] = 0                      # nothing masked
    masked0[1] = 1                      # everything masked
    d = rng.integers(0, 152064, (B, Lblk)).astype(np.int32)
    a = make_tok_ar(torch.from_numpy(d), 0.9, 152064, Lblk).numpy()
    a[1] = d[1]                         # full agreement
    _compare_guided(dev, oracle, d, a, masked0)


def test_guided_config_statistics(dev, oracle):
    """Config 5's recipe: per-token agreement 0.8 over 32 masked positions accepts about 4.2 per step."""
    cfg = get_config(4)
    B, Lblk = 4096, cfg.block_len
    rng = np.random.default_rng(1)
    d = rng.integers(0, cfg.vocab, (B, Lblk)).astype(np.int32)
    a = make_tok_ar(torch.from_numpy(d), cfg.p_agree, cfg.vocab, 2).numpy()
    n = _compare_guided(dev, oracle, d, a, np.ones((B, Lblk), np.uint8))
    assert abs(n.mean() - (0.2 + 4 * (1 - 0.8 ** 32))) < 0.25


@pytest.mark.parametrize("K", [1, 2, 5])
def test_guided_topk_match_variant(dev, oracle, K):
    """Top-K match: bit-exact against the oracle on random blocks with a small vocabulary (agreements at every
    rank are common), both fallback sources, block lengths on both sides of a warp."""
    rng = np.random.default_rng(40 + K)
    for Lblk in (7, 32, 70):
        B, V = 64, 6
        d = rng.integers(0, V, (B, Lblk)).astype(np.int32)
        a = np.stack([rng.permutation(V)[:K] for _ in range(B * Lblk)]).reshape(B, Lblk, K).astype(np.int32)
        masked0 = (rng.random((B, Lblk)) < 0.6).astype(np.uint8)
        for source in (0, 1):
            o_m, o_t = masked0.copy(), np.full((B, Lblk), -1, np.int32)
            o_acc, o_idx, o_n = oracle.guided_accept_topk(d, a, o_m, o_t, source)
            g_m = torch.from_numpy(masked0.copy()).cuda()
            g_t = torch.full((B, Lblk), -1, dtype=torch.int32, device="cuda")
            accept = torch.empty(B, Lblk, dtype=torch.uint8, device="cuda")
            acc_idx = torch.empty(B, Lblk, dtype=torch.int32, device="cuda")
            n_acc = torch.empty(B, dtype=torch.int32, device="cuda")
            dlm.dlm_guided_accept_topk(dev.ctx, torch.from_numpy(d).cuda(), torch.from_numpy(a).cuda(), K, B, Lblk, g_m, g_t,
                                       source, accept, acc_idx, n_acc)
            np.testing.assert_array_equal(accept.cpu().numpy(), o_acc)
            np.testing.assert_array_equal(acc_idx.cpu().numpy(), o_idx)
            np.testing.assert_array_equal(n_acc.cpu().numpy(), o_n)
            np.testing.assert_array_equal(g_m.cpu().numpy(), o_m)
            np.testing.assert_array_equal(g_t.cpu().numpy(), o_t)
    assert dev.status() == 0
