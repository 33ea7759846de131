"""Parity at the full shapes of the five configs, in the launch form the benchmark uses (all layers in one call).

What the oracle can do in seconds is checked element by element: attention on sampled (block, step, layer)
triples - steps {first, last} of blocks {first, last}, layers {0, NL/2, NL-1}, all heads and rows -, every integer
output of every step of the generation schedules, and the cache bytes of sampled layers; the layers the oracle does
not visit are checked on the device through properties that hold at any size (committed rows equal their sources,
every other row is unchanged)."""
import numpy as np
import pytest
import torch

import paper_2505_21467_b200 as dlm
from helpers import ATTN_MAX_ERR, ATTN_MEAN_ERR, CONF_RTOL, Dev, topk_margin
from workloads import (bf16_bits, get_config, make_attn_inputs, make_cache, make_kv_rows, make_logits, make_tok_ar,
                       seed_for, widen)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev():
    return Dev()


def _attn_all_layers(dev, cfg, cache, q, kn, vn, q_len, hint):
    out = torch.full_like(q, float("nan"))
    ws = dev.workspace(dlm.dlm_attn_workspace_bytes(dev.ctx, cache, cfg.n_layers, cfg.n_q_heads, cfg.block_len))
    dlm.dlm_freecache_attn_step(dev.ctx, cache, 0, cfg.n_layers, q, kn, vn, cfg.n_q_heads, cfg.block_len, q_len, 0.0, hint,
                                out, None, ws)
    return out


def _check_attn_layers(oracle, ck, cv, cache_len, q, kn, vn, q_len, out, layers):
    """ck, cv: device tensors [NL, ...]; the sampled layers are copied back and run through the oracle."""
    cl = cache_len.cpu().numpy().astype(np.int32)
    ql = None if q_len is None else q_len.cpu().numpy().astype(np.int32)
    for layer in layers:
        ref, _ = oracle.attn_step(widen(ck[layer]), widen(cv[layer]), cl, widen(q[layer]), widen(kn[layer]), widen(vn[layer]), ql)
        got = out[layer].float().cpu().numpy()
        assert np.isfinite(got).all()
        err = np.abs(got - ref)
        assert err.max() <= ATTN_MAX_ERR and err.mean() <= ATTN_MEAN_ERR, (layer, float(err.max()), float(err.mean()))


def _rows_equal(cache_t, new_t, b, dst, src):
    """cache[:, b, :, dst, :] == new[:, b, :, src, :] for index lists dst, src, on the device."""
    d = torch.as_tensor(dst, device="cuda", dtype=torch.long)
    s = torch.as_tensor(src, device="cuda", dtype=torch.long)
    return torch.equal(cache_t[:, b].index_select(2, d), new_t[:, b].index_select(2, s))


# ----------------------------------------------------------------------------------------------- config 3
def test_llada8b_attention_first_and_last_steps_of_first_and_last_blocks(dev, oracle):
    """Config 3 at full size (32 layers, batch 4, 32 heads, capacity 2560): the visible length is 2048 throughout the
    first block and 2496 throughout the last; the first and the last step of each have their own fresh rows."""
    cfg = get_config(2)
    ck, cv = make_cache(cfg.n_layers, cfg.batch, cfg.n_kv_heads, cfg.capacity, cfg.head_dim, seed_for(2, 1), device="cuda")
    layers = [0, cfg.n_layers // 2, cfg.n_layers - 1]
    for block, step in ((0, 0), (0, cfg.steps_per_block - 1), (cfg.n_blocks - 1, 0), (cfg.n_blocks - 1, cfg.steps_per_block - 1)):
        Lc = cfg.prompt_len + block * cfg.block_len
        cache_len = torch.full((cfg.batch,), Lc, dtype=torch.int32, device="cuda")
        cache = dlm.make_kv_cache(ck, cv, cache_len)
        q, kn, vn = make_attn_inputs(cfg.n_layers, cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.block_len, cfg.head_dim,
                                     seed_for(2, 100 * block + step), device="cuda")
        out = _attn_all_layers(dev, cfg, cache, q, kn, vn, None, Lc)
        assert dev.status() == 0
        _check_attn_layers(oracle, ck, cv, cache_len, q, kn, vn, None, out, layers if step == 0 else layers[1:2])


def test_llada8b_per_step_commit_and_block_freeze(dev, oracle):
    """Config 3's commits at full size: the 4 rows unmasked in a step staged behind the visible rows, then the
    whole 64-row block frozen.  Layers {0, 16, 31} byte for byte against the oracle; every layer on the device."""
    cfg = get_config(2)
    NL, B, H, D, L = cfg.n_layers, cfg.batch, cfg.n_kv_heads, cfg.head_dim, cfg.block_len
    ck, cv = make_cache(NL, B, H, cfg.capacity, D, seed_for(2, 2), device="cuda")
    ck0, cv0 = ck.clone(), cv.clone()
    kn = make_kv_rows((NL, B, H, L, D), seed_for(2, 3), device="cuda")
    vn = make_kv_rows((NL, B, H, L, D), seed_for(2, 4), device="cuda")
    Lc = cfg.prompt_len + 3 * L
    cache_len = torch.full((B,), Lc, dtype=torch.int32, device="cuda")
    cache = dlm.make_kv_cache(ck, cv, cache_len)
    rng = np.random.default_rng(3)
    sel = np.stack([np.sort(rng.choice(L, 4, replace=False)) for _ in range(B)]).astype(np.int32)
    n_sel = np.array([4, 3, 4, 0], np.int32)
    layers = [0, NL // 2, NL - 1]
    o_ck, o_cv = bf16_bits(ck[layers]).copy(), bf16_bits(cv[layers]).copy()
    o_len = np.full((B,), Lc, np.int32)
    # staged commit of the selected rows (window placement, lengths unchanged)
    dlm.dlm_kv_cache_commit(dev.ctx, cache, kn, vn, L, torch.from_numpy(sel).cuda(), None, dlm.DLM_DST_WINDOW,
                            torch.from_numpy(n_sel).cuda(), 4, 0, 0, NL)
    oracle.kv_cache_commit(o_ck, o_cv, o_len, bf16_bits(kn[layers]), bf16_bits(vn[layers]), sel, None, n_sel, 4, False, dst_mode=1)
    assert dev.status() == 0
    np.testing.assert_array_equal(bf16_bits(ck[layers]), o_ck)
    np.testing.assert_array_equal(bf16_bits(cv[layers]), o_cv)
    touched = torch.zeros(B, cfg.capacity, dtype=torch.bool, device="cuda")
    for b in range(B):
        src = sel[b, :n_sel[b]].tolist()
        if src:
            assert _rows_equal(ck, kn, b, [Lc + p for p in src], src) and _rows_equal(cv, vn, b, [Lc + p for p in src], src)
            touched[b, [Lc + p for p in src]] = True
    for now, before in ((ck, ck0), (cv, cv0)):      # rows that changed anywhere are exactly the staged ones
        changed = (now != before).any(dim=4).any(dim=2).any(dim=0)
        assert not bool((changed & ~touched).any())
    assert torch.equal(cache_len, torch.full_like(cache_len, Lc))
    # block complete: all 64 rows appended and made visible
    dlm.dlm_kv_cache_commit(dev.ctx, cache, kn, vn, L, None, None, dlm.DLM_DST_APPEND, None, L, 1, 0, NL)
    oracle.kv_cache_commit(o_ck, o_cv, o_len, bf16_bits(kn[layers]), bf16_bits(vn[layers]), None, None, None, L, True)
    assert dev.status() == 0
    np.testing.assert_array_equal(bf16_bits(ck[layers]), o_ck)
    np.testing.assert_array_equal(bf16_bits(cv[layers]), o_cv)
    np.testing.assert_array_equal(cache_len.cpu().numpy(), o_len)
    assert torch.equal(ck[:, :, :, Lc:Lc + L], kn) and torch.equal(cv[:, :, :, Lc:Lc + L], vn)
    assert torch.equal(ck[:, :, :, :Lc], ck0[:, :, :, :Lc]) and torch.equal(ck[:, :, :, Lc + L:], ck0[:, :, :, Lc + L:])
    assert torch.equal(cv[:, :, :, :Lc], cv0[:, :, :, :Lc]) and torch.equal(cv[:, :, :, Lc + L:], cv0[:, :, :, Lc + L:])


# ----------------------------------------------------------------------------------------------- config 4
def test_longctx_prompt_refresh_and_four_row_stage(dev, oracle):
    """Config 4's commits at full size: the refresh that writes all 16384 prompt rows of all 28 layers (940 MB moved
    each way), then a 4-row stage behind them.  Layers {0, 14, 27} byte for byte against the oracle."""
    cfg = get_config(3)
    NL, B, H, D, P = cfg.n_layers, cfg.batch, cfg.n_kv_heads, cfg.head_dim, cfg.prompt_len
    ck, cv = make_cache(NL, B, H, cfg.capacity, D, seed_for(3, 1), device="cuda")
    ck0, cv0 = ck.clone(), cv.clone()
    pk = make_kv_rows((NL, B, H, P, D), seed_for(3, 2), device="cuda")
    pv = make_kv_rows((NL, B, H, P, D), seed_for(3, 3), device="cuda")
    cache_len = torch.zeros(B, dtype=torch.int32, device="cuda")
    cache = dlm.make_kv_cache(ck, cv, cache_len)
    layers = [0, NL // 2, NL - 1]
    o_ck, o_cv, o_len = bf16_bits(ck[layers]).copy(), bf16_bits(cv[layers]).copy(), np.zeros((B,), np.int32)
    dlm.dlm_kv_cache_commit(dev.ctx, cache, pk, pv, P, None, None, dlm.DLM_DST_APPEND, None, P, 1, 0, NL)
    oracle.kv_cache_commit(o_ck, o_cv, o_len, bf16_bits(pk[layers]), bf16_bits(pv[layers]), None, None, None, P, True)
    assert dev.status() == 0
    np.testing.assert_array_equal(bf16_bits(ck[layers]), o_ck)
    np.testing.assert_array_equal(bf16_bits(cv[layers]), o_cv)
    np.testing.assert_array_equal(cache_len.cpu().numpy(), o_len)
    assert torch.equal(ck[:, :, :, :P], pk) and torch.equal(cv[:, :, :, :P], pv)
    assert torch.equal(ck[:, :, :, P:], ck0[:, :, :, P:]) and torch.equal(cv[:, :, :, P:], cv0[:, :, :, P:])
    # the 4 rows unmasked in a step, staged at their own slots behind the 16384 visible rows
    kn = make_kv_rows((NL, B, H, cfg.block_len, D), seed_for(3, 4), device="cuda")
    vn = make_kv_rows((NL, B, H, cfg.block_len, D), seed_for(3, 5), device="cuda")
    sel, n_sel = np.array([[1, 7, 20, 31]], np.int32), np.array([4], np.int32)
    dlm.dlm_kv_cache_commit(dev.ctx, cache, kn, vn, cfg.block_len, torch.from_numpy(sel).cuda(), None, dlm.DLM_DST_WINDOW,
                            torch.from_numpy(n_sel).cuda(), 4, 0, 0, NL)
    oracle.kv_cache_commit(o_ck, o_cv, o_len, bf16_bits(kn[layers]), bf16_bits(vn[layers]), sel, None, n_sel, 4, False, dst_mode=1)
    assert dev.status() == 0
    np.testing.assert_array_equal(bf16_bits(ck[layers]), o_ck)
    np.testing.assert_array_equal(bf16_bits(cv[layers]), o_cv)
    assert _rows_equal(ck, kn, 0, (P + sel[0]).tolist(), sel[0].tolist()) and _rows_equal(cv, vn, 0, (P + sel[0]).tolist(), sel[0].tolist())
    assert torch.equal(ck[:, :, :, :P], pk) and int(cache_len[0]) == P


# ----------------------------------------------------------------------------------------------- config 2
def test_dream7b_whole_generation_schedule_integer_outputs_of_every_step(dev, oracle):
    """Config 2: all 64 steps (8 blocks x 8 steps) at vocabulary 152064 with the state kept on the device: token ids,
    selected positions, counts, masks, tokens and lengths of every step equal the oracle's; the cache bytes of all 28
    layers at the end; attention on layers {0, 14, 27} at the first and last step of the first and last block."""
    cfg = get_config(1)
    NL, B, H, D, L, V, k = cfg.n_layers, cfg.batch, cfg.n_kv_heads, cfg.head_dim, cfg.block_len, cfg.vocab, cfg.top_k
    ck, cv = make_cache(NL, B, H, cfg.capacity, D, seed_for(1, 500), device="cuda")
    o_ck, o_cv = bf16_bits(ck).copy(), bf16_bits(cv).copy()
    cache_len = torch.full((B,), cfg.prompt_len, dtype=torch.int32, device="cuda")
    o_len = np.full((B,), cfg.prompt_len, np.int32)
    cache = dlm.make_kv_cache(ck, cv, cache_len)
    uws = dev.workspace(dlm.dlm_unmask_workspace_bytes(dev.ctx, B, L, V))
    tok = torch.empty(B, L, dtype=torch.int32, device="cuda")
    conf = torch.empty(B, L, device="cuda")
    sel = torch.empty(B, k, dtype=torch.int32, device="cuda")
    n_sel = torch.empty(B, dtype=torch.int32, device="cuda")
    seed = seed_for(1, 1000)
    for block in range(cfg.n_blocks):
        g_masked = torch.ones(B, L, dtype=torch.uint8, device="cuda")
        g_tokens = torch.full((B, L), -1, dtype=torch.int32, device="cuda")
        o_masked, o_tokens = np.ones((B, L), np.uint8), np.full((B, L), -1, np.int32)
        for step in range(cfg.steps_per_block):
            seed += 1
            q, kn, vn = make_attn_inputs(NL, B, cfg.n_q_heads, H, L, D, seed, device="cuda")
            out = _attn_all_layers(dev, cfg, cache, q, kn, vn, None, int(o_len[0]))
            if block in (0, cfg.n_blocks - 1) and step in (0, cfg.steps_per_block - 1):
                _check_attn_layers(oracle, ck, cv, cache_len, q, kn, vn, None, out, [0, NL // 2, NL - 1])
            while True:   # logits whose k-th and (k+1)-th confidences are not a near-tie
                seed += 1
                logits = make_logits(B, L, V, cfg.logit_sigma, seed, device="cuda")
                m2, t2 = o_masked.copy(), o_tokens.copy()
                o_tok, o_conf, o_sel, o_n = oracle.unmask_select(logits.cpu().numpy(), m2, t2, k)
                if topk_margin(o_conf, o_masked, k) > 1e-4:
                    break
            on = o_masked.astype(bool)
            o_masked, o_tokens = m2, t2
            dlm.dlm_unmask_select(dev.ctx, logits, B, L, V, g_masked, g_tokens, k, tok, conf, sel, n_sel, uws)
            if step == cfg.steps_per_block - 1:
                dlm.dlm_kv_cache_commit(dev.ctx, cache, kn, vn, L, None, None, dlm.DLM_DST_APPEND, None, L, 1, 0, NL)
                oracle.kv_cache_commit(o_ck, o_cv, o_len, bf16_bits(kn), bf16_bits(vn), None, None, None, L, True)
            else:
                dlm.dlm_kv_cache_commit(dev.ctx, cache, kn, vn, L, sel, None, dlm.DLM_DST_WINDOW, n_sel, k, 0, 0, NL)
                oracle.kv_cache_commit(o_ck, o_cv, o_len, bf16_bits(kn), bf16_bits(vn), o_sel, None, o_n, k, False, dst_mode=1)
            np.testing.assert_array_equal(tok.cpu().numpy(), o_tok)
            np.testing.assert_allclose(conf.cpu().numpy()[on], o_conf[on], rtol=CONF_RTOL)
            np.testing.assert_array_equal(sel.cpu().numpy(), o_sel)
            np.testing.assert_array_equal(n_sel.cpu().numpy(), o_n)
            np.testing.assert_array_equal(g_masked.cpu().numpy(), o_masked)
            np.testing.assert_array_equal(g_tokens.cpu().numpy(), o_tokens)
            np.testing.assert_array_equal(cache_len.cpu().numpy(), o_len)
        assert not o_masked.any()
    assert dev.status() == 0 and int(o_len[0]) == cfg.capacity
    np.testing.assert_array_equal(bf16_bits(ck), o_ck)
    np.testing.assert_array_equal(bf16_bits(cv), o_cv)


# ----------------------------------------------------------------------------------------------- config 5
def test_guided_propose_over_the_full_block_and_vocabulary(dev, oracle):
    """Config 5's vocabulary pass: 8 x 32 rows of 152064 logits, propose only: token ids bit-exact, confidences 2e-5."""
    cfg = get_config(4)
    B, L, V = cfg.batch, cfg.block_len, cfg.vocab
    logits = make_logits(B, L, V, cfg.logit_sigma, seed_for(4, 9), device="cuda")
    masked = torch.ones(B, L, dtype=torch.uint8, device="cuda")
    tokens = torch.full((B, L), -1, dtype=torch.int32, device="cuda")
    tok = torch.empty(B, L, dtype=torch.int32, device="cuda")
    conf = torch.empty(B, L, device="cuda")
    dlm.dlm_unmask_select(dev.ctx, logits, B, L, V, masked, tokens, 0, tok, conf, None, None,
                          dev.workspace(dlm.dlm_unmask_workspace_bytes(dev.ctx, B, L, V)))
    o_tok, o_conf, _, _ = oracle.unmask_select(logits.cpu().numpy(), np.ones((B, L), np.uint8), np.zeros((B, L), np.int32), 0)
    assert dev.status() == 0
    np.testing.assert_array_equal(tok.cpu().numpy(), o_tok)
    np.testing.assert_allclose(conf.cpu().numpy(), o_conf, rtol=CONF_RTOL)
    assert bool(masked.all()) and bool((tokens == -1).all())


def test_guided_whole_generation_until_every_sequence_finishes(dev, oracle):
    """Config 5 at full size (batch 8, 28 layers, vocabulary 152064): propose, accept the agreeing prefix, append the
    accepted rows, block after block until all 8 sequences have their 256 tokens; a sequence that finishes its block
    early idles (q_len 0) until the slowest one is done.  Every integer output of every step equals the oracle's,
    the cache bytes of all layers at the end, attention on sampled steps and layers."""
    cfg = get_config(4)
    NL, B, H, D, L, V = cfg.n_layers, cfg.batch, cfg.n_kv_heads, cfg.head_dim, cfg.block_len, cfg.vocab
    ck, cv = make_cache(NL, B, H, cfg.capacity, D, seed_for(4, 500), device="cuda")
    o_ck, o_cv = bf16_bits(ck).copy(), bf16_bits(cv).copy()
    cache_len = torch.full((B,), cfg.prompt_len, dtype=torch.int32, device="cuda")
    o_len = np.full((B,), cfg.prompt_len, np.int32)
    cache = dlm.make_kv_cache(ck, cv, cache_len)
    uws = dev.workspace(dlm.dlm_unmask_workspace_bytes(dev.ctx, B, L, V))
    tok = torch.empty(B, L, dtype=torch.int32, device="cuda")
    conf = torch.empty(B, L, device="cuda")
    accept = torch.empty(B, L, dtype=torch.uint8, device="cuda")
    acc_idx = torch.empty(B, L, dtype=torch.int32, device="cuda")
    n_acc = torch.empty(B, dtype=torch.int32, device="cuda")
    seed, total_steps = seed_for(4, 1000), 0
    for block in range(cfg.n_blocks):
        g_masked = torch.ones(B, L, dtype=torch.uint8, device="cuda")
        g_tokens = torch.full((B, L), -1, dtype=torch.int32, device="cuda")
        o_masked, o_tokens = np.ones((B, L), np.uint8), np.full((B, L), -1, np.int32)
        step = 0
        while o_masked.any():
            seed += 1
            q_len = o_masked.sum(1).astype(np.int32)           # the still-masked suffix is the active window
            g_qlen = torch.from_numpy(q_len).cuda()
            q, kn, vn = make_attn_inputs(NL, B, cfg.n_q_heads, H, L, D, seed, device="cuda")
            out = _attn_all_layers(dev, cfg, cache, q, kn, vn, g_qlen, int(o_len.max()))
            last_step = bool((o_masked.sum(1) <= 1).all())
            if block in (0, cfg.n_blocks - 1) and (step == 0 or last_step):
                _check_attn_layers(oracle, ck, cv, cache_len, q, kn, vn, g_qlen, out, [0, NL // 2, NL - 1])
            logits = make_logits(B, L, V, cfg.logit_sigma, seed, device="cuda")
            o_tok, o_conf, _, _ = oracle.unmask_select(logits.cpu().numpy(), o_masked.copy(), o_tokens.copy(), 0)
            dlm.dlm_unmask_select(dev.ctx, logits, B, L, V, g_masked, g_tokens, 0, tok, conf, None, None, uws)
            np.testing.assert_array_equal(tok.cpu().numpy(), o_tok)
            on = o_masked.astype(bool)
            np.testing.assert_allclose(conf.cpu().numpy()[on], o_conf[on], rtol=CONF_RTOL)
            tok_dlm = torch.from_numpy(np.where(o_tok < 0, 0, o_tok).astype(np.int32))
            tok_ar = make_tok_ar(tok_dlm, cfg.p_agree, V, seed)
            dlm.dlm_guided_accept(dev.ctx, tok_dlm.cuda(), tok_ar.cuda(), B, L, g_masked, g_tokens, 0, accept, acc_idx, n_acc)
            o_acc, o_idx, o_n = oracle.guided_accept(tok_dlm.numpy(), tok_ar.numpy(), o_masked, o_tokens, 0)
            # accepted rows are appended and visible at once; rows are named by block position, as the bench does
            dlm.dlm_kv_cache_commit(dev.ctx, cache, kn, vn, L, acc_idx, None, dlm.DLM_DST_APPEND, n_acc, L, 1, 0, NL)
            oracle.kv_cache_commit(o_ck, o_cv, o_len, bf16_bits(kn), bf16_bits(vn), o_idx, None, o_n, L, True)
            np.testing.assert_array_equal(accept.cpu().numpy(), o_acc)
            np.testing.assert_array_equal(acc_idx.cpu().numpy(), o_idx)
            np.testing.assert_array_equal(n_acc.cpu().numpy(), o_n)
            np.testing.assert_array_equal(g_masked.cpu().numpy(), o_masked)
            np.testing.assert_array_equal(g_tokens.cpu().numpy(), o_tokens)
            np.testing.assert_array_equal(cache_len.cpu().numpy(), o_len)
            step += 1
        total_steps += step
        np.testing.assert_array_equal(o_len, np.full((B,), cfg.prompt_len + (block + 1) * L, np.int32))
    assert dev.status() == 0
    assert 8 * cfg.n_blocks <= total_steps <= L * cfg.n_blocks      # about 79 expected at p_agree 0.8
    np.testing.assert_array_equal(bf16_bits(ck), o_ck)
    np.testing.assert_array_equal(bf16_bits(cv), o_cv)
