"""Whole denoising loops through the C-ABI with the state kept on the device between calls (cache, cache_len, mask,
tokens, selection lists), mirrored step by step by the CPU oracle on the same seeded inputs: the top-k policy with staged
commits and a block-end freeze, and the guided policy with prefix accepts, appends and a shrinking window."""
import numpy as np
import pytest
import torch

import paper_2505_21467_b200 as dlm
from workloads import bf16_bits, make_attn_inputs, make_cache, make_logits, make_tok_ar, widen
from helpers import ATTN_MAX_ERR, ATTN_MEAN_ERR, Dev, topk_margin

pytestmark = pytest.mark.gpu

NL, B, HQ, HKV, D, PROMPT, LBLK, V = 2, 2, 4, 2, 64, 100, 16, 3000


@pytest.fixture(scope="module")
def dev():
    return Dev()


def _attn_both(dev, oracle, g_cache, g_len, o_ck, o_cv, o_len, q, kn, vn, q_len=None):
    out = torch.empty(NL, B, HQ, LBLK, D, dtype=torch.bfloat16, device="cuda")
    ws = dev.workspace(dlm.dlm_attn_workspace_bytes(dev.ctx, g_cache, NL, HQ, LBLK))
    g_qlen = None if q_len is None else torch.from_numpy(q_len).cuda()
    dlm.dlm_freecache_attn_step(dev.ctx, g_cache, 0, NL, q.cuda(), kn.cuda(), vn.cuda(), HQ, LBLK, g_qlen, 0.0, 0, out, None, ws)
    for layer in range(NL):
        ck32 = (o_ck[layer].astype(np.uint32) << 16).view(np.float32)
        cv32 = (o_cv[layer].astype(np.uint32) << 16).view(np.float32)
        ref, _ = oracle.attn_step(ck32, cv32, o_len, widen(q[layer]), widen(kn[layer]), widen(vn[layer]), q_len)
        err = np.abs(out[layer].float().cpu().numpy() - ref)
        assert err.max() <= ATTN_MAX_ERR and err.mean() <= ATTN_MEAN_ERR, (layer, err.max(), err.mean())


def _state(seed):
    ck, cv = make_cache(NL, B, HKV, PROMPT + 2 * LBLK, D, seed)
    g_ck, g_cv = ck.cuda(), cv.cuda()
    g_len = torch.full((B,), PROMPT, dtype=torch.int32, device="cuda")
    return (g_ck, g_cv, g_len, dlm.make_kv_cache(g_ck, g_cv, g_len), bf16_bits(ck).copy(), bf16_bits(cv).copy(),
            np.full((B,), PROMPT, np.int32))


def test_topk_policy_two_blocks(dev, oracle):
    k, steps = 4, LBLK // 4
    g_ck, g_cv, g_len, g_cache, o_ck, o_cv, o_len = _state(501)
    uws = dev.workspace(dlm.dlm_unmask_workspace_bytes(dev.ctx, B, LBLK, V))
    seed = 600
    for block in range(2):
        g_masked = torch.ones(B, LBLK, dtype=torch.uint8, device="cuda")
        g_tokens = torch.full((B, LBLK), -1, dtype=torch.int32, device="cuda")
        o_masked, o_tokens = np.ones((B, LBLK), np.uint8), np.full((B, LBLK), -1, np.int32)
        for step in range(steps):
            q, kn, vn = make_attn_inputs(NL, B, HQ, HKV, LBLK, D, seed)
            _attn_both(dev, oracle, g_cache, g_len, o_ck, o_cv, o_len, q, kn, vn)
            while True:   # inputs whose k-th and (k+1)-th confidences are not a near-tie
                seed += 1
                logits = make_logits(B, LBLK, V, (1.0, 8.0), seed)
                m2, t2 = o_masked.copy(), o_tokens.copy()
                o_tok, o_conf, o_sel, o_n = oracle.unmask_select(logits.numpy(), m2, t2, k)
                if topk_margin(o_conf, o_masked, k) > 1e-4:
                    break
            o_masked, o_tokens = m2, t2
            tok = torch.empty(B, LBLK, dtype=torch.int32, device="cuda")
            conf = torch.empty(B, LBLK, device="cuda")
            sel = torch.empty(B, k, dtype=torch.int32, device="cuda")
            n_sel = torch.empty(B, dtype=torch.int32, device="cuda")
            dlm.dlm_unmask_select(dev.ctx, logits.cuda(), B, LBLK, V, g_masked, g_tokens, k, tok, conf, sel, n_sel, uws)
            last = step == steps - 1
            if last:   # block complete: freeze all its rows
                dlm.dlm_kv_cache_commit(dev.ctx, g_cache, kn.cuda(), vn.cuda(), LBLK, None, None, dlm.DLM_DST_APPEND, None,
                                        LBLK, 1, 0, NL)
                oracle.kv_cache_commit(o_ck, o_cv, o_len, bf16_bits(kn), bf16_bits(vn), None, None, None, LBLK, True)
            else:      # stage the rows just unmasked; the counts stay on the device
                dlm.dlm_kv_cache_commit(dev.ctx, g_cache, kn.cuda(), vn.cuda(), LBLK, sel, None, dlm.DLM_DST_WINDOW, n_sel,
                                        k, 0, 0, NL)
                oracle.kv_cache_commit(o_ck, o_cv, o_len, bf16_bits(kn), bf16_bits(vn), o_sel, None, o_n, k, False, dst_mode=1)
            np.testing.assert_array_equal(tok.cpu().numpy(), o_tok)
            np.testing.assert_array_equal(sel.cpu().numpy(), o_sel)
            np.testing.assert_array_equal(n_sel.cpu().numpy(), o_n)
            np.testing.assert_array_equal(g_masked.cpu().numpy(), o_masked)
            np.testing.assert_array_equal(g_tokens.cpu().numpy(), o_tokens)
        assert not o_masked.any()
    assert dev.status() == 0
    np.testing.assert_array_equal(g_len.cpu().numpy(), o_len)
    np.testing.assert_array_equal(bf16_bits(g_ck), o_ck)
    np.testing.assert_array_equal(bf16_bits(g_cv), o_cv)


def test_guided_policy_one_block(dev, oracle):
    g_ck, g_cv, g_len, g_cache, o_ck, o_cv, o_len = _state(701)
    uws = dev.workspace(dlm.dlm_unmask_workspace_bytes(dev.ctx, B, LBLK, V))
    g_masked = torch.ones(B, LBLK, dtype=torch.uint8, device="cuda")
    g_tokens = torch.full((B, LBLK), -1, dtype=torch.int32, device="cuda")
    o_masked, o_tokens = np.ones((B, LBLK), np.uint8), np.full((B, LBLK), -1, np.int32)
    seed, n_steps = 800, 0
    while o_masked.any():
        seed += 1
        n_steps += 1
        q_len = o_masked.sum(1).astype(np.int32)            # the window shrinks as prefixes are accepted
        q, kn, vn = make_attn_inputs(NL, B, HQ, HKV, LBLK, D, seed)
        _attn_both(dev, oracle, g_cache, g_len, o_ck, o_cv, o_len, q, kn, vn, q_len)
        logits = make_logits(B, LBLK, V, (1.0, 8.0), seed)
        o_tok, _, _, _ = oracle.unmask_select(logits.numpy(), o_masked.copy(), o_tokens.copy(), 0)
        tok = torch.empty(B, LBLK, dtype=torch.int32, device="cuda")
        conf = torch.empty(B, LBLK, device="cuda")
        dlm.dlm_unmask_select(dev.ctx, logits.cuda(), B, LBLK, V, g_masked, g_tokens, 0, tok, conf, None, None, uws)
        np.testing.assert_array_equal(tok.cpu().numpy(), o_tok)
        tok_dlm = torch.from_numpy(np.where(o_tok < 0, 0, o_tok).astype(np.int32))
        tok_ar = make_tok_ar(tok_dlm, 0.8, V, seed)
        accept = torch.empty(B, LBLK, dtype=torch.uint8, device="cuda")
        acc_idx = torch.empty(B, LBLK, dtype=torch.int32, device="cuda")
        n_acc = torch.empty(B, dtype=torch.int32, device="cuda")
        dlm.dlm_guided_accept(dev.ctx, tok_dlm.cuda(), tok_ar.cuda(), B, LBLK, g_masked, g_tokens, 0, accept, acc_idx, n_acc)
        o_acc, o_idx, o_n = oracle.guided_accept(tok_dlm.numpy(), tok_ar.numpy(), o_masked, o_tokens, 0)
        # accepted rows are appended and become visible at once
        dlm.dlm_kv_cache_commit(dev.ctx, g_cache, kn.cuda(), vn.cuda(), LBLK, acc_idx, None, dlm.DLM_DST_APPEND, n_acc, LBLK,
                                1, 0, NL)
        oracle.kv_cache_commit(o_ck, o_cv, o_len, bf16_bits(kn), bf16_bits(vn), o_idx, None, o_n, LBLK, True)
        np.testing.assert_array_equal(accept.cpu().numpy(), o_acc)
        np.testing.assert_array_equal(acc_idx.cpu().numpy(), o_idx)
        np.testing.assert_array_equal(n_acc.cpu().numpy(), o_n)
        np.testing.assert_array_equal(g_masked.cpu().numpy(), o_masked)
        np.testing.assert_array_equal(g_tokens.cpu().numpy(), o_tokens)
        np.testing.assert_array_equal(g_len.cpu().numpy(), o_len)
    assert 1 < n_steps <= LBLK and dev.status() == 0
    np.testing.assert_array_equal(o_len, np.full((B,), PROMPT + LBLK, np.int32))
    np.testing.assert_array_equal(bf16_bits(g_ck), o_ck)
    np.testing.assert_array_equal(bf16_bits(g_cv), o_cv)
