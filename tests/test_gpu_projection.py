"""GPU parity of dlm_window_qkv_project and dlm_window_out_project against the oracle, through the C-ABI.
bf16 inputs and outputs, fp32 accumulation; unit-scale outputs, so the attention step's tolerance applies:
max |err| <= 2e-2, mean |err| <= 2e-3 against the oracle's fp64 sums of the same bf16 inputs."""
import numpy as np
import pytest
import torch

import paper_2505_21467_b200 as dlm
from helpers import ATTN_MAX_ERR, ATTN_MEAN_ERR, Dev
from workloads import make_kv_rows, widen

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev():
    return Dev()


def _close(got, ref, what):
    g = got.float().cpu().numpy()
    assert np.isfinite(g).all(), what
    err = np.abs(g - ref)
    assert err.max() <= ATTN_MAX_ERR and err.mean() <= ATTN_MEAN_ERR, (what, float(err.max()), float(err.mean()))


def _qkv_case(dev, oracle, B, q_cap, dm, Hq, Hkv, D, with_bias, seed):
    n_out = (Hq + 2 * Hkv) * D
    x = make_kv_rows((B, q_cap, dm), seed, "cuda")
    w = (torch.randn(n_out, dm, generator=torch.Generator("cuda").manual_seed(seed + 1), device="cuda") * dm ** -0.5).to(torch.bfloat16)
    bias = make_kv_rows((n_out,), seed + 2, "cuda") if with_bias else None
    nan = float("nan")
    q = torch.full((B, Hq, q_cap, D), nan, dtype=torch.bfloat16, device="cuda")
    k = torch.full((B, Hkv, q_cap, D), nan, dtype=torch.bfloat16, device="cuda")
    v = torch.full((B, Hkv, q_cap, D), nan, dtype=torch.bfloat16, device="cuda")
    ws = dev.workspace(dlm.dlm_window_proj_workspace_bytes(dev.ctx, B * q_cap, n_out, dm))
    dlm.dlm_window_qkv_project(dev.ctx, x, w, bias, B, q_cap, dm, Hq, Hkv, D, q, k, v, ws)
    assert dev.status() == 0
    rq, rk, rv = oracle.qkv_project(widen(x), widen(w), None if bias is None else widen(bias), Hq, Hkv, D)
    _close(q, rq, "q"); _close(k, rk, "k"); _close(v, rv, "v")
    return q, k, v


@pytest.mark.parametrize("B,q_cap,dm,Hq,Hkv,D,with_bias", [
    (1, 32, 3584, 28, 4, 128, True),      # Dream-7B widths, one block of 32 rows: K split over the SMs
    (8, 32, 3584, 28, 4, 128, True),      # the guided config's batch: 256 rows
    (1, 256, 3584, 28, 4, 128, False),    # the paper's window of 256 rows
    (4, 64, 4096, 32, 32, 128, False),    # LLaDA-8B widths (no bias), batch 4 x block 64
    (1, 20, 512, 4, 2, 128, True),        # ragged rows (20 of 32)
    (3, 100, 256, 2, 1, 128, True),       # 300 rows: two row chunks, the second ragged
    (2, 7, 128, 4, 2, 64, False),         # head_dim 64 (two heads per feature tile), K too short to split
])
def test_qkv_projection(dev, oracle, B, q_cap, dm, Hq, Hkv, D, with_bias):
    _qkv_case(dev, oracle, B, q_cap, dm, Hq, Hkv, D, with_bias, seed=B * 1000 + q_cap)


def test_qkv_projection_feeds_the_attention_step(dev, oracle):
    """The projection writes Q / Kn / Vn where the attention step reads them: project, attend, compare the attention
    output with the oracle run on the projected (bf16) tensors."""
    B, q_cap, dm, Hq, Hkv, D, Lc = 2, 32, 1024, 8, 2, 128, 300
    q, kn, vn = _qkv_case(dev, oracle, B, q_cap, dm, Hq, Hkv, D, True, seed=77)
    ck, cv = make_kv_rows((1, B, Hkv, Lc + q_cap, D), 5, "cuda"), make_kv_rows((1, B, Hkv, Lc + q_cap, D), 6, "cuda")
    cache_len = torch.full((B,), Lc, dtype=torch.int32, device="cuda")
    cache = dlm.make_kv_cache(ck, cv, cache_len)
    out = torch.empty(1, B, Hq, q_cap, D, dtype=torch.bfloat16, device="cuda")
    ws = dev.workspace(dlm.dlm_attn_workspace_bytes(dev.ctx, cache, 1, Hq, q_cap))
    dlm.dlm_freecache_attn_step(dev.ctx, cache, 0, 1, q[None], kn[None], vn[None], Hq, q_cap, None, 0.0, Lc, out, None, ws)
    assert dev.status() == 0
    ref, _ = oracle.attn_step(widen(ck[0]), widen(cv[0]), cache_len.cpu().numpy(), widen(q), widen(kn), widen(vn))
    _close(out[0], ref, "attention over projected rows")


@pytest.mark.parametrize("B,q_cap,dm,Hq,D,with_bias", [
    (1, 32, 3584, 28, 128, False),       # Dream-7B widths
    (8, 32, 3584, 28, 128, True),        # 256 rows: one box of 32 rows per batch element
    (2, 40, 512, 4, 64, True),           # head_dim 64, 80 rows
    (1, 13, 256, 2, 128, False),         # ragged rows, short K
])
def test_out_projection(dev, oracle, B, q_cap, dm, Hq, D, with_bias):
    seed = 31 * B + q_cap
    o = make_kv_rows((B, Hq, q_cap, D), seed, "cuda")
    wo = (torch.randn(dm, Hq * D, generator=torch.Generator("cuda").manual_seed(seed + 1), device="cuda") * (Hq * D) ** -0.5).to(torch.bfloat16)
    bias = make_kv_rows((dm,), seed + 2, "cuda") if with_bias else None
    y = torch.full((B, q_cap, dm), float("nan"), dtype=torch.bfloat16, device="cuda")
    ws = dev.workspace(dlm.dlm_window_proj_workspace_bytes(dev.ctx, B * q_cap, dm, Hq * D))
    dlm.dlm_window_out_project(dev.ctx, o, wo, bias, B, q_cap, dm, Hq, D, y, ws)
    assert dev.status() == 0
    _close(y, oracle.out_project(widen(o), widen(wo), None if bias is None else widen(bias)), "y")


def test_projection_argument_errors(dev):
    x = torch.zeros(64 * 64, dtype=torch.bfloat16, device="cuda")
    ws = dev.workspace(1 << 20)
    bad = [((1, 4, 100, 4, 2, 128), dlm.DLM_ERR_UNSUPPORTED),      # d_model not a multiple of 64
           ((1, 4, 128, 1, 1, 24), dlm.DLM_ERR_UNSUPPORTED),       # output features not a multiple of 128
           ((0, 4, 128, 4, 2, 128), dlm.DLM_ERR_SHAPE)]
    for (B, q_cap, dm, Hq, Hkv, D), code in bad:
        with pytest.raises(dlm.DlmError) as e:
            dlm.dlm_window_qkv_project(dev.ctx, x, x, None, B, q_cap, dm, Hq, Hkv, D, x, x, x, ws)
        assert e.value.code == code
    with pytest.raises(dlm.DlmError) as e:
        dlm.dlm_window_out_project(dev.ctx, x, x, None, 2, 13, 128, 2, 128, x, ws)     # batch > 1 needs q_cap % 8 == 0
    assert e.value.code == dlm.DLM_ERR_UNSUPPORTED
    assert dev.status() == 0


def _rope_tables(B, q_cap, D, seed, positions=None):
    """cos / sin fp32 [B][q_cap][D/2]: angles position * base^(-2 d / D), the rows' positions drawn at random."""
    rng = np.random.default_rng(seed)
    pos = rng.integers(0, 4096, (B, q_cap)) if positions is None else positions
    inv = 10000.0 ** (-np.arange(D // 2) * 2.0 / D)
    th = pos[..., None] * inv
    return torch.from_numpy(np.cos(th).astype(np.float32)).cuda(), torch.from_numpy(np.sin(th).astype(np.float32)).cuda()


@pytest.mark.parametrize("B,q_cap,dm,Hq,Hkv,D,with_bias", [
    (1, 32, 3584, 28, 4, 128, True),      # Dream-7B widths: K split, the partner feature is 16 lanes away in the final reduction
    (8, 32, 3584, 28, 4, 128, False),     # 256 rows
    (4, 64, 4096, 32, 32, 128, False),    # LLaDA-8B widths
    (1, 20, 512, 4, 2, 128, True),        # ragged rows
    (3, 100, 256, 2, 1, 128, True),       # two row chunks
    (2, 7, 128, 4, 2, 64, False),         # head_dim 64, K too short to split: the partner comes through shared memory
    (2, 40, 1024, 6, 3, 64, True),        # head_dim 64 with the K split: two heads per tile, partner 8 lanes away; a tile
                                          # straddles the last key head and the first value head
    (1, 9, 128, 1, 1, 128, True),         # K too short to split, head_dim 128: the partner sits in another warp
])
def test_qkv_projection_with_rotary_embedding(dev, oracle, B, q_cap, dm, Hq, Hkv, D, with_bias):
    seed = 7 * B + q_cap
    n_out = (Hq + 2 * Hkv) * D
    x = make_kv_rows((B, q_cap, dm), seed, "cuda")
    w = (torch.randn(n_out, dm, generator=torch.Generator("cuda").manual_seed(seed + 1), device="cuda") * dm ** -0.5).to(torch.bfloat16)
    bias = make_kv_rows((n_out,), seed + 2, "cuda") if with_bias else None
    cs, sn = _rope_tables(B, q_cap, D, seed + 3)
    nan = float("nan")
    q = torch.full((B, Hq, q_cap, D), nan, dtype=torch.bfloat16, device="cuda")
    k = torch.full((B, Hkv, q_cap, D), nan, dtype=torch.bfloat16, device="cuda")
    v = torch.full((B, Hkv, q_cap, D), nan, dtype=torch.bfloat16, device="cuda")
    ws = dev.workspace(dlm.dlm_window_proj_workspace_bytes(dev.ctx, B * q_cap, n_out, dm))
    dlm.dlm_window_qkv_project_rope(dev.ctx, x, w, bias, cs, sn, B, q_cap, dm, Hq, Hkv, D, q, k, v, ws)
    assert dev.status() == 0
    rq, rk, rv = oracle.qkv_project_rope(widen(x), widen(w), None if bias is None else widen(bias), cs.cpu().numpy(),
                                         sn.cpu().numpy(), Hq, Hkv, D)
    _close(q, rq, "q"); _close(k, rk, "k"); _close(v, rv, "v")
    # the value heads are exactly those of the plain call
    q2, k2, v2 = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    dlm.dlm_window_qkv_project(dev.ctx, x, w, bias, B, q_cap, dm, Hq, Hkv, D, q2, k2, v2, ws)
    assert torch.equal(v, v2) and not torch.equal(q, q2)


def test_rotary_projection_argument_errors(dev):
    x = torch.zeros(1, 8, 64, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(3 * 32 * 4, 64, dtype=torch.bfloat16, device="cuda")
    t = torch.zeros(1, 8, 16, device="cuda")
    o = torch.zeros(1, 4, 8, 32, dtype=torch.bfloat16, device="cuda")
    ws = dev.workspace(1 << 20)
    with pytest.raises(dlm.DlmError) as e:     # head_dim 32
        dlm.dlm_window_qkv_project_rope(dev.ctx, x, w, None, t, t, 1, 8, 64, 4, 4, 32, o, o, o, ws)
    assert e.value.code == dlm.DLM_ERR_UNSUPPORTED
    with pytest.raises(dlm.DlmError) as e:
        dlm.dlm_window_qkv_project_rope(dev.ctx, x, w, None, None, t, 1, 8, 64, 4, 4, 32, o, o, o, ws)
    assert e.value.code == dlm.DLM_ERR_NULL
    assert dev.status() == 0


@pytest.mark.parametrize("B,q_cap,dm,Hq,Hkv,D,Lcap,cache_len,q_len,rope", [
    (1, 32, 3584, 28, 4, 128, 1100, [1024], None, True),          # Dream-7B widths: K split, 8-byte stores into the cache
    (4, 64, 1024, 8, 8, 128, 300, [200, 0, 236, 17], [64, 5, 64, 0], False),   # ragged active rows, one slot range ending at capacity
    (2, 7, 128, 4, 2, 64, 40, [3, 30], [7, 6], True),             # unsplit K: element-wise stores
])
def test_projection_stages_the_window_rows_in_the_cache(dev, oracle, B, q_cap, dm, Hq, Hkv, D, Lcap, cache_len, q_len, rope):
    """K/V of the window written by the projection's epilogue to cache rows cache_len[b] + i of one layer: those rows
    match the oracle's projection, carry the same bits as k_out / v_out, and nothing else in the cache changes."""
    NL, layer, seed = 3, 1, 50 + B
    n_out = (Hq + 2 * Hkv) * D
    x = make_kv_rows((B, q_cap, dm), seed, "cuda")
    w = (torch.randn(n_out, dm, generator=torch.Generator("cuda").manual_seed(seed + 1), device="cuda") * dm ** -0.5).to(torch.bfloat16)
    bias = make_kv_rows((n_out,), seed + 2, "cuda")
    cs, sn = _rope_tables(B, q_cap, D, seed + 3) if rope else (None, None)
    ck, cv = make_kv_rows((NL, B, Hkv, Lcap, D), seed + 4, "cuda"), make_kv_rows((NL, B, Hkv, Lcap, D), seed + 5, "cuda")
    ck0, cv0 = ck.clone(), cv.clone()
    cl = torch.tensor(cache_len, dtype=torch.int32, device="cuda")
    ql = None if q_len is None else torch.tensor(q_len, dtype=torch.int32, device="cuda")
    cache = dlm.make_kv_cache(ck, cv, cl)
    q = torch.empty(B, Hq, q_cap, D, dtype=torch.bfloat16, device="cuda")
    k = torch.empty(B, Hkv, q_cap, D, dtype=torch.bfloat16, device="cuda")
    v = torch.empty_like(k)
    ws = dev.workspace(dlm.dlm_window_proj_workspace_bytes(dev.ctx, B * q_cap, n_out, dm))
    dlm.dlm_window_qkv_project_stage(dev.ctx, x, w, bias, cs, sn, B, q_cap, dm, Hq, Hkv, D, ql, q, k, v, cache, layer, ws)
    assert dev.status() == 0
    assert torch.equal(cl.cpu(), torch.tensor(cache_len, dtype=torch.int32))
    if rope:
        rq, rk, rv = oracle.qkv_project_rope(widen(x), widen(w), widen(bias), cs.cpu().numpy(), sn.cpu().numpy(), Hq, Hkv, D)
    else:
        rq, rk, rv = oracle.qkv_project(widen(x), widen(w), widen(bias), Hq, Hkv, D)
    _close(q, rq, "q"); _close(k, rk, "k"); _close(v, rv, "v")
    touched = torch.zeros(NL, B, Hkv, Lcap, dtype=torch.bool, device="cuda")
    for b in range(B):
        n = q_cap if q_len is None else q_len[b]
        lo = cache_len[b]
        touched[layer, b, :, lo:lo + n] = True
        if n:
            for got, out, ref in ((ck, k, rk), (cv, v, rv)):
                assert torch.equal(got[layer, b, :, lo:lo + n], out[b, :, :n])            # the same bits as the fresh copy
                _close(got[layer, b, :, lo:lo + n], ref[b, :, :n], "staged rows")         # and the oracle's values
    assert torch.equal(ck[~touched], ck0[~touched]) and torch.equal(cv[~touched], cv0[~touched])


def test_projection_staging_reports_rows_without_room_and_argument_errors(dev):
    B, q_cap, dm, Hq, Hkv, D, Lcap = 2, 8, 128, 2, 1, 128, 20
    n_out = (Hq + 2 * Hkv) * D
    x = make_kv_rows((B, q_cap, dm), 1, "cuda")
    w = make_kv_rows((n_out, dm), 2, "cuda")
    ck, cv = make_kv_rows((1, B, Hkv, Lcap, D), 3, "cuda"), make_kv_rows((1, B, Hkv, Lcap, D), 4, "cuda")
    ck0 = ck.clone()
    cl = torch.tensor([15, 2], dtype=torch.int32, device="cuda")        # sequence 0: rows 5..7 have no slot
    cache = dlm.make_kv_cache(ck, cv, cl)
    q = torch.empty(B, Hq, q_cap, D, dtype=torch.bfloat16, device="cuda")
    k = torch.empty(B, Hkv, q_cap, D, dtype=torch.bfloat16, device="cuda")
    v = torch.empty_like(k)
    ws = dev.workspace(dlm.dlm_window_proj_workspace_bytes(dev.ctx, B * q_cap, n_out, dm))
    dlm.dlm_window_qkv_project_stage(dev.ctx, x, w, None, None, None, B, q_cap, dm, Hq, Hkv, D, None, q, k, v, cache, 0, ws)
    assert dev.status() == dlm.DLM_ERR_CAPACITY
    assert torch.equal(ck[0, 0, :, 15:20], k[0, :, :5]) and torch.equal(ck[0, 1, :, 2:10], k[1]) and torch.equal(ck[0, 0, :, :15], ck0[0, 0, :, :15])
    for kwargs, code in ((dict(layer=1), dlm.DLM_ERR_SHAPE), (dict(layer=-1), dlm.DLM_ERR_SHAPE)):
        with pytest.raises(dlm.DlmError) as e:
            dlm.dlm_window_qkv_project_stage(dev.ctx, x, w, None, None, None, B, q_cap, dm, Hq, Hkv, D, None, q, k, v, cache,
                                             kwargs["layer"], ws)
        assert e.value.code == code
    t = torch.zeros(B, q_cap, D // 2, device="cuda")
    with pytest.raises(dlm.DlmError) as e:      # one table without the other
        dlm.dlm_window_qkv_project_stage(dev.ctx, x, w, None, t, None, B, q_cap, dm, Hq, Hkv, D, None, q, k, v, cache, 0, ws)
    assert e.value.code == dlm.DLM_ERR_NULL
    assert dev.status() == 0


def test_two_steps_without_a_commit_call(dev, oracle):
    """A block's life without dlm_kv_cache_commit: every step projects and stages the window, attends over the visible
    cache and the fresh rows; completing the block is adding its length to cache_len, after which the next block's
    attention sees the rows staged by the last step.  The oracle runs projection, an explicit commit and attention."""
    B, q_cap, dm, Hq, Hkv, D, Lcap, L0 = 2, 32, 512, 8, 2, 128, 400, 150
    n_out = (Hq + 2 * Hkv) * D
    w = (torch.randn(n_out, dm, generator=torch.Generator("cuda").manual_seed(5), device="cuda") * dm ** -0.5).to(torch.bfloat16)
    ck, cv = make_kv_rows((1, B, Hkv, Lcap, D), 6, "cuda"), make_kv_rows((1, B, Hkv, Lcap, D), 7, "cuda")
    o_ck, o_cv = widen(ck[0]).copy(), widen(cv[0]).copy()
    cl = torch.full((B,), L0, dtype=torch.int32, device="cuda")
    cache = dlm.make_kv_cache(ck, cv, cl)
    q = torch.empty(B, Hq, q_cap, D, dtype=torch.bfloat16, device="cuda")
    k = torch.empty(B, Hkv, q_cap, D, dtype=torch.bfloat16, device="cuda")
    v = torch.empty_like(k)
    out = torch.empty(1, B, Hq, q_cap, D, dtype=torch.bfloat16, device="cuda")
    ws = dev.workspace(max(dlm.dlm_window_proj_workspace_bytes(dev.ctx, B * q_cap, n_out, dm),
                           dlm.dlm_attn_workspace_bytes(dev.ctx, cache, 1, Hq, q_cap)))
    o_len = np.full((B,), L0, np.int32)
    for step in range(2):
        x = make_kv_rows((B, q_cap, dm), 20 + step, "cuda")
        cs, sn = _rope_tables(B, q_cap, D, 0, positions=np.tile(np.arange(q_cap) + L0 + step * q_cap, (B, 1)))
        dlm.dlm_window_qkv_project_stage(dev.ctx, x, w, None, cs, sn, B, q_cap, dm, Hq, Hkv, D, None, q, k, v, cache, 0, ws)
        dlm.dlm_freecache_attn_step(dev.ctx, cache, 0, 1, q[None], k[None], v[None], Hq, q_cap, None, 0.0, 0, out, None, ws)
        assert dev.status() == 0
        rq, rk, rv = oracle.qkv_project_rope(widen(x), widen(w), None, cs.cpu().numpy(), sn.cpu().numpy(), Hq, Hkv, D)
        rq, rk, rv = (torch.from_numpy(a).to(torch.bfloat16).float().numpy() for a in (rq, rk, rv))   # what bf16 storage keeps
        ref, _ = oracle.attn_step(o_ck, o_cv, o_len, rq, rk, rv)
        _close(out[0], ref, f"attention of step {step}")
        # the block is complete: its rows become visible (GPU: the staged rows; oracle: an explicit copy)
        cl += q_cap
        for b in range(B):
            o_ck[b, :, o_len[b]:o_len[b] + q_cap] = rk[b]
            o_cv[b, :, o_len[b]:o_len[b] + q_cap] = rv[b]
        o_len += q_cap
