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
