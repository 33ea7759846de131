"""GPU parity of dlm_freecache_attn_step against the CPU oracle, through the C-ABI.
Tolerance (fp32 oracle, unit-scale bf16 inputs, bf16 output): max |err| <= 2e-2, mean |err| <= 2e-3."""
import numpy as np
import pytest
import torch

import paper_2505_21467_b200 as dlm
from workloads import get_config, make_attn_inputs, make_cache, seed_for
from helpers import Dev, assert_attn_close, gpu_attn_step, oracle_attn_layers

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev():
    return Dev()


def _i32(a):
    return torch.tensor(np.asarray(a), dtype=torch.int32, device="cuda")


def _case(dev, oracle, NL, B, Hq, Hkv, D, Lcap, q_cap, cache_len, q_len=None, seed=1, layer_begin=0, nl=None,
          scale=0.0, layers=None, hint=0, device="cpu"):
    nl = NL - layer_begin if nl is None else nl
    ck, cv = make_cache(NL, B, Hkv, Lcap, D, seed, device=device)
    q, kn, vn = make_attn_inputs(nl, B, Hq, Hkv, q_cap, D, seed + 1, device=device)
    cl = _i32(cache_len)
    ql = None if q_len is None else _i32(q_len)
    out, lse = gpu_attn_step(dev, ck.cuda(), cv.cuda(), cl, q.cuda(), kn.cuda(), vn.cuda(), ql, scale, layer_begin,
                             layer_begin + nl, hint=hint)
    assert dev.status() == 0
    ref = oracle_attn_layers(oracle, ck, cv, cl, q, kn, vn, ql, scale if scale > 0 else None, layer_begin, layers)
    errs = [assert_attn_close(out, lse, ref[lc], lc) for lc in ref]
    return out, lse, errs


def test_tiny_config_full(dev, oracle):
    cfg = get_config(0)
    _case(dev, oracle, cfg.n_layers, cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.capacity,
          cfg.block_len, [cfg.prompt_len], seed=seed_for(0))


@pytest.mark.parametrize("Hq,Hkv,D,Lcap,q_cap,cache_len,q_len", [
    (28, 4, 128, 700, 32, [517, 640], None),            # Dream group of 7: two M tiles, several K tiles, ragged tail
    (28, 4, 128, 700, 32, [517, 0], [32, 7]),           # ragged active rows, one empty cache
    (8, 8, 128, 400, 64, [333, 128], [64, 64]),         # MHA (LLaDA-like), block 64
    (4, 2, 64, 300, 32, [1, 299], [5, 32]),             # head_dim 64
    (2, 1, 64, 200, 128, [130, 77], [128, 100]),        # 256 query rows per KV head, fresh part spans a full tile
    (6, 2, 128, 260, 20, [256, 255], [20, 0]),          # q_cap not a multiple of 16; one element fully inactive
    (3, 3, 128, 129, 1, [129, 128], None),              # a single active row
])
def test_shapes_and_ragged_lengths(dev, oracle, Hq, Hkv, D, Lcap, q_cap, cache_len, q_len):
    out, lse, _ = _case(dev, oracle, 2, 2, Hq, Hkv, D, Lcap, q_cap, cache_len, q_len, seed=Hq * 100 + q_cap)
    if q_len is not None:
        for b, n in enumerate(q_len):
            assert torch.all(out[:, b, :, n:] == 0)


@pytest.mark.parametrize("hint", [1, 0])
def test_both_schedules_whole_units_and_split(dev, oracle, hint):
    """The length hint only picks the schedule: a tiny hint deals the units whole, the default (capacity)
    splits these 16 long units across the SMs; both must match the oracle."""
    _case(dev, oracle, 2, 2, 28, 4, 128, 1400, 32, [1368, 900], [32, 17], seed=77, hint=hint)


@pytest.mark.parametrize("Hq,Hkv,D,Lcap,q_cap,cache_len,q_len", [
    (28, 4, 128, 600, 256, [300], None),                # the paper's window: 256 active rows, Dream heads (7 chunks of 256 rows)
    (4, 4, 128, 520, 512, [0, 0], [512, 333]),          # initial full pass: empty cache, 512 active rows, ragged
    (4, 2, 64, 400, 300, [77, 100], [300, 130]),        # rows per KV head not a multiple of 256, head_dim 64
])
def test_large_windows_in_row_chunks(dev, oracle, Hq, Hkv, D, Lcap, q_cap, cache_len, q_len):
    B = len(cache_len)
    for hint in (1, 0):   # both schedules
        out, lse, _ = _case(dev, oracle, 1, B, Hq, Hkv, D, Lcap, q_cap, cache_len, q_len, seed=Hq * 1000 + q_cap, hint=hint)
        if q_len is not None:
            for b, n in enumerate(q_len):
                assert torch.all(out[:, b, :, n:] == 0)


@pytest.mark.parametrize("scale", [0.2, 1.0])
def test_scores_that_keep_outgrowing_the_running_maximum(dev, oracle, scale):
    """Keys grow along the cache and the softmax scale is large, so later tiles bring scores far above the
    maximum in use (by tens of powers of two): the deferred rescaling of O has to fire, repeatedly, and the result
    must still match.  Both schedules."""
    NL, B, Hq, Hkv, D, Lc, q_cap = 1, 2, 14, 2, 128, 1500, 32
    ck, cv = make_cache(NL, B, Hkv, Lc + 40, D, 91)
    q, kn, vn = make_attn_inputs(NL, B, Hq, Hkv, q_cap, D, 92)
    grow = (1.0 + 4.0 * torch.arange(Lc + 40, dtype=torch.float32) / Lc).view(1, 1, 1, -1, 1)
    ck = (ck.float() * grow).to(torch.bfloat16)
    cl = _i32([Lc, Lc - 333])
    for hint in (1, 0):
        out, lse = gpu_attn_step(dev, ck.cuda(), cv.cuda(), cl, q.cuda(), kn.cuda(), vn.cuda(), None, scale, hint=hint)
        assert dev.status() == 0
        ref = oracle_attn_layers(oracle, ck, cv, cl, q, kn, vn, None, scale)
        assert_attn_close(out, lse, ref[0], 0)


def test_many_batch_elements_with_random_lengths(dev, oracle):
    """600 sequences (the limit is 1024), each with its own cache length and window length, some empty."""
    rng = np.random.default_rng(3)
    B, Lcap, q_cap = 600, 70, 8
    cache_len = rng.integers(0, Lcap + 1, B).tolist()
    q_len = rng.integers(0, q_cap + 1, B).tolist()
    out, lse, _ = _case(dev, oracle, 1, B, 2, 1, 64, Lcap, q_cap, cache_len, q_len, seed=606)
    for b, n in enumerate(q_len):
        assert torch.all(out[:, b, :, n:] == 0)


def test_layer_range_and_explicit_scale(dev, oracle):
    _case(dev, oracle, 5, 1, 4, 2, 128, 300, 32, [290], seed=9, layer_begin=2, nl=2, scale=0.05)


def test_poisoned_invisible_rows_do_not_leak(dev, oracle):
    """Rows at or beyond cache_len / q_len may hold NaN: the result must not change (bit for bit)."""
    NL, B, Hq, Hkv, D, Lcap, q_cap = 1, 2, 14, 2, 128, 520, 32
    ck, cv = make_cache(NL, B, Hkv, Lcap, D, 31, device="cuda")
    q, kn, vn = make_attn_inputs(NL, B, Hq, Hkv, q_cap, D, 32, device="cuda")
    cl, ql = _i32([300, 5]), _i32([32, 9])
    base, base_lse = gpu_attn_step(dev, ck, cv, cl, q, kn, vn, ql)
    nan = float("nan")
    ck[:, 0, :, 300:] = nan; cv[:, 0, :, 300:] = nan
    ck[:, 1, :, 5:] = nan; cv[:, 1, :, 5:] = nan
    kn[:, 1, :, 9:] = nan; vn[:, 1, :, 9:] = nan; q[:, 1, :, 9:] = nan
    out, lse = gpu_attn_step(dev, ck, cv, cl, q, kn, vn, ql)
    assert dev.status() == 0
    assert torch.equal(out, base) and torch.equal(lse, base_lse)
    assert torch.isfinite(out.float()).all()


def test_deterministic(dev):
    ck, cv = make_cache(2, 1, 4, 1100, 128, 41, device="cuda")
    q, kn, vn = make_attn_inputs(2, 1, 28, 4, 32, 128, 42, device="cuda")
    cl = _i32([1056])
    a, al = gpu_attn_step(dev, ck, cv, cl, q, kn, vn)
    b, bl = gpu_attn_step(dev, ck, cv, cl, q, kn, vn)
    assert torch.equal(a, b) and torch.equal(al, bl)


def test_argument_errors(dev):
    ck, cv = make_cache(1, 1, 2, 64, 128, 1, device="cuda")
    cl = _i32([10])
    cache = dlm.make_kv_cache(ck, cv, cl)
    ws = dev.workspace(1 << 20)

    def call(Hq=4, q_cap=32, D=128, layer_end=1, ws_=ws):
        q = torch.zeros(1, 1, Hq, q_cap, D, dtype=torch.bfloat16, device="cuda")
        kn = torch.zeros(1, 1, 2, q_cap, D, dtype=torch.bfloat16, device="cuda")
        dlm.dlm_freecache_attn_step(dev.ctx, cache, 0, layer_end, q, kn, kn, Hq, q_cap, None, 0.0, 0,
                                    torch.empty_like(q), None, ws_)

    before = dlm.dlm_launch_count(dev.ctx)
    for kwargs, code in ((dict(Hq=3), dlm.DLM_ERR_UNSUPPORTED), (dict(Hq=4, q_cap=5000), dlm.DLM_ERR_UNSUPPORTED),
                         (dict(layer_end=2), dlm.DLM_ERR_SHAPE),
                         (dict(ws_=ws[8:]), dlm.DLM_ERR_WORKSPACE)):
        with pytest.raises(dlm.DlmError) as e:
            call(**kwargs)
        assert e.value.code == code, kwargs
    assert dlm.dlm_launch_count(dev.ctx) == before
    ck96, cv96 = make_cache(1, 1, 2, 64, 96, 1, device="cuda")
    cache96 = dlm.make_kv_cache(ck96, cv96, cl)
    q = torch.zeros(1, 1, 2, 8, 96, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(dlm.DlmError) as e:
        dlm.dlm_freecache_attn_step(dev.ctx, cache96, 0, 1, q, q, q, 2, 8, None, 0.0, 0, torch.empty_like(q), None, ws)
    assert e.value.code == dlm.DLM_ERR_UNSUPPORTED


def test_out_of_range_lengths_are_clamped_and_reported(dev):
    ck, cv = make_cache(1, 2, 2, 64, 128, 1, device="cuda")
    q, kn, vn = make_attn_inputs(1, 2, 4, 2, 16, 128, 2, device="cuda")
    out, _ = gpu_attn_step(dev, ck, cv, _i32([65, 10]), q, kn, vn)
    assert dev.status() == dlm.DLM_ERR_CAPACITY
    ref, _ = gpu_attn_step(dev, ck, cv, _i32([64, 10]), q, kn, vn)
    assert dev.status() == 0 and torch.equal(out, ref)


def test_dream7b_full_size_layer_batched_first_and_last_step(dev, oracle):
    """The benchmark's launch: all 28 layers in one call at the Dream-7B shape, at the first step
    (cache 1024) and the last (cache 1248); oracle on layers {0, 14, 27}, all heads and rows."""
    cfg = get_config(1)
    for cache_len in (cfg.prompt_len, cfg.capacity - cfg.block_len):
        _case(dev, oracle, cfg.n_layers, cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.capacity,
              cfg.block_len, [cache_len], seed=seed_for(1, cache_len), layers=[0, 14, 27], hint=cache_len,
              device="cuda")


def test_guided_shape_ragged_batch8(dev, oracle):
    """Config 5's shape: batch 8 with ragged cache_len and q_len (accepted prefixes shrink the window)."""
    cfg = get_config(4)
    cache_len = [1024, 1031, 1056, 1100, 1247, 1279, 1088, 1150]
    q_len = [32, 25, 32, 20, 1, 1, 32, 2]
    _case(dev, oracle, 3, cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.capacity, cfg.block_len,
          cache_len, q_len, seed=seed_for(4), layers=[0, 2])


def test_guided_shape_more_units_than_sms_split_schedule(dev, oracle):
    """Config 5's launch form: more units (10 layers x 8 sequences x 4 KV heads = 320) than SMs and still split,
    so a block's share holds whole units and a partial unit at each end, with ragged lengths."""
    cfg = get_config(4)
    cache_len = [1024, 1031, 1056, 1100, 1247, 1279, 1088, 1150]
    q_len = [32, 25, 32, 20, 1, 1, 32, 2]
    _case(dev, oracle, 10, cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.capacity, cfg.block_len,
          cache_len, q_len, seed=seed_for(4, 7), layers=[0, 9], device="cuda")


def test_longctx_shape_sampled_layers(dev, oracle):
    """Config 4: 16384 cached rows, Dream heads; 4 of the 28 layers resident, oracle on two of them."""
    cfg = get_config(3)
    _case(dev, oracle, 4, cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.prompt_len + cfg.block_len,
          cfg.block_len, [cfg.prompt_len], seed=seed_for(3), layers=[0, 3], device="cuda")


def test_llada_shape_sampled(dev, oracle):
    """Config 3's shape at full batch / heads / lengths, 2 layers resident; oracle on one layer."""
    cfg = get_config(2)
    _case(dev, oracle, 2, cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.capacity, cfg.block_len,
          [2048, 2112, 2496, 2300], seed=seed_for(2), layers=[1], device="cuda")


def test_a_wait_that_runs_out_reports_timeout_and_leaves_the_context_usable(dev, oracle):
    """The bounded device-side wait gives up after its limit (here 2 ms on a barrier nothing arrives at): the kernel
    ends normally, the status word says DLM_ERR_TIMEOUT, it is cleared by the read, and the next calls work."""
    dlm.dlm_selftest_wait_timeout(dev.ctx, 2_000_000)
    assert dev.status() == dlm.DLM_ERR_TIMEOUT
    assert dev.status() == 0
    _case(dev, oracle, 1, 1, 4, 2, 64, 200, 16, [150], seed=5)
    with pytest.raises(dlm.DlmError) as e:
        dlm.dlm_selftest_wait_timeout(dev.ctx, 5_000_000_000)
    assert e.value.code == dlm.DLM_ERR_SHAPE


@pytest.mark.parametrize("hint", [1, 0])
def test_the_attention_kernel_gives_up_cleanly_when_its_waits_may_not_wait(dev, oracle, hint):
    """The kernel's own unwinding, in both schedules: with the wait limit set to 0 the first wait whose data is still
    on its way gives up; the producer lets its copies land, the MMA issuers drain, every role reaches the teardown,
    TMEM is released and the kernel ends normally with DLM_ERR_TIMEOUT.  With the limit restored the next call on the
    same context is correct again (nothing of the aborted launch is left behind, ticket words included)."""
    args = dict(NL=2, B=2, Hq=28, Hkv=4, D=128, Lcap=700, q_cap=32, cache_len=[517, 640], seed=4242, hint=hint)
    dlm.dlm_selftest_set_wait_limit(dev.ctx, 0)
    try:
        ck, cv = make_cache(2, 2, 4, 700, 128, 1, device="cuda")
        q, kn, vn = make_attn_inputs(2, 2, 28, 4, 32, 128, 2, device="cuda")
        gpu_attn_step(dev, ck, cv, _i32([517, 640]), q, kn, vn, hint=hint)
        torch.cuda.synchronize()
        assert dev.status() == dlm.DLM_ERR_TIMEOUT
    finally:
        dlm.dlm_selftest_set_wait_limit(dev.ctx, 2_000_000_000)
    assert dev.status() == 0
    _case(dev, oracle, **args)
    with pytest.raises(dlm.DlmError) as e:
        dlm.dlm_selftest_set_wait_limit(dev.ctx, 3_000_000_000)
    assert e.value.code == dlm.DLM_ERR_SHAPE


def _schedule(dev, NL, B, Hq, Hkv, D, Lcap, q_cap, nl, hint=0):
    ck = torch.empty(NL, B, Hkv, Lcap, D, dtype=torch.bfloat16, device="cuda")
    cache = dlm.make_kv_cache(ck, ck, _i32([0] * B))
    return dlm.dlm_selftest_attn_schedule(dev.ctx, cache, nl, Hq, q_cap, hint)


@pytest.mark.parametrize("NL,B,Hq,Hkv,D,Lcap,q_cap,cache_len,q_len", [
    (1, 1, 28, 4, 128, 2200, 32, [2048], None),          # one Dream layer at batch 1: 8 units of 128 rows, 17 key tiles each
    (1, 1, 28, 4, 128, 2200, 32, [2048], [19]),          # ragged active rows
    (1, 2, 28, 4, 128, 900, 32, [517, 0], [32, 7]),      # an empty cache: one key tile, most ranks get none
    (1, 2, 6, 2, 128, 700, 20, [256, 255], [20, 0]),     # one element fully inactive; 60 rows per unit
    (2, 1, 4, 2, 64, 1000, 32, [901], [5]),              # head_dim 64, 64 rows per unit
    (1, 1, 2, 1, 64, 700, 128, [650], [100]),            # 256 rows per unit (two M tiles), fresh part a whole tile
    (1, 1, 8, 8, 128, 1100, 64, [1000], None),           # MHA, 64 rows per unit
    (1, 1, 3, 3, 128, 300, 1, [129], None),              # a single row per unit
])
def test_team_schedule_against_the_oracle_at_every_team_size(dev, oracle, NL, B, Hq, Hkv, D, Lcap, q_cap, cache_len, q_len):
    """Calls with few units give each unit a team of blocks, which split its key tiles and then each reduce a share
    of its outputs over all the team's pieces.  Every team size, and the same call with the schedule switched off,
    matches the oracle."""
    outs = []
    try:
        for tmax in (1 << 20, 8, 3, 2, 1):
            dlm.dlm_selftest_set_attn_team_max(dev.ctx, tmax, force=True)
            sch = _schedule(dev, NL, B, Hq, Hkv, D, Lcap, q_cap, NL)
            assert (sch["team"] > 1) == (tmax > 1) and sch["team"] <= tmax and sch["grid"] % sch["team"] == 0
            out, lse, _ = _case(dev, oracle, NL, B, Hq, Hkv, D, Lcap, q_cap, cache_len, q_len, seed=Hq * 10 + q_cap)
            outs.append(out.float())
            if q_len is not None:
                for b, n in enumerate(q_len):
                    assert torch.all(out[:, b, :, n:] == 0)
    finally:
        dlm.dlm_selftest_set_attn_team_max(dev.ctx, 1 << 20)
    for o in outs[1:]:
        assert (o - outs[0]).abs().max().item() <= 2e-2
    with pytest.raises(dlm.DlmError) as e:
        dlm.dlm_selftest_set_attn_team_max(dev.ctx, 0)
    assert e.value.code == dlm.DLM_ERR_SHAPE
    with pytest.raises(dlm.DlmError) as e:
        dlm.dlm_selftest_set_attn_team_max(dev.ctx, 4, 2)
    assert e.value.code == dlm.DLM_ERR_SHAPE


def test_team_schedule_repeated_launches_leave_the_counters_clean(dev, oracle):
    """The team's arrival and departure counters are cleared by the last warp to leave: many launches in a row on
    the same units (also of different team sizes) stay correct, and so does a split-schedule call afterwards."""
    shape = dict(NL=1, B=1, Hq=28, Hkv=4, D=128, Lcap=2200, q_cap=32)
    try:
        for i, tmax in enumerate((1 << 20, 5, 1 << 20, 2, 9)):
            dlm.dlm_selftest_set_attn_team_max(dev.ctx, tmax, force=True)
            assert _schedule(dev, nl=1, **shape)["team"] > 1
            _case(dev, oracle, cache_len=[1500 + 100 * i], seed=300 + i, **shape)
    finally:
        dlm.dlm_selftest_set_attn_team_max(dev.ctx, 1 << 20)
    _case(dev, oracle, 2, 2, 28, 4, 128, 1400, 32, [1368, 900], [32, 17], seed=77)


def test_team_schedule_gives_up_cleanly_when_its_waits_may_not_wait(dev, oracle):
    """The give-up path under the team schedule: with the wait limit at 0 every wait, the one for the team's other
    blocks included, gives up at once.  The kernel ends normally with DLM_ERR_TIMEOUT, reading the status clears
    the half-counted team counters, and the next call is correct."""
    shape = dict(NL=1, B=1, Hq=28, Hkv=4, D=128, Lcap=2200, q_cap=32)
    assert _schedule(dev, nl=1, **shape)["team"] > 1
    dlm.dlm_selftest_set_wait_limit(dev.ctx, 0)
    try:
        ck, cv = make_cache(1, 1, 4, 2200, 128, 1, device="cuda")
        q, kn, vn = make_attn_inputs(1, 1, 28, 4, 32, 128, 2, device="cuda")
        gpu_attn_step(dev, ck, cv, _i32([2048]), q, kn, vn)
        torch.cuda.synchronize()
        assert dev.status() == dlm.DLM_ERR_TIMEOUT
    finally:
        dlm.dlm_selftest_set_wait_limit(dev.ctx, 2_000_000_000)
    assert dev.status() == 0
    _case(dev, oracle, cache_len=[2048], seed=99, **shape)
