"""Shared helpers of the GPU parity tests (argument plumbing only)."""
import numpy as np
import torch

import paper_2505_21467_b200 as dlm
from workloads import widen

ATTN_MAX_ERR = 2e-2      # max |err| against the fp32 oracle for unit-scale bf16 inputs
ATTN_MEAN_ERR = 2e-3     # mean |err|
CONF_RTOL = 2e-5         # fp32 confidence: approximate exp and a different summation order


GUARD_BYTES = 512
GUARD_FILL = 0xA5


class Dev:
    """A context plus scratch, created once per test session.  Output tensors handed out by `guarded` sit between
    two guard regions of sentinel bytes inside a larger buffer; `status` (which synchronises) checks that no kernel
    wrote outside its outputs."""

    def __init__(self):
        self.ctx = dlm.dlm_create(0)
        self._ws = {}
        self._guards = []

    def guarded(self, shape, dtype, fill):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        body = (n + 255) // 256 * 256
        buf = torch.full((GUARD_BYTES + body + GUARD_BYTES,), GUARD_FILL, dtype=torch.uint8, device="cuda")
        t = buf[GUARD_BYTES:GUARD_BYTES + n].view(dtype).view(*shape)
        t.fill_(fill)
        self._guards.append((buf, n))
        return t

    def check_guards(self):
        for buf, n in self._guards:
            assert bool((buf[:GUARD_BYTES] == GUARD_FILL).all()), "a kernel wrote before the start of an output"
            assert bool((buf[GUARD_BYTES + n + ((-n) % 256):] == GUARD_FILL).all()) and \
                bool((buf[GUARD_BYTES + n:GUARD_BYTES + n + ((-n) % 256)] == GUARD_FILL).all()), \
                "a kernel wrote past the end of an output"
        self._guards.clear()

    def workspace(self, nbytes):
        nbytes = max(int(nbytes), 256)
        key = 1 << (nbytes - 1).bit_length()
        if key not in self._ws:
            self._ws[key] = torch.empty(key, dtype=torch.uint8, device="cuda")
        return self._ws[key]

    def status(self):
        code = dlm.dlm_get_status(self.ctx)     # synchronises the stream
        self.check_guards()
        return code


def gpu_attn_step(dev, ck, cv, cache_len, q, kn, vn, q_len=None, scale=0.0, layer_begin=0, layer_end=None,
                  want_lse=True, hint=0):
    """ck/cv [NL,B,Hkv,Lcap,D]; q [nl,B,Hq,q_cap,D]; returns (out bf16, lse fp32) CUDA tensors."""
    NL, B, Hkv, Lcap, D = ck.shape
    nl, _, Hq, q_cap, _ = q.shape
    layer_end = NL if layer_end is None else layer_end
    cache = dlm.make_kv_cache(ck, cv, cache_len)
    out = dev.guarded(tuple(q.shape), torch.bfloat16, float("nan"))
    lse = dev.guarded((nl, B, Hq, q_cap), torch.float32, float("nan")) if want_lse else None
    ws = dev.workspace(dlm.dlm_attn_workspace_bytes(dev.ctx, cache, nl, Hq, q_cap))
    dlm.dlm_freecache_attn_step(dev.ctx, cache, layer_begin, layer_end, q, kn, vn, Hq, q_cap, q_len, scale,
                                hint, out, lse, ws)
    return out, lse


def oracle_attn_layers(oracle, ck, cv, cache_len, q, kn, vn, q_len=None, scale=None, layer_begin=0,
                       layers=None):
    """Runs the oracle layer by layer on CPU copies; returns {layer_in_call: (out, lse)}."""
    nl = q.shape[0]
    res = {}
    cl = cache_len.cpu().numpy().astype(np.int32)
    ql = None if q_len is None else q_len.cpu().numpy().astype(np.int32)
    for lc in (range(nl) if layers is None else layers):
        res[lc] = oracle.attn_step(widen(ck[layer_begin + lc]), widen(cv[layer_begin + lc]), cl, widen(q[lc]),
                                   widen(kn[lc]), widen(vn[lc]), ql, scale)
    return res


def assert_attn_close(out_gpu, lse_gpu, ref, lc):
    ref_out, ref_lse = ref
    got = out_gpu[lc].float().cpu().numpy()
    assert np.isfinite(got).all(), "non-finite attention output"
    err = np.abs(got - ref_out)
    assert err.max() <= ATTN_MAX_ERR, f"layer {lc}: max |err| {err.max():.4g}"
    assert err.mean() <= ATTN_MEAN_ERR, f"layer {lc}: mean |err| {err.mean():.4g}"
    if lse_gpu is not None:
        got_lse = lse_gpu[lc].cpu().numpy()
        active = np.isfinite(ref_lse)
        np.testing.assert_array_equal(np.isneginf(got_lse), ~active)
        np.testing.assert_allclose(got_lse[active], ref_lse[active], rtol=0, atol=2e-3)
    return float(err.max()), float(err.mean())


def gpu_unmask(dev, logits, masked, tokens, k):
    """Runs dlm_unmask_select in place on CUDA tensors; returns (tok, conf, sel_idx, n_sel)."""
    B, Lblk, V = logits.shape
    tok = dev.guarded((B, Lblk), torch.int32, -9)
    conf = dev.guarded((B, Lblk), torch.float32, float("nan"))
    sel_idx = dev.guarded((B, max(k, 1)), torch.int32, -9) if k > 0 else None
    n_sel = dev.guarded((B,), torch.int32, -9) if k > 0 else None
    ws = dev.workspace(dlm.dlm_unmask_workspace_bytes(dev.ctx, B, Lblk, V))
    dlm.dlm_unmask_select(dev.ctx, logits, B, Lblk, V, masked, tokens, k, tok, conf, sel_idx, n_sel, ws)
    return tok, conf, sel_idx, n_sel


def topk_margin(conf, masked0, k):
    """Smallest relative gap between the k_eff-th and (k_eff+1)-th largest confidences of any batch
    element, ignoring exact ties (bit-identical rows).  conf: oracle fp32 [B, Lblk]."""
    worst = np.inf
    for b in range(conf.shape[0]):
        c = np.sort(conf[b][masked0[b] != 0].astype(np.float64))[::-1]
        if k < len(c) and c[k - 1] != c[k]:
            worst = min(worst, (c[k - 1] - c[k]) / c[k - 1])
    return worst
