"""Pins for the oracle's projections either side of the attention step (Table 1 rows "Q/K/V projection" and "output
projection"): a float64 library matmul with the layout written as an einsum, and closed forms that fix which output
feature lands in which head."""
import numpy as np
import pytest


def _rand(shape, seed, scale=1.0):
    return (np.random.default_rng(seed).standard_normal(shape) * scale).astype(np.float32)


@pytest.mark.parametrize("B,q_cap,dm,Hq,Hkv,D,with_bias", [(2, 5, 24, 4, 2, 8, True), (1, 3, 16, 2, 2, 4, False), (3, 7, 40, 6, 1, 16, True)])
def test_qkv_projection_against_float64_matmul(oracle, B, q_cap, dm, Hq, Hkv, D, with_bias):
    x, w = _rand((B, q_cap, dm), 1), _rand(((Hq + 2 * Hkv) * D, dm), 2, dm ** -0.5)
    bias = _rand(((Hq + 2 * Hkv) * D,), 3) if with_bias else None
    q, k, v = oracle.qkv_project(x, w, bias, Hq, Hkv, D)
    y = np.einsum("bic,nc->bin", x.astype(np.float64), w.astype(np.float64)) + (0 if bias is None else bias.astype(np.float64))
    heads = y.reshape(B, q_cap, Hq + 2 * Hkv, D).transpose(0, 2, 1, 3)           # [B, head, i, d]
    np.testing.assert_allclose(q, heads[:, :Hq], rtol=1e-6, atol=1e-6)
    np.testing.assert_allclose(k, heads[:, Hq:Hq + Hkv], rtol=1e-6, atol=1e-6)
    np.testing.assert_allclose(v, heads[:, Hq + Hkv:], rtol=1e-6, atol=1e-6)


def test_qkv_projection_closed_forms(oracle):
    B, q_cap, Hq, Hkv, D = 2, 3, 2, 1, 4
    dm = (Hq + 2 * Hkv) * D
    x = _rand((B, q_cap, dm), 5)
    # identity weights: output feature n is input feature n, so head h holds input columns [h D, (h + 1) D)
    q, k, v = oracle.qkv_project(x, np.eye(dm, dtype=np.float32), None, Hq, Hkv, D)
    for h in range(Hq):
        np.testing.assert_array_equal(q[:, h], x[:, :, h * D:(h + 1) * D])
    np.testing.assert_array_equal(k[:, 0], x[:, :, Hq * D:(Hq + 1) * D])
    np.testing.assert_array_equal(v[:, 0], x[:, :, (Hq + 1) * D:])
    # zero input: the bias alone, broadcast over batch and rows
    bias = np.arange(dm, dtype=np.float32)
    q, k, v = oracle.qkv_project(np.zeros_like(x), _rand((dm, dm), 6), bias, Hq, Hkv, D)
    assert np.all(q[1, 1, 2] == bias[D:2 * D]) and np.all(k[0, 0, 0] == bias[2 * D:3 * D]) and np.all(v[1, 0, 2] == bias[3 * D:])
    # a weight matrix with a single one picks one input column into one (head, d)
    w = np.zeros((dm, dm), np.float32); w[1 * D + 2, 7] = 1.0
    q, k, v = oracle.qkv_project(x, w, None, Hq, Hkv, D)
    np.testing.assert_array_equal(q[:, 1, :, 2], x[:, :, 7])
    assert np.count_nonzero(q) == np.count_nonzero(x[:, :, 7]) and not k.any() and not v.any()


@pytest.mark.parametrize("B,q_cap,dm,Hq,D,with_bias", [(2, 5, 24, 3, 8, True), (1, 4, 12, 2, 4, False)])
def test_out_projection_against_float64_matmul(oracle, B, q_cap, dm, Hq, D, with_bias):
    o, wo = _rand((B, Hq, q_cap, D), 7), _rand((dm, Hq * D), 8, (Hq * D) ** -0.5)
    bias = _rand((dm,), 9) if with_bias else None
    y = oracle.out_project(o, wo, bias)
    flat = o.transpose(0, 2, 1, 3).reshape(B, q_cap, Hq * D).astype(np.float64)     # features ordered (head, d)
    ref = flat @ wo.astype(np.float64).T + (0 if bias is None else bias.astype(np.float64))
    np.testing.assert_allclose(y, ref, rtol=1e-6, atol=1e-6)
    # the two projections compose to the plain product when the middle is the identity: y = x Wq^T Wo^T
    x, wq = _rand((B, q_cap, dm), 10), _rand((Hq * D, dm), 11, dm ** -0.5)
    wfull = np.concatenate([wq, np.zeros((2 * D, dm), np.float32)])
    q, _, _ = oracle.qkv_project(x, wfull, None, Hq, 1, D)
    y2 = oracle.out_project(q, wo, None)
    np.testing.assert_allclose(y2, (x.astype(np.float64) @ wq.astype(np.float64).T) @ wo.astype(np.float64).T, rtol=2e-5, atol=2e-5)
