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


# ------------------------------------------------------------------------------------------ rotary embedding
def _angles(B, q_cap, D, seed):
    th = np.random.default_rng(seed).uniform(-np.pi, np.pi, (B, q_cap, D // 2))
    return np.cos(th).astype(np.float32), np.sin(th).astype(np.float32)


def _parse_rope_fixture():
    import os
    rows, cur = [], {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "rope_handworked.txt")) as f:
        for line in f:
            line = line.split("#")[0].split()
            if not line:
                continue
            cur[line[0]] = np.array([float(t) for t in line[1:]])
            if line[0] == "v":
                rows.append(cur)
                cur = {}
    return rows


def test_rope_handworked_fixture(oracle):
    rows = _parse_rope_fixture()
    assert len(rows) == 2
    x = np.stack([r["x"] for r in rows]).astype(np.float32)[None]           # [1, 2 rows, 12]
    th = np.deg2rad(np.stack([r["angles"] for r in rows]))[None]            # [1, 2, 2]
    q, k, v = oracle.qkv_project_rope(x, np.eye(12, dtype=np.float32), None, np.cos(th).astype(np.float32),
                                      np.sin(th).astype(np.float32), 1, 1, 4)
    for i, r in enumerate(rows):
        np.testing.assert_allclose(q[0, 0, i], r["q"], atol=1e-6)
        np.testing.assert_allclose(k[0, 0, i], r["k"], atol=1e-6)
        np.testing.assert_array_equal(v[0, 0, i], r["v"])


def test_rope_zero_angle_is_the_plain_projection_and_values_are_never_rotated(oracle):
    B, q_cap, dm, Hq, Hkv, D = 2, 5, 24, 3, 2, 8
    x, w, bias = _rand((B, q_cap, dm), 21), _rand(((Hq + 2 * Hkv) * D, dm), 22, dm ** -0.5), _rand(((Hq + 2 * Hkv) * D,), 23)
    q0, k0, v0 = oracle.qkv_project(x, w, bias, Hq, Hkv, D)
    ones, zeros = np.ones((B, q_cap, D // 2), np.float32), np.zeros((B, q_cap, D // 2), np.float32)
    q, k, v = oracle.qkv_project_rope(x, w, bias, ones, zeros, Hq, Hkv, D)
    np.testing.assert_array_equal(q, q0); np.testing.assert_array_equal(k, k0); np.testing.assert_array_equal(v, v0)
    cs, sn = _angles(B, q_cap, D, 24)
    q, k, v = oracle.qkv_project_rope(x, w, bias, cs, sn, Hq, Hkv, D)
    np.testing.assert_array_equal(v, v0)
    assert np.abs(q - q0).max() > 0.1 and np.abs(k - k0).max() > 0.1


def test_rope_is_a_rotation_of_each_pair(oracle):
    """Each pair (d, d + D/2) keeps its length, and turning by theta then by -theta (a second projection with identity
    weights) gives the input back: a wrong sign in either formula or a wrong pairing breaks one of the two."""
    B, q_cap, dm, Hq, Hkv, D = 1, 6, 16, 2, 1, 8
    x, w = _rand((B, q_cap, dm), 31), _rand(((Hq + 2 * Hkv) * D, dm), 32, dm ** -0.5)
    cs, sn = _angles(B, q_cap, D, 33)
    q0, k0, _ = oracle.qkv_project(x, w, None, Hq, Hkv, D)
    q, k, _ = oracle.qkv_project_rope(x, w, None, cs, sn, Hq, Hkv, D)
    h = D // 2
    for a, a0 in ((q, q0), (k, k0)):
        np.testing.assert_allclose(a[..., :h] ** 2 + a[..., h:] ** 2, a0[..., :h] ** 2 + a0[..., h:] ** 2, rtol=1e-5, atol=1e-6)
    # back-rotation: feed the rotated query head 0 through an identity projection with the opposite angles
    n = 3 * D
    xin = np.zeros((B, q_cap, n), np.float32); xin[..., :D] = q[:, 0]
    qb, _, _ = oracle.qkv_project_rope(xin, np.eye(n, dtype=np.float32), None, cs, -sn, 1, 1, D)
    np.testing.assert_allclose(qb[:, 0], q0[:, 0], rtol=1e-5, atol=1e-6)


def test_rope_scores_depend_on_the_position_difference_only(oracle):
    """The property the embedding exists for: with angles theta_j * position, the dot product of a query at position m
    and a key at position n equals that of the same vectors at positions m - n and 0."""
    D, base = 16, 10000.0
    inv = base ** (-np.arange(D // 2) * 2.0 / D)
    pos = np.array([7, 3, 12, 0, 4])                          # rows: m = 7, n = 3, another pair 12 / 0, and m - n = 4
    th = (pos[:, None] * inv[None, :])[None]
    vq, vk = _rand((D,), 41), _rand((D,), 42)
    x = np.zeros((1, len(pos), 3 * D), np.float32); x[..., :D] = vq; x[..., D:2 * D] = vk
    q, k, _ = oracle.qkv_project_rope(x, np.eye(3 * D, dtype=np.float32), None, np.cos(th).astype(np.float32),
                                      np.sin(th).astype(np.float32), 1, 1, D)
    q, k = q[0, 0].astype(np.float64), k[0, 0].astype(np.float64)
    np.testing.assert_allclose(q[0] @ k[1], q[4] @ k[3], rtol=1e-5, atol=1e-5)      # (7, 3) against (4, 0)
    assert abs(q[0] @ k[1] - q[0] @ k[0]) > 1e-3                                      # and it does depend on the difference
