"""Pins of the oracle's LSTM gradient program (Section 4.2 applied to the recursion over time): central
finite differences on every partial, the single-step closed form, the zero-recurrence special case that
reduces to the dense gradient group, linearity in the upstream partials, and the bias / input identities."""
import numpy as np
import pytest

import oracle

F64 = oracle.F64


def inputs(T, B, In, H, seed, scale=0.5):
    r = np.random.default_rng(seed)
    return dict(x=r.normal(0, 1, (T, B, In)), w_ih=r.normal(0, scale, (In, 4 * H)), w_hh=r.normal(0, scale, (H, 4 * H)),
                b=r.normal(0, 0.3, (4 * H,)), h0=r.normal(0, 0.5, (B, H)), c0=r.normal(0, 0.5, (B, H))), r


def scalar(p, dh_all, dc_fin):
    h_all, c = oracle.lstm_cell_seq(p["x"], p["w_ih"], p["w_hh"], p["b"], p["h0"], p["c0"], rec_dtype=F64, state_dtype=F64)
    return float((dh_all * h_all).sum() + (dc_fin * c).sum())


def grads(p, dh_all, dc_fin, **kw):
    kw = dict(dict(rec_dtype=F64, state_dtype=F64, dz_dtype=F64), **kw)
    out = oracle.lstm_cell_seq_grad(p["x"], p["w_ih"], p["w_hh"], p["b"], p["h0"], p["c0"], dh_all, dc_fin, **kw)
    return dict(zip(("x", "w_ih", "w_hh", "b", "h0", "c0"), out))


@pytest.mark.parametrize("T,B,In,H", [(1, 2, 3, 2), (3, 2, 3, 2), (4, 1, 2, 3)])
def test_every_partial_matches_central_finite_differences(T, B, In, H):
    p, r = inputs(T, B, In, H, 100 + T)
    dh_all, dc_fin = r.normal(0, 1, (T, B, H)), r.normal(0, 1, (B, H))
    g = grads(p, dh_all, dc_fin)
    h = 1e-6
    for name in ("x", "w_ih", "w_hh", "b", "h0", "c0"):
        fd = np.zeros_like(p[name])
        it = np.nditer(p[name], flags=["multi_index"])
        for _ in it:
            k = it.multi_index
            keep = p[name][k]
            p[name][k] = keep + h; up = scalar(p, dh_all, dc_fin)
            p[name][k] = keep - h; dn = scalar(p, dh_all, dc_fin)
            p[name][k] = keep
            fd[k] = (up - dn) / (2 * h)
        np.testing.assert_allclose(g[name], fd, rtol=2e-6, atol=2e-8, err_msg=name)


def test_single_step_closed_form():
    p, r = inputs(1, 3, 4, 2, 7)
    dh_all, dc_fin = r.normal(0, 1, (1, 3, 2)), r.normal(0, 1, (3, 2))
    g = grads(p, dh_all, dc_fin)
    H = 2
    z = p["x"][0] @ p["w_ih"] + p["h0"] @ p["w_hh"] + p["b"]
    sg = lambda v: 1 / (1 + np.exp(-v))
    i, f, gg, o = sg(z[:, :H]), sg(z[:, H:2 * H]), np.tanh(z[:, 2 * H:3 * H]), sg(z[:, 3 * H:])
    c = f * p["c0"] + i * gg
    dh = dh_all[0]
    dc = dc_fin + dh * o * (1 - np.tanh(c) ** 2)
    dz = np.concatenate([dc * gg * i * (1 - i), dc * p["c0"] * f * (1 - f), dc * i * (1 - gg ** 2), dh * np.tanh(c) * o * (1 - o)], axis=1)
    np.testing.assert_allclose(g["x"][0], dz @ p["w_ih"].T, rtol=1e-12)
    np.testing.assert_allclose(g["w_ih"], p["x"][0].T @ dz, rtol=1e-12)
    np.testing.assert_allclose(g["w_hh"], p["h0"].T @ dz, rtol=1e-12)
    np.testing.assert_allclose(g["b"], dz.sum(axis=0), rtol=1e-12)
    np.testing.assert_allclose(g["h0"], dz @ p["w_hh"].T, rtol=1e-12)
    np.testing.assert_allclose(g["c0"], dc * f, rtol=1e-12)


def test_zero_recurrent_weights_and_no_cell_carry_reduce_to_the_dense_gradient_group():
    """With W_hh = 0 and only the o-gate path alive (dc_final = 0, c0 = 0 and f's path removed by looking at
    the partial with respect to the o-gate columns), dz_o = dh tanh(c) o (1 - o): the dense anchor's sigmoid
    gradient group applied to the o columns, whose dW and db the dense oracle gives independently."""
    T, B, In, H = 1, 5, 4, 3
    p, r = inputs(T, B, In, H, 31)
    p["w_hh"][:] = 0.0
    p["c0"][:] = 0.0
    dh_all = r.normal(0, 1, (T, B, H))
    g = grads(p, dh_all, np.zeros((B, H)))
    _, c = oracle.lstm_cell_seq(p["x"], p["w_ih"], p["w_hh"], p["b"], p["h0"], p["c0"], rec_dtype=F64, state_dtype=F64)
    wo, bo = p["w_ih"][:, 3 * H:], p["b"][3 * H:]
    o = oracle.dense_act(p["x"][0], wo, bo, oracle.ACT_SIGMOID, F64)
    _, dwo, dbo = oracle.dense_act_grad(p["x"][0], wo, o, dh_all[0] * np.tanh(c), oracle.ACT_SIGMOID, F64, F64, F64, want_dx=False)
    np.testing.assert_allclose(g["w_ih"][:, 3 * H:], dwo, rtol=1e-12)
    np.testing.assert_allclose(g["b"][3 * H:], dbo, rtol=1e-12)
    np.testing.assert_allclose(g["h0"], 0.0, atol=0)                     # h0 reaches nothing when W_hh = 0


def test_linear_in_the_upstream_partials_and_zero_for_zero():
    p, r = inputs(3, 2, 3, 2, 55)
    a, bq = r.normal(0, 1, (3, 2, 2)), r.normal(0, 1, (2, 2))
    a2, b2 = r.normal(0, 1, (3, 2, 2)), r.normal(0, 1, (2, 2))
    g1, g2, g12 = grads(p, a, bq), grads(p, a2, b2), grads(p, 2 * a - a2, 2 * bq - b2)
    for k in g1:
        np.testing.assert_allclose(g12[k], 2 * g1[k] - g2[k], rtol=1e-10, atol=1e-12)
    g0 = grads(p, np.zeros_like(a), None)
    assert all(not v.any() for v in g0.values())


def test_rounded_operands_change_little_and_dz_rounding_is_applied():
    p, r = inputs(4, 3, 8, 8, 77, scale=0.2)
    p = {k: oracle.cast_array(v, oracle.BF16) if k in ("x", "w_ih", "w_hh") else oracle.cast_array(v, oracle.F32) for k, v in p.items()}
    dh_all = r.normal(0, 1, (4, 3, 8))
    exact = grads(p, dh_all, None)
    rounded = grads(p, dh_all, None, rec_dtype=oracle.BF16, state_dtype=oracle.F32, dz_dtype=oracle.BF16)
    for k in exact:
        rms = np.sqrt(np.mean(exact[k] ** 2))
        assert np.max(np.abs(exact[k] - rounded[k])) < 2e-2 * rms, k       # bf16 effects only
        assert np.max(np.abs(exact[k] - rounded[k])) > 0, k                # but the casts are really applied
    # T = 1, dz in bf16: db is a sum of bf16 values
    one = grads({**p, "x": p["x"][:1]}, dh_all[:1], None, dz_dtype=oracle.BF16)
    full = grads({**p, "x": p["x"][:1]}, dh_all[:1], None)
    assert np.max(np.abs(one["b"] - full["b"])) <= 3 * 2.0 ** -9 * np.max(np.abs(full["b"])) + 1e-12
