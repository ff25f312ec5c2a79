"""Pins for the oracle's dense / conv2d anchors, their gradient groups and the LSTM sequence.

Forward definitions are tied to NumPy library routines and to special cases with known
answers; every gradient group is tied to central finite differences of the FORWARD oracle
(paper Section 4.2: the partials of the final scalar) and to adjoint identities."""
import itertools

import numpy as np
import pytest

import oracle
from relay_workloads import inputs as I
from relay_workloads import program as P

F64 = 5
ACTS = (oracle.ACT_NONE, oracle.ACT_RELU, oracle.ACT_TANH, oracle.ACT_SIGMOID)


def _np_act(z, a):
    return {0: z, 1: np.maximum(z, 0), 2: np.tanh(z), 3: 1 / (1 + np.exp(-z))}[a]


# ---------------------------------------------------------------------------------------------
# dense forward
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("act", ACTS)
def test_dense_against_numpy_matmul(act):
    rng = np.random.default_rng(10)
    x, w, b = rng.standard_normal((7, 13)), rng.standard_normal((13, 5)), rng.standard_normal(5)
    got = oracle.dense_act(x, w, b, act, F64)
    np.testing.assert_allclose(got, _np_act(x @ w + b, act), rtol=1e-13, atol=1e-14)
    nob = oracle.dense_act(x, w, None, act, F64)
    np.testing.assert_allclose(nob, _np_act(x @ w, act), rtol=1e-13, atol=1e-14)


def test_dense_special_cases():
    rng = np.random.default_rng(11)
    x, b = rng.standard_normal((4, 6)), rng.standard_normal(6)
    # W = I  ->  y = act(x + b)
    np.testing.assert_allclose(oracle.dense_act(x, np.eye(6), b, oracle.ACT_TANH, F64), np.tanh(x + b), rtol=1e-15)
    # one-hot rows of x pick rows of W (catches a transposed operand: W is not symmetric/square)
    w = rng.standard_normal((6, 3))
    onehot = np.eye(6)[[4, 0, 2]]
    assert np.array_equal(oracle.dense_act(onehot, w, None, oracle.ACT_NONE, F64), w[[4, 0, 2]])
    # relu output is >= 0 and exactly 0 where z < 0
    y = oracle.dense_act(x, rng.standard_normal((6, 9)), None, oracle.ACT_RELU, F64)
    assert np.all(y >= 0) and np.any(y == 0)


def test_dense_output_is_stored_in_declared_dtype():
    rng = np.random.default_rng(12)
    x, w = rng.standard_normal((3, 8)), rng.standard_normal((8, 4))
    y64 = oracle.dense_act(x, w, None, oracle.ACT_NONE, F64)
    assert np.array_equal(oracle.dense_act(x, w, None, oracle.ACT_NONE, oracle.BF16), oracle.cast_array(y64, oracle.BF16))
    assert np.array_equal(oracle.dense_act(x, w, None, oracle.ACT_NONE, oracle.F32), y64.astype(np.float32).astype(np.float64))


# ---------------------------------------------------------------------------------------------
# dense gradient group
# ---------------------------------------------------------------------------------------------
def _fd_check(loss, params, grads, h=1e-5, skip=None, tol=1e-7):
    for name in params:
        arr, g = params[name], grads[name]
        for idx in np.ndindex(arr.shape):
            if skip is not None and skip(name, idx):
                continue
            keep = arr[idx]
            arr[idx] = keep + h; lp = loss()
            arr[idx] = keep - h; lm = loss()
            arr[idx] = keep
            fd = (lp - lm) / (2 * h)
            assert abs(fd - g[idx]) <= tol * max(1.0, abs(fd)), (name, idx, fd, g[idx])


@pytest.mark.parametrize("act", ACTS)
def test_dense_grad_finite_differences_every_element_tiny_mlp(act):
    """Configuration 1 in full: x[8,64] W[64,32] b[32] dy[8,32], every element of dx, dW, db."""
    t = I.cfg1_tiny_mlp()
    x, w, b, dy = (I.as_f64(t[k]).copy() for k in ("x", "w", "b", "dy"))
    y = oracle.dense_act(x, w, b, act, F64)
    dx, dw, db = oracle.dense_act_grad(x, w, y, dy, act, F64, F64, F64)
    z = x @ w + b
    if act == oracle.ACT_RELU:
        assert np.min(np.abs(z)) > 1e-3  # no element sits on the kink for this seed

    def loss():
        return float(np.sum(dy * oracle.dense_act(x, w, b, act, F64)))

    _fd_check(loss, dict(x=x, w=w, b=b), dict(x=dx, w=dw, b=db))


def test_dense_grad_randomised_shapes_property():
    rng = np.random.default_rng(13)
    for trial in range(6):
        M, K, N = (int(v) for v in rng.integers(1, 7, 3))
        act = ACTS[trial % 4]
        x, w, b, dy = rng.standard_normal((M, K)), rng.standard_normal((K, N)), rng.standard_normal(N), rng.standard_normal((M, N))
        y = oracle.dense_act(x, w, b, act, F64)
        dx, dw, db = oracle.dense_act_grad(x, w, y, dy, act, F64, F64, F64)
        z = x @ w + b

        def loss():
            return float(np.sum(dy * oracle.dense_act(x, w, b, act, F64)))

        if act == oracle.ACT_RELU and np.min(np.abs(z)) < 1e-3:
            continue
        _fd_check(loss, dict(x=x, w=w, b=b), dict(x=dx, w=dw, b=db))


def test_dense_grad_adjoint_identities_and_optional_outputs():
    rng = np.random.default_rng(14)
    M, K, N = 9, 11, 6
    x, w, dy = rng.standard_normal((M, K)), rng.standard_normal((K, N)), rng.standard_normal((M, N))
    y = oracle.dense_act(x, w, None, oracle.ACT_NONE, F64)
    dx, dw, db = oracle.dense_act_grad(x, w, y, dy, oracle.ACT_NONE, F64, F64, F64)
    u, v = rng.standard_normal((M, K)), rng.standard_normal((K, N))
    # <dZ, U W> = <dZ W^T, U>,  <dZ, X V> = <X^T dZ, V>,  db = 1^T dZ
    assert abs(np.sum(dy * (u @ w)) - np.sum(dx * u)) < 1e-11
    assert abs(np.sum(dy * (x @ v)) - np.sum(dw * v)) < 1e-11
    np.testing.assert_allclose(db, dy.sum(0), rtol=1e-14)
    only_dw = oracle.dense_act_grad(x, w, y, dy, oracle.ACT_NONE, F64, F64, F64, want_dx=False, want_db=False)
    assert only_dw[0] is None and only_dw[2] is None and np.array_equal(only_dw[1], dw)


def test_dense_grad_uses_saved_output_for_mask():
    # the relu mask comes from the saved y passed in: y = 0 exactly -> no gradient flows
    x, w = np.ones((2, 2)), np.ones((2, 2))
    y = np.array([[0.0, 2.0], [2.0, 0.0]])
    dy = np.ones((2, 2))
    dx, dw, db = oracle.dense_act_grad(x, w, y, dy, oracle.ACT_RELU, F64, F64, F64)
    assert db.tolist() == [1.0, 1.0] and np.array_equal(dw, np.ones((2, 2)))
    assert np.array_equal(dx, np.ones((2, 2)))


# ---------------------------------------------------------------------------------------------
# conv2d forward
# ---------------------------------------------------------------------------------------------
def test_conv_output_extent_counts_window_positions():
    for n, k, p, s in itertools.product(range(1, 7), range(1, 7), range(0, 4), range(1, 4)):
        if n + 2 * p < k:
            assert oracle.conv2d_out_extent(n, k, s, p) is None
            continue
        count = sum(1 for start in range(-p, n + p - k + 1, s))  # window starts that fit
        assert oracle.conv2d_out_extent(n, k, s, p) == count


def _im2col(x, R, S, stride, pad):
    Nb, C, H, W = x.shape
    P_ = (H + 2 * pad - R) // stride + 1
    Q_ = (W + 2 * pad - S) // stride + 1
    xp = np.zeros((Nb, C, H + 2 * pad, W + 2 * pad))
    xp[:, :, pad:pad + H, pad:pad + W] = x
    cols = np.empty((Nb * P_ * Q_, C * R * S))
    row = 0
    for n in range(Nb):
        for p in range(P_):
            for q in range(Q_):
                cols[row] = xp[n, :, p * stride:p * stride + R, q * stride:q * stride + S].reshape(-1)
                row += 1
    return cols, P_, Q_


@pytest.mark.parametrize("stride,pad,R,S", [(1, 1, 3, 3), (2, 1, 3, 3), (1, 0, 5, 5), (2, 2, 3, 5), (1, 0, 1, 1)])
def test_conv_equals_im2col_then_dense(stride, pad, R, S):
    """Second, independent route: explicit patch matrix, then the (separately pinned) dense."""
    rng = np.random.default_rng(15)
    Nb, C, H, W, O = 2, 3, 7, 6, 4
    x, wt, b = rng.standard_normal((Nb, C, H, W)), rng.standard_normal((O, C, R, S)), rng.standard_normal(O)
    y = oracle.conv2d_act(x, wt, b, stride, pad, oracle.ACT_TANH, F64)
    cols, P_, Q_ = _im2col(x, R, S, stride, pad)
    yd = oracle.dense_act(cols, wt.reshape(O, -1).T.copy(), b, oracle.ACT_TANH, F64)
    want = yd.reshape(Nb, P_, Q_, O).transpose(0, 3, 1, 2)
    assert y.shape == want.shape
    np.testing.assert_allclose(y, want, rtol=1e-13, atol=1e-14)


def test_conv_delta_image_returns_flipped_taps():
    # cross-correlation of a unit impulse: y[o, p, q] = Wt[o, 0, i0-p+1, j0-q+1] (taps mirrored)
    wt = np.arange(2 * 1 * 3 * 3, dtype=np.float64).reshape(2, 1, 3, 3) + 1
    x = np.zeros((1, 1, 5, 5)); x[0, 0, 2, 2] = 1.0
    y = oracle.conv2d_act(x, wt, None, 1, 1, oracle.ACT_NONE, F64)
    for o in range(2):
        assert np.array_equal(y[0, o, 1:4, 1:4], wt[o, 0, ::-1, ::-1])
    assert y[0, :, 0, :].sum() == 0 and y[0, :, :, 0].sum() == 0


def test_conv_centre_tap_is_dense_over_channels_and_1x1_image():
    rng = np.random.default_rng(16)
    Nb, C, H, W, O = 2, 5, 4, 3, 6
    x = rng.standard_normal((Nb, C, H, W))
    wt = np.zeros((O, C, 3, 3)); wc = rng.standard_normal((O, C)); wt[:, :, 1, 1] = wc
    y = oracle.conv2d_act(x, wt, None, 1, 1, oracle.ACT_NONE, F64)
    np.testing.assert_allclose(y, np.einsum("oc,nchw->nohw", wc, x), rtol=1e-13, atol=1e-14)
    # H = W = 1 with pad 1: only the centre tap touches data
    wfull = rng.standard_normal((O, C, 3, 3)); x1 = rng.standard_normal((1, C, 1, 1))
    y1 = oracle.conv2d_act(x1, wfull, None, 1, 1, oracle.ACT_NONE, F64)
    np.testing.assert_allclose(y1[0, :, 0, 0], wfull[:, :, 1, 1] @ x1[0, :, 0, 0], rtol=1e-13)


# ---------------------------------------------------------------------------------------------
# conv2d gradient group
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("stride,pad,act", [(1, 1, oracle.ACT_RELU), (2, 1, oracle.ACT_TANH), (1, 0, oracle.ACT_NONE), (2, 0, oracle.ACT_SIGMOID)])
def test_conv_grad_finite_differences(stride, pad, act):
    rng = np.random.default_rng(17)
    Nb, C, H, W, O, R, S = 2, 2, 5, 4, 3, 3, 3
    x, wt, b = rng.standard_normal((Nb, C, H, W)), rng.standard_normal((O, C, R, S)) * 0.5, rng.standard_normal(O)
    y = oracle.conv2d_act(x, wt, b, stride, pad, act, F64)
    dy = rng.standard_normal(y.shape)
    dx, dw, db = oracle.conv2d_act_grad(x, wt, y, dy, stride, pad, act, F64, F64, F64)
    if act == oracle.ACT_RELU:
        z = oracle.conv2d_act(x, wt, b, stride, pad, oracle.ACT_NONE, F64)
        assert np.min(np.abs(z)) > 1e-3

    def loss():
        return float(np.sum(dy * oracle.conv2d_act(x, wt, b, stride, pad, act, F64)))

    _fd_check(loss, dict(x=x, w=wt, b=b), dict(x=dx, w=dw, b=db))


def test_conv_grad_adjoint_identities():
    rng = np.random.default_rng(18)
    Nb, C, H, W, O = 2, 3, 6, 5, 4
    x, wt = rng.standard_normal((Nb, C, H, W)), rng.standard_normal((O, C, 3, 3))
    y = oracle.conv2d_act(x, wt, None, 1, 1, oracle.ACT_NONE, F64)
    dz = rng.standard_normal(y.shape)
    dx, dw, db = oracle.conv2d_act_grad(x, wt, y, dz, 1, 1, oracle.ACT_NONE, F64, F64, F64)
    u, v = rng.standard_normal(x.shape), rng.standard_normal(wt.shape)
    assert abs(np.sum(dz * oracle.conv2d_act(u, wt, None, 1, 1, 0, F64)) - np.sum(dx * u)) < 1e-10
    assert abs(np.sum(dz * oracle.conv2d_act(x, v, None, 1, 1, 0, F64)) - np.sum(dw * v)) < 1e-10
    np.testing.assert_allclose(db, dz.sum((0, 2, 3)), rtol=1e-13)


# ---------------------------------------------------------------------------------------------
# LSTM over a sequence
# ---------------------------------------------------------------------------------------------
def _lstm_inputs(T, B, In, H, seed, scale=0.5):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((T, B, In)), rng.uniform(-scale, scale, (In, 4 * H)),
            rng.uniform(-scale, scale, (H, 4 * H)), rng.uniform(-scale, scale, 4 * H))


def test_lstm_single_step_closed_form():
    T, B, In, H = 1, 3, 5, 4
    x, wi, wh, b = _lstm_inputs(T, B, In, H, 19)
    z0 = np.zeros((B, H))
    h_all, c = oracle.lstm_cell_seq(x, wi, wh, b, z0, z0, rec_dtype=F64, state_dtype=F64)
    z = x[0] @ wi + b
    sg = lambda v: 1 / (1 + np.exp(-v))
    i, g, o = sg(z[:, :H]), np.tanh(z[:, 2 * H:3 * H]), sg(z[:, 3 * H:])
    np.testing.assert_allclose(c, i * g, rtol=1e-13)           # c0 = 0 kills the forget term
    np.testing.assert_allclose(h_all[0], o * np.tanh(i * g), rtol=1e-13)


def test_lstm_is_composition_of_dense_and_ewise_groups():
    """Monolithic loop == per-step composition of the oracle's dense anchor and an elementwise
    program (two routes through separately pinned pieces), including the bf16 cast of h."""
    T, B, In, H = 4, 3, 6, 5
    x, wi, wh, b = _lstm_inputs(T, B, In, H, 20)
    x, wi, wh = (oracle.cast_array(v, oracle.BF16) for v in (x, wi, wh))
    rng = np.random.default_rng(21)
    h0 = oracle.cast_array(rng.standard_normal((B, H)) * 0.3, oracle.F32)
    c0 = oracle.cast_array(rng.standard_normal((B, H)) * 0.3, oracle.F32)
    h_all, c_fin = oracle.lstm_cell_seq(x, wi, wh, b, h0, c0)

    p = P.Program([F64] * 5)   # zi, zf, zg, zo, c
    i_, f_, g_, o_ = p.sigmoid(0), p.sigmoid(1), p.tanh(2), p.sigmoid(3)
    cn = p.cast(p.add(p.mul(f_, 4), p.mul(i_, g_)), P.F32)
    hn = p.cast(p.mul(o_, p.tanh(cn)), P.F32)
    h, c = h0, c0
    for t in range(T):
        hq = oracle.cast_array(h, oracle.BF16)
        z = oracle.dense_act(np.concatenate([x[t], hq], 1), np.concatenate([wi, wh], 0), b, oracle.ACT_NONE, F64)
        c, h = oracle.ewise(p.arrays(), [z[:, :H], z[:, H:2 * H], z[:, 2 * H:3 * H], z[:, 3 * H:], c], [cn, hn])
        np.testing.assert_allclose(h_all[t], h, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(c_fin, c, rtol=1e-12, atol=1e-14)
    assert np.array_equal(h_all, h_all.astype(np.float32).astype(np.float64))   # stored as fp32


def test_lstm_zero_recurrent_weights_make_steps_independent():
    T, B, In, H = 5, 2, 4, 3
    x, wi, wh, b = _lstm_inputs(T, B, In, H, 22)
    z0 = np.zeros((B, H))
    h_all, _ = oracle.lstm_cell_seq(x, wi, 0 * wh, b, z0, z0, rec_dtype=F64, state_dtype=F64)
    # the output gate of step t depends on x_t only: h_t / tanh(c_t) = sigmoid(z_o(x_t))
    perm = [3, 1, 4, 0, 2]
    h_perm, _ = oracle.lstm_cell_seq(x[perm], wi, 0 * wh, b, z0, z0, rec_dtype=F64, state_dtype=F64)
    sg = lambda v: 1 / (1 + np.exp(-v))
    # first step has no history at all, so it must agree wherever it is placed first
    first, _ = oracle.lstm_cell_seq(x[perm][:1], wi, 0 * wh, b, z0, z0, rec_dtype=F64, state_dtype=F64)
    np.testing.assert_allclose(h_perm[0], first[0], rtol=1e-14)
    assert not np.allclose(h_all[1], h_perm[1])                 # c still carries history
    assert np.all(np.abs(h_all) < 1)


def test_lstm_recurrence_matters_and_invariants():
    T, B, In, H = 12, 2, 4, 6
    x, wi, wh, b = _lstm_inputs(T, B, In, H, 23, scale=1.0)
    z0 = np.zeros((B, H))
    h_all, c_fin = oracle.lstm_cell_seq(x, wi, wh, b, z0, z0)
    h_norec, _ = oracle.lstm_cell_seq(x, wi, 0 * wh, b, z0, z0)
    assert np.array_equal(h_all[0], h_norec[0]) and not np.allclose(h_all[1:], h_norec[1:])
    assert np.all(np.abs(h_all) < 1) and np.all(np.abs(c_fin) <= T)
    # batch rows are independent: running one row alone gives the same row
    h_row, c_row = oracle.lstm_cell_seq(x[:, 1:2], wi, wh, b, z0[1:2], z0[1:2])
    assert np.array_equal(h_row[:, 0], h_all[:, 1]) and np.array_equal(c_row[0], c_fin[1])
