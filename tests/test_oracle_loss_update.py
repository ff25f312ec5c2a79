"""Pins of the oracle's softmax cross-entropy loss, its gradient group and the SGD parameter update
(Fig. 3: relay.softmax_cross_entropy, relay.update_model_params; Section 4.2 for the gradient) against
closed forms, SciPy's log-softmax, invariants and central finite differences."""
import numpy as np
import pytest
from scipy import special

import oracle


def rng_case(seed, B=5, C=7, scale=2.0):
    r = np.random.default_rng(seed)
    z = r.normal(0, scale, (B, C))
    t = r.uniform(0, 1, (B, C))
    return r, z, t


def test_uniform_scores_give_log_of_class_count_times_target_mass():
    for C in (1, 2, 10, 1000):
        z = np.full((3, C), 0.37)
        t = np.zeros((3, C)); t[:, 0] = 1.0; t[2, :] = 0.25     # row 2: mass C/4
        want = np.log(C) * t.sum(axis=1)
        np.testing.assert_allclose(oracle.softmax_xent(z, t), want, rtol=1e-13, atol=1e-15)


def test_two_classes_reduce_to_the_logistic_loss():
    # one-hot target on class 0: loss = log(1 + exp(z1 - z0))
    d = np.linspace(-30, 30, 41)
    z = np.stack([np.zeros_like(d), d], axis=1)
    t = np.tile([1.0, 0.0], (len(d), 1))
    np.testing.assert_allclose(oracle.softmax_xent(z, t), np.logaddexp(0.0, d), rtol=1e-13, atol=1e-15)


def test_against_scipy_log_softmax_and_softmax():
    r, z, t = rng_case(1, B=9, C=33)
    want = -(t * special.log_softmax(z, axis=1)).sum(axis=1)
    np.testing.assert_allclose(oracle.softmax_xent(z, t), want, rtol=1e-13)
    dl = r.normal(0, 1, 9)
    loss, dz = oracle.softmax_xent_grad(z, t, dl)
    np.testing.assert_allclose(loss, want, rtol=1e-13)
    onehot = np.eye(33)[r.integers(0, 33, 9)]
    _, dz1 = oracle.softmax_xent_grad(z, onehot, dl)
    np.testing.assert_allclose(dz1, dl[:, None] * (special.softmax(z, axis=1) - onehot), rtol=1e-12, atol=1e-15)
    assert dz.shape == z.shape


def test_shift_invariance_linearity_in_targets_and_no_overflow():
    r, z, t = rng_case(2)
    l0 = oracle.softmax_xent(z, t)
    np.testing.assert_allclose(oracle.softmax_xent(z + 123.456, t), l0, rtol=1e-11)
    t2 = r.uniform(0, 1, t.shape)
    np.testing.assert_allclose(oracle.softmax_xent(z, 0.3 * t + 2.0 * t2), 0.3 * l0 + 2.0 * oracle.softmax_xent(z, t2), rtol=1e-12)
    big = np.array([[1000.0, 0.0], [-1000.0, 0.0]])
    tt = np.array([[0.0, 1.0], [1.0, 0.0]])
    np.testing.assert_allclose(oracle.softmax_xent(big, tt), [1000.0, 1000.0], rtol=1e-15)
    _, dz = oracle.softmax_xent_grad(big, tt, np.ones(2))
    np.testing.assert_allclose(dz, [[1.0, -1.0], [-1.0, 1.0]], atol=1e-300)


def test_gradient_rows_sum_to_zero_and_match_finite_differences():
    r, z, t = rng_case(3, B=4, C=6, scale=1.5)
    dl = r.normal(0, 1, 4)
    _, dz = oracle.softmax_xent_grad(z, t, dl)
    np.testing.assert_allclose(dz.sum(axis=1), 0.0, atol=1e-14)      # sum_j p_j = 1, whatever the targets
    h = 1e-5
    fd = np.empty_like(z)
    for i in range(z.shape[0]):
        for j in range(z.shape[1]):
            zp, zm = z.copy(), z.copy()
            zp[i, j] += h; zm[i, j] -= h
            fd[i, j] = (dl @ oracle.softmax_xent(zp, t) - dl @ oracle.softmax_xent(zm, t)) / (2 * h)
    np.testing.assert_allclose(dz, fd, rtol=1e-7, atol=1e-9)


def test_stored_dtypes_round_once():
    r, z, t = rng_case(4)
    l64 = oracle.softmax_xent(z, t)
    l32 = oracle.softmax_xent(z, t, oracle.F32)
    np.testing.assert_array_equal(l32, l64.astype(np.float32).astype(np.float64))
    _, dzb = oracle.softmax_xent_grad(z, t, np.ones(5), dz_dtype=oracle.BF16)
    _, dz = oracle.softmax_xent_grad(z, t, np.ones(5))
    np.testing.assert_array_equal(dzb, oracle.cast_array(dz, oracle.BF16))


def test_sgd_update_closed_forms_and_rounding():
    p = np.array([1.0, -2.0, 0.5, 8.0])
    g = np.array([4.0, 4.0, -1.0, 0.0])
    np.testing.assert_array_equal(oracle.sgd_update(p, g, 0.25), [0.0, -3.0, 0.75, 8.0])
    np.testing.assert_array_equal(oracle.sgd_update(p, g, 0.0), p)
    np.testing.assert_array_equal(oracle.sgd_update(p, np.zeros(4), 7.0), p)
    # bf16 storage: 1 - 2^-9 lies halfway between 1 - 2^-8 and 1; ties go to the even mantissa (1.0);
    # 1 - 3*2^-10 is nearer to 1 - 2^-8
    out = oracle.sgd_update(np.array([1.0, 1.0]), np.array([2.0 ** -9, 3 * 2.0 ** -10]), 1.0, oracle.BF16)
    np.testing.assert_array_equal(out, [1.0, 1.0 - 2.0 ** -8])
    # fp32 storage rounds the fp64 difference once
    r = np.random.default_rng(0)
    pp, gg = r.normal(0, 1, 100), r.normal(0, 1, 100)
    np.testing.assert_array_equal(oracle.sgd_update(pp, gg, 0.01, oracle.F32), (pp - 0.01 * gg).astype(np.float32).astype(np.float64))


def test_sgd_step_decreases_the_loss_of_a_linear_softmax_model():
    """One descent step along the oracle's own gradient lowers the oracle's loss (first-order check that the
    sign conventions of the two functions agree)."""
    r = np.random.default_rng(9)
    x, w = r.normal(0, 1, (16, 8)), r.normal(0, 0.1, (8, 5))
    t = np.eye(5)[r.integers(0, 5, 16)]
    loss0, dz = oracle.softmax_xent_grad(x @ w, t, np.full(16, 1 / 16))
    w1 = oracle.sgd_update(w, x.T @ dz, 0.5)
    assert oracle.softmax_xent(x @ w1, t).mean() < loss0.mean() - 1e-3
