"""Pins of the oracle's max pooling and its gradient (Fig. 3, relay.max_pool; Section 4.2) against NumPy's
sliding windows, tie and placement rules, conservation of the upstream partial and finite differences."""
import itertools

import numpy as np
import pytest

import oracle


def windows(x, kh, kw, sh, sw):
    v = np.lib.stride_tricks.sliding_window_view(x, (kh, kw), axis=(2, 3))[:, :, ::sh, ::sw]
    return v.reshape(*v.shape[:4], kh * kw)


@pytest.mark.parametrize("H,W,kh,kw,sh,sw", [(4, 4, 2, 2, 2, 2), (5, 7, 2, 2, 2, 2), (6, 6, 3, 3, 1, 1), (7, 5, 3, 2, 2, 1),
                                           (28, 28, 2, 2, 2, 2), (3, 3, 3, 3, 1, 1), (5, 5, 1, 1, 1, 1), (9, 8, 2, 3, 3, 2)])
def test_against_numpy_sliding_windows(H, W, kh, kw, sh, sw):
    r = np.random.default_rng(H * 100 + W)
    x = r.normal(0, 1, (2, 3, H, W))
    y, idx = oracle.max_pool2d(x, kh, kw, sh, sw)
    v = windows(x, kh, kw, sh, sw)
    np.testing.assert_array_equal(y, v.max(axis=-1))
    am = v.argmax(axis=-1)                                     # first maximum, row-major inside the window
    P, Q = y.shape[2:]
    pp, qq = np.meshgrid(np.arange(P), np.arange(Q), indexing="ij")
    want = (pp * sh + am // kw) * W + (qq * sw + am % kw)
    np.testing.assert_array_equal(idx, want)
    assert y.shape == (2, 3, (H - kh) // sh + 1, (W - kw) // sw + 1)
    # the index addresses the maximum inside the plane
    np.testing.assert_array_equal(np.take_along_axis(x.reshape(2, 3, -1), idx.reshape(2, 3, -1), axis=2).reshape(y.shape), y)


def test_ties_pick_the_first_position_of_the_window():
    x = np.ones((1, 1, 4, 6))
    y, idx = oracle.max_pool2d(x, 2, 2, 2, 2)
    np.testing.assert_array_equal(idx[0, 0], [[0, 2, 4], [12, 14, 16]])
    x[0, 0, 1, 1] = 1.0; x[0, 0, 0, 1] = 2.0; x[0, 0, 1, 0] = 2.0   # two equal maxima: row-major first
    _, idx = oracle.max_pool2d(x, 2, 2, 2, 2)
    assert idx[0, 0, 0, 0] == 1


def test_windows_that_do_not_fit_are_rejected():
    with pytest.raises(ValueError):
        oracle.max_pool2d(np.zeros((1, 1, 2, 5)), 3, 2, 1, 1)


def test_gradient_places_and_conserves_the_upstream_partial():
    r = np.random.default_rng(7)
    x = r.normal(0, 1, (2, 2, 6, 8))
    for (kh, kw, sh, sw) in [(2, 2, 2, 2), (3, 3, 1, 1), (2, 3, 1, 2)]:
        y, idx = oracle.max_pool2d(x, kh, kw, sh, sw)
        dy = r.normal(0, 1, y.shape)
        dx = oracle.max_pool2d_grad(idx, dy, 6, 8)
        np.testing.assert_allclose(dx.sum(axis=(2, 3)), dy.sum(axis=(2, 3)), rtol=1e-12, atol=1e-12)
        if sh >= kh and sw >= kw:                               # disjoint windows: dx is dy at the maxima, zero elsewhere
            np.testing.assert_array_equal(np.take_along_axis(dx.reshape(2, 2, -1), idx.reshape(2, 2, -1), axis=2).reshape(y.shape), dy)
            assert np.count_nonzero(dx) == dy.size
        # brute force from the input's side: sum of dy over the windows whose maximum sits here
        want = np.zeros_like(x)
        for n, c, p, q in itertools.product(*(range(s) for s in y.shape)):
            h, w = divmod(int(idx[n, c, p, q]), 8)
            assert p * sh <= h < p * sh + kh and q * sw <= w < q * sw + kw
            want[n, c, h, w] += dy[n, c, p, q]
        np.testing.assert_allclose(dx, want, rtol=1e-14, atol=1e-15)


def test_gradient_matches_finite_differences_with_overlapping_windows():
    r = np.random.default_rng(11)
    x = r.permutation(5 * 6).reshape(1, 1, 5, 6).astype(np.float64)      # distinct values, gaps of 1: no ties near h
    y, idx = oracle.max_pool2d(x, 3, 2, 1, 2)
    dy = r.normal(0, 1, y.shape)
    dx = oracle.max_pool2d_grad(idx, dy, 5, 6)
    h = 1e-3
    fd = np.zeros_like(x)
    for i, j in itertools.product(range(5), range(6)):
        xp, xm = x.copy(), x.copy()
        xp[0, 0, i, j] += h; xm[0, 0, i, j] -= h
        fd[0, 0, i, j] = ((dy * oracle.max_pool2d(xp, 3, 2, 1, 2)[0]).sum() - (dy * oracle.max_pool2d(xm, 3, 2, 1, 2)[0]).sum()) / (2 * h)
    np.testing.assert_allclose(dx, fd, rtol=1e-9, atol=1e-9)


def test_gradient_storage_rounding_and_bad_indices():
    idx = np.array([[[[0, 0]]]], dtype=np.int32)               # both windows point at the same input: contributions add
    dy = np.array([[[[1.0, 2.0 ** -9]]]])
    np.testing.assert_array_equal(oracle.max_pool2d_grad(idx, dy, 1, 2), [[[[1.0 + 2.0 ** -9, 0.0]]]])
    np.testing.assert_array_equal(oracle.max_pool2d_grad(idx, dy, 1, 2, oracle.BF16), [[[[1.0, 0.0]]]])   # tie to even
    with pytest.raises(ValueError):
        oracle.max_pool2d_grad(np.array([[[[2]]]], dtype=np.int32), np.ones((1, 1, 1, 1)), 1, 2)
