"""Tolerances and helpers shared by the GPU parity tests.

fp32 paths:  max_i |g_i - o_i| / max(|o_i|, 1e-2 * RMS(o))  <=  1e-4.
bf16-input / fp32-accumulate paths:  |g_i - o_i| <= 1e-2 * RMS(o) (+ half a bf16 ulp of o_i when
the result itself is stored in bf16: the nearest bf16 to a value inside the stated bound), with
o the oracle's fp64 value before any storage rounding; in addition the RMS of the error must
stay below 4e-3 * RMS(o), a much tighter guard that a wrong term cannot pass.
"""
import numpy as np
import torch


def rms(a) -> float:
    a = np.asarray(a, dtype=np.float64)
    return float(np.sqrt(np.mean(np.square(a)))) if a.size else 0.0


def to_np(t) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float64).numpy() if isinstance(t, torch.Tensor) else np.asarray(t, dtype=np.float64)


def bf16_ulp(v: np.ndarray) -> np.ndarray:
    a = np.maximum(np.abs(v), 2.0 ** -126)
    return 2.0 ** (np.floor(np.log2(a)) - 7)


# Per test: the largest PLAIN relative error |g - o| / |o| over the elements with o != 0 that assert_f32 has seen, i.e. the
# criterion without the floor on the denominator.  It is not the gate (an element that is the difference of two nearly
# equal terms can have any relative error in fp32) but it is reported at the end of the run (conftest.py), so that a reader
# sees how far the plain criterion is met.
STRICT_REL = {}


def assert_f32(got, want, what=""):
    g, o = to_np(got), np.asarray(want, dtype=np.float64)
    assert g.shape == o.shape, (what, g.shape, o.shape)
    if o.size == 0:
        return
    assert np.all(np.isfinite(g)), what
    nz = o != 0
    if nz.any():
        import os
        key = os.environ.get("PYTEST_CURRENT_TEST", "?").split(" ")[0]
        STRICT_REL[key] = max(STRICT_REL.get(key, 0.0), float((np.abs(g - o)[nz] / np.abs(o[nz])).max()))
    err = np.abs(g - o) / np.maximum(np.abs(o), 1e-2 * rms(o) + 1e-30)
    assert err.max() <= 1e-4, (what, float(err.max()), np.unravel_index(err.argmax(), err.shape))


def assert_bf16(got, want, stored_bf16=True, what=""):
    g, o = to_np(got), np.asarray(want, dtype=np.float64)
    assert g.shape == o.shape, (what, g.shape, o.shape)
    if o.size == 0:
        return
    assert np.all(np.isfinite(g)), what
    r = rms(o)
    bound = 1e-2 * r + (0.5 * bf16_ulp(o) if stored_bf16 else 0.0) + 1e-30
    err = np.abs(g - o)
    bad = err > bound
    assert not bad.any(), (what, int(bad.sum()), float(err.max()), float(r), np.unravel_index(err.argmax(), err.shape))
    assert rms(g - o) <= 4e-3 * r + 1e-30, (what, rms(g - o), r)


class Guarded:
    """Output buffer with sentinel-filled margins on both sides to catch out-of-range writes.  The view itself starts
    out holding a value no result can take (NaN for floating types, the most negative integer for signed ones, 255 for bytes), and
    `check` asserts that none of it survives: an output element that no work unit wrote shows at any size."""

    def __init__(self, shape, dtype, device, margin=256):
        n = int(np.prod(shape)) if len(shape) else 1
        item = torch.empty((), dtype=dtype).element_size()
        m = (margin * 16) // item          # keeps the view 16-byte aligned
        self.full = torch.full((n + 2 * m,), 7, dtype=dtype, device=device)
        self.m, self.n = m, n
        self.t = self.full[m:m + n].view(tuple(shape))
        self.unwritten = float("nan") if dtype.is_floating_point else (0 if dtype == torch.bool else 255 if dtype == torch.uint8 else torch.iinfo(dtype).min)
        if dtype != torch.bool:
            self.t.fill_(self.unwritten)

    def check(self, all_written=True):
        assert bool((self.full[:self.m] == 7).all()) and bool((self.full[self.m + self.n:] == 7).all()), "out-of-range write"
        if all_written and self.n and self.t.dtype != torch.bool:
            left = torch.isnan(self.t) if self.t.dtype.is_floating_point else (self.t == self.unwritten)
            assert not bool(left.any()), ("elements never written", int(left.sum()), left.nonzero()[:4].tolist())
        return self.t


def workspace(nbytes, device):
    return torch.empty(max(int(nbytes), 16), dtype=torch.uint8, device=device)
