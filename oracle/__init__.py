"""TEST INFRASTRUCTURE ONLY: ctypes front end of the fp64 CPU oracle (relay_oracle.c).

The oracle restates, as plain loops in fp64, what each primitive-operator group of a Relay
program computes (paper Section 3, Fig. 1; Section 4.2; Section 4.3, Fig. 5).  It is used by
the tests, by the smoke check and by the benchmark's CPU-baseline leg, and by nothing else;
it imports nothing from the CUDA package and the CUDA package imports nothing from here.

All tensors cross this interface as C-contiguous float64 numpy arrays holding the exact
values of the stored (bf16 / fp32) tensors.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "relay_oracle.c")
_LIB = os.path.join(_HERE, "_relay_oracle.so")

# dtype / activation / opcode / reduction codes (the oracle's own copy of the tables)
F32, BF16, I32, I64, BOOL, F64 = 0, 1, 2, 3, 4, 5
ACT_NONE, ACT_RELU, ACT_TANH, ACT_SIGMOID = 0, 1, 2, 3
RED_NONE, RED_SUM, RED_MAX, RED_MEAN, RED_ARGMAX = 0, 1, 2, 3, 4


def build(force: bool = False) -> str:
    """Compile relay_oracle.c with gcc (plain -O2, no fast-math so sums keep their order)."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _L():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.orc_round_bf16.restype = ctypes.c_double
        _lib.orc_round_bf16.argtypes = [ctypes.c_double]
        _lib.orc_round_f32.restype = ctypes.c_double
        _lib.orc_round_f32.argtypes = [ctypes.c_double]
        _lib.orc_act.restype = ctypes.c_double
        _lib.orc_act.argtypes = [ctypes.c_double, ctypes.c_int]
        _lib.orc_act_grad_from_output.restype = ctypes.c_double
        _lib.orc_act_grad_from_output.argtypes = [ctypes.c_double, ctypes.c_int]
    return _lib


_dp = ctypes.POINTER(ctypes.c_double)
_i64p = ctypes.POINTER(ctypes.c_int64)
_i32p = ctypes.POINTER(ctypes.c_int32)


def _f64(a) -> np.ndarray:
    return np.asarray(a, dtype=np.float64, order="C")  # (ascontiguousarray would promote rank 0)


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(_dp)


def _i32(v) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(v, dtype=np.int32))


def _i64(v) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(v, dtype=np.int64))


def round_bf16(v: float) -> float:
    return _L().orc_round_bf16(float(v))


def round_f32(v: float) -> float:
    return _L().orc_round_f32(float(v))


def act(z: float, code: int) -> float:
    return _L().orc_act(float(z), int(code))


def act_grad_from_output(y: float, code: int) -> float:
    return _L().orc_act_grad_from_output(float(y), int(code))


def cast_array(a, dtype: int) -> np.ndarray:
    """Elementwise cast through the oracle's own rounding routines."""
    a = _f64(a)
    out = np.empty_like(a)
    _L().orc_cast_array(_ptr(a), ctypes.c_int64(a.size), int(dtype), _ptr(out))
    return out


# ---------------------------------------------------------------------------------------------
# shapes
# ---------------------------------------------------------------------------------------------
def broadcast_shape(sa: Sequence[int], sb: Sequence[int]) -> Optional[tuple]:
    """NumPy-style broadcast of two shapes; None when illegal."""
    a, b = _i64(list(sa)), _i64(list(sb))
    out = np.zeros(max(len(sa), len(sb), 1), dtype=np.int64)
    r = _L().orc_broadcast_shape(
        len(sa), a.ctypes.data_as(_i64p), len(sb), b.ctypes.data_as(_i64p), out.ctypes.data_as(_i64p)
    )
    return None if r < 0 else tuple(int(v) for v in out[:r])


def reduce_shape(shape: Sequence[int], axes: Sequence[int], keepdims: bool) -> tuple:
    s = _i64(list(shape))
    mask = 0
    for ax in axes:
        mask |= 1 << ax
    out = np.zeros(max(len(shape), 1), dtype=np.int64)
    r = _L().orc_reduce_shape(len(shape), s.ctypes.data_as(_i64p), mask, int(keepdims), out.ctypes.data_as(_i64p))
    return tuple(int(v) for v in out[:r])


def conv2d_out_extent(n: int, k: int, stride: int, pad: int) -> Optional[int]:
    out = ctypes.c_int64(0)
    rc = _L().orc_conv2d_out_extent(
        ctypes.c_int64(n), ctypes.c_int64(k), ctypes.c_int64(stride), ctypes.c_int64(pad), ctypes.byref(out)
    )
    return None if rc else int(out.value)


# ---------------------------------------------------------------------------------------------
# elementwise / reduce groups
# ---------------------------------------------------------------------------------------------
def _aligned_shapes(inputs, rank):
    shapes = np.ones((max(len(inputs), 1), max(rank, 1)), dtype=np.int64)
    for i, a in enumerate(inputs):
        if a.ndim > rank:
            raise ValueError("input rank exceeds output rank")
        if a.ndim:
            shapes[i, rank - a.ndim:rank] = a.shape
    return np.ascontiguousarray(shapes[:, :rank].reshape(-1)) if rank else np.zeros(0, dtype=np.int64)


def _common_shape(inputs):
    shape: tuple = ()
    for a in inputs:
        shape = broadcast_shape(shape, a.shape)
        if shape is None:
            raise ValueError("inputs do not broadcast")
    return shape


def _prog_arrays(prog):
    """prog: dict with integer lists op, a, b, c, dtype and float list imm (the instruction
    list of the group; value ids 0..n_in-1 name inputs, n_in+j the result of instruction j)."""
    return (
        _i32(prog["op"]), _i32(prog["a"]), _i32(prog["b"]), _i32(prog["c"]),
        _f64(prog["imm"]), _i32(prog["dtype"]),
    )


def ewise(prog, inputs: Sequence[np.ndarray], out_ids: Sequence[int]):
    """Evaluate an elementwise program over NumPy-broadcast inputs; returns one fp64 array per
    requested value id."""
    ins = [_f64(a) for a in inputs]
    shape = _common_shape(ins)
    rank = len(shape)
    oshape = _i64(list(shape))
    ishapes = _aligned_shapes(ins, rank)
    op, a, b, c, imm, dt = _prog_arrays(prog)
    outs = [np.empty(shape, dtype=np.float64) for _ in out_ids]
    in_ptrs = (_dp * max(len(ins), 1))(*[_ptr(x) for x in ins])
    out_ptrs = (_dp * max(len(outs), 1))(*[_ptr(x) for x in outs])
    oid = _i32(list(out_ids))
    rc = _L().orc_ewise(
        rank, oshape.ctypes.data_as(_i64p), len(ins), in_ptrs, ishapes.ctypes.data_as(_i64p),
        len(op), op.ctypes.data_as(_i32p), a.ctypes.data_as(_i32p), b.ctypes.data_as(_i32p),
        c.ctypes.data_as(_i32p), imm.ctypes.data_as(_dp), dt.ctypes.data_as(_i32p),
        len(outs), oid.ctypes.data_as(_i32p), out_ptrs,
    )
    if rc:
        raise ValueError(f"oracle ewise failed: {rc}")
    return outs


def reduce(prog, inputs: Sequence[np.ndarray], out_specs):
    """out_specs: list of (value_id, red_op, axes, keepdims, out_dtype).  Returns one array per
    spec: unreduced fp64 for RED_NONE; fp64 of the reduced shape otherwise (int64 for argmax)."""
    ins = [_f64(a) for a in inputs]
    shape = _common_shape(ins)
    rank = len(shape)
    oshape = _i64(list(shape))
    ishapes = _aligned_shapes(ins, rank)
    op, a, b, c, imm, dt = _prog_arrays(prog)
    outs, masks, rshapes = [], [], []
    for (vid, red, axes, keep, odt) in out_specs:
        mask = 0
        for ax in axes:
            mask |= 1 << (ax % rank if rank else 0)
        masks.append(mask if red != RED_NONE else 0)
        if red == RED_NONE:
            rshapes.append(shape)
        else:
            rshapes.append(reduce_shape(shape, [d for d in range(rank) if mask >> d & 1], keep))
        outs.append(np.empty(rshapes[-1], dtype=np.float64))
    in_ptrs = (_dp * max(len(ins), 1))(*[_ptr(x) for x in ins])
    out_ptrs = (_dp * max(len(outs), 1))(*[_ptr(x) for x in outs])
    oid = _i32([s[0] for s in out_specs])
    red = _i32([s[1] for s in out_specs])
    msk = _i32(masks)
    odt = _i32([s[4] for s in out_specs])
    rc = _L().orc_reduce(
        rank, oshape.ctypes.data_as(_i64p), len(ins), in_ptrs, ishapes.ctypes.data_as(_i64p),
        len(op), op.ctypes.data_as(_i32p), a.ctypes.data_as(_i32p), b.ctypes.data_as(_i32p),
        c.ctypes.data_as(_i32p), imm.ctypes.data_as(_dp), dt.ctypes.data_as(_i32p),
        len(outs), oid.ctypes.data_as(_i32p), red.ctypes.data_as(_i32p), msk.ctypes.data_as(_i32p),
        odt.ctypes.data_as(_i32p), out_ptrs,
    )
    if rc:
        raise ValueError(f"oracle reduce failed: {rc}")
    return [o.astype(np.int64) if s[1] == RED_ARGMAX else o for o, s in zip(outs, out_specs)]


# ---------------------------------------------------------------------------------------------
# dense / conv2d anchors and their gradient groups
# ---------------------------------------------------------------------------------------------
def dense_act(x, w, b, act_code: int, y_dtype: int) -> np.ndarray:
    x, w = _f64(x), _f64(w)
    b = None if b is None else _f64(b)
    M, K = x.shape
    K2, N = w.shape
    assert K == K2 and (b is None or b.shape == (N,))
    y = np.empty((M, N), dtype=np.float64)
    i64 = ctypes.c_int64
    rc = _L().orc_dense_act(_ptr(x), _ptr(w), _ptr(b), i64(M), i64(K), i64(N), int(act_code), int(y_dtype), _ptr(y))
    assert rc == 0
    return y


def dense_act_grad(x, w, y, dy, act_code: int, dx_dtype: int, dw_dtype: int, db_dtype: int,
                   want_dx=True, want_dw=True, want_db=True, dz_dtype: int = F64):
    x, w, y, dy = _f64(x), _f64(w), _f64(y), _f64(dy)
    M, K = x.shape
    _, N = w.shape
    assert w.shape == (K, N) and y.shape == (M, N) and dy.shape == (M, N)
    dx = np.empty((M, K)) if want_dx else None
    dw = np.empty((K, N)) if want_dw else None
    db = np.empty((N,)) if want_db else None
    i64 = ctypes.c_int64
    rc = _L().orc_dense_act_grad(
        _ptr(x), _ptr(w), _ptr(y), _ptr(dy), i64(M), i64(K), i64(N), int(act_code), int(dz_dtype),
        int(dx_dtype), int(dw_dtype), int(db_dtype), _ptr(dx), _ptr(dw), _ptr(db),
    )
    assert rc == 0
    return dx, dw, db


def softmax_xent(z, t, loss_dtype: int = F64) -> np.ndarray:
    """loss[i] = -sum_j t[i,j] log softmax(z[i,:])_j (Fig. 3, relay.softmax_cross_entropy)."""
    z, t = _f64(z), _f64(t)
    Bn, C = z.shape
    assert t.shape == (Bn, C)
    loss = np.empty((Bn,), dtype=np.float64)
    i64 = ctypes.c_int64
    rc = _L().orc_softmax_xent(_ptr(z), _ptr(t), i64(Bn), i64(C), int(loss_dtype), _ptr(loss))
    assert rc == 0
    return loss


def softmax_xent_grad(z, t, dloss, loss_dtype: int = F64, dz_dtype: int = F64):
    """Returns (loss, dz): the result bundled with the partial with respect to the scores (Section 4.2)."""
    z, t, dloss = _f64(z), _f64(t), _f64(dloss)
    Bn, C = z.shape
    assert t.shape == (Bn, C) and dloss.shape == (Bn,)
    loss = np.empty((Bn,), dtype=np.float64)
    dz = np.empty((Bn, C), dtype=np.float64)
    i64 = ctypes.c_int64
    rc = _L().orc_softmax_xent_grad(_ptr(z), _ptr(t), _ptr(dloss), i64(Bn), i64(C), int(loss_dtype), int(dz_dtype),
                                    _ptr(loss), _ptr(dz))
    assert rc == 0
    return loss, dz


def max_pool2d(x, kh: int, kw: int, sh: int, sw: int):
    """(y, idx): window maxima of an NCHW tensor and the in-plane position h*W+w of the first maximum
    (Fig. 3, relay.max_pool)."""
    x = _f64(x)
    Nb, C, H, W = x.shape
    if kh > H or kw > W or min(kh, kw, sh, sw) <= 0:
        raise ValueError("window does not fit")
    P, Q = (H - kh) // sh + 1, (W - kw) // sw + 1
    y = np.empty((Nb, C, P, Q), dtype=np.float64)
    idx = np.empty((Nb, C, P, Q), dtype=np.int32)
    i64 = ctypes.c_int64
    rc = _L().orc_max_pool2d(_ptr(x), i64(Nb), i64(C), i64(H), i64(W), i64(kh), i64(kw), i64(sh), i64(sw), _ptr(y),
                             idx.ctypes.data_as(_i32p))
    assert rc == 0
    return y, idx


def max_pool2d_grad(idx, dy, H: int, W: int, dx_dtype: int = F64) -> np.ndarray:
    idx = np.asarray(idx, dtype=np.int32, order="C")
    dy = _f64(dy)
    Nb, C, P, Q = dy.shape
    assert idx.shape == dy.shape
    dx = np.empty((Nb, C, H, W), dtype=np.float64)
    i64 = ctypes.c_int64
    rc = _L().orc_max_pool2d_grad(idx.ctypes.data_as(_i32p), _ptr(dy), i64(Nb), i64(C), i64(H), i64(W), i64(P), i64(Q),
                                  int(dx_dtype), _ptr(dx))
    if rc != 0:
        raise ValueError("index outside the plane")
    return dx


def sgd_update(p, g, lr: float, p_dtype: int = F64) -> np.ndarray:
    """p - lr * g stored in p_dtype (Section 4.1, relay.update_model_params)."""
    p, g = _f64(p), _f64(g)
    assert p.shape == g.shape
    out = np.empty(p.shape, dtype=np.float64)
    fn = _L().orc_sgd_update
    fn.restype = None
    fn(_ptr(p), _ptr(g), ctypes.c_int64(p.size), ctypes.c_double(lr), int(p_dtype), _ptr(out))
    return out


def conv2d_act(x, wt, b, stride: int, pad: int, act_code: int, y_dtype: int) -> np.ndarray:
    x, wt = _f64(x), _f64(wt)
    b = None if b is None else _f64(b)
    Nb, C, H, W = x.shape
    O, C2, R, S = wt.shape
    assert C == C2
    P, Q = conv2d_out_extent(H, R, stride, pad), conv2d_out_extent(W, S, stride, pad)
    y = np.empty((Nb, O, P, Q), dtype=np.float64)
    i64 = ctypes.c_int64
    rc = _L().orc_conv2d_act(
        _ptr(x), _ptr(wt), _ptr(b), i64(Nb), i64(C), i64(H), i64(W), i64(O), i64(R), i64(S),
        i64(stride), i64(pad), int(act_code), int(y_dtype), _ptr(y),
    )
    assert rc == 0
    return y


def conv2d_act_grad(x, wt, y, dy, stride: int, pad: int, act_code: int, dx_dtype: int,
                    dw_dtype: int, db_dtype: int, want_dx=True, want_dw=True, want_db=True,
                    dz_dtype: int = F64):
    x, wt, y, dy = _f64(x), _f64(wt), _f64(y), _f64(dy)
    Nb, C, H, W = x.shape
    O, _, R, S = wt.shape
    dx = np.empty_like(x) if want_dx else None
    dw = np.empty_like(wt) if want_dw else None
    db = np.empty((O,)) if want_db else None
    i64 = ctypes.c_int64
    rc = _L().orc_conv2d_act_grad(
        _ptr(x), _ptr(wt), _ptr(y), _ptr(dy), i64(Nb), i64(C), i64(H), i64(W), i64(O), i64(R),
        i64(S), i64(stride), i64(pad), int(act_code), int(dz_dtype), int(dx_dtype), int(dw_dtype),
        int(db_dtype), _ptr(dx), _ptr(dw), _ptr(db),
    )
    assert rc == 0
    return dx, dw, db


def lstm_cell_seq(x, w_ih, w_hh, b, h0, c0, rec_dtype: int = BF16, state_dtype: int = F32):
    x, w_ih, w_hh, b, h0, c0 = (_f64(v) for v in (x, w_ih, w_hh, b, h0, c0))
    T, B, I = x.shape
    H = h0.shape[1]
    assert w_ih.shape == (I, 4 * H) and w_hh.shape == (H, 4 * H) and b.shape == (4 * H,)
    assert h0.shape == (B, H) and c0.shape == (B, H)
    h_all = np.empty((T, B, H), dtype=np.float64)
    c_fin = np.empty((B, H), dtype=np.float64)
    i64 = ctypes.c_int64
    rc = _L().orc_lstm_cell_seq(
        _ptr(x), _ptr(w_ih), _ptr(w_hh), _ptr(b), _ptr(h0), _ptr(c0), i64(T), i64(B), i64(I), i64(H),
        int(rec_dtype), int(state_dtype), _ptr(h_all), _ptr(c_fin),
    )
    assert rc == 0
    return h_all, c_fin


def lstm_cell_seq_grad(x, w_ih, w_hh, b, h0, c0, dh_all, dc_final=None, rec_dtype: int = BF16, state_dtype: int = F32,
                       dz_dtype: int = BF16):
    """Partials (dx, dw_ih, dw_hh, db, dh0, dc0) of sum(dh_all * h_all) + sum(dc_final * c_final), as fp64."""
    x, w_ih, w_hh, b, h0, c0, dh_all = (_f64(v) for v in (x, w_ih, w_hh, b, h0, c0, dh_all))
    dc_final = None if dc_final is None else _f64(dc_final)
    T, B, I = x.shape
    H = h0.shape[1]
    assert w_ih.shape == (I, 4 * H) and w_hh.shape == (H, 4 * H) and b.shape == (4 * H,)
    assert h0.shape == (B, H) and c0.shape == (B, H) and dh_all.shape == (T, B, H)
    assert dc_final is None or dc_final.shape == (B, H)
    dx, dwi, dwh = np.empty((T, B, I)), np.empty((I, 4 * H)), np.empty((H, 4 * H))
    db, dh0, dc0 = np.empty((4 * H,)), np.empty((B, H)), np.empty((B, H))
    i64 = ctypes.c_int64
    rc = _L().orc_lstm_cell_seq_grad(
        _ptr(x), _ptr(w_ih), _ptr(w_hh), _ptr(b), _ptr(h0), _ptr(c0), _ptr(dh_all), _ptr(dc_final), i64(T), i64(B), i64(I),
        i64(H), int(rec_dtype), int(state_dtype), int(dz_dtype), _ptr(dx), _ptr(dwi), _ptr(dwh), _ptr(db), _ptr(dh0), _ptr(dc0))
    assert rc == 0
    return dx, dwi, dwh, db, dh0, dc0
