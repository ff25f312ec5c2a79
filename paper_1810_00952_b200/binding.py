"""Thin ctypes binding of the C-ABI library (librelay_b200.so): argument marshalling only.

Every function here has the name and the meaning of the C entry point it calls
(include/relay_b200.h); torch supplies device memory and the current stream, nothing else.
A missing library or a non-OK status raises -- there is no other code path.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# RELAY_B200_LIB names another build of the same library (the bounds-check variant librelay_b200_check.so)
LIB_PATH = os.environ.get("RELAY_B200_LIB") or os.path.join(_HERE, "librelay_b200.so")
CHECK_LIB_PATH = os.path.join(_HERE, "librelay_b200_check.so")

MAX_RANK = 6
F32, BF16, I32, I64, BOOL = 0, 1, 2, 3, 4
ROWMAJOR, NCHW, NHWC, OIHW = 0, 1, 2, 3
ACT_NONE, ACT_RELU, ACT_TANH, ACT_SIGMOID = 0, 1, 2, 3
RED_NONE, RED_SUM, RED_MAX, RED_MEAN, RED_ARGMAX = 0, 1, 2, 3, 4

STATUS_NAMES = ["OK", "ERR_NULL", "ERR_RANK", "ERR_SHAPE", "ERR_DTYPE", "ERR_LAYOUT", "ERR_ALIGN", "ERR_ATTR",
                "ERR_UNSUPPORTED", "ERR_WORKSPACE", "ERR_CUDA", "ERR_TIMEOUT"]

_TORCH2RELAY = {torch.float32: F32, torch.bfloat16: BF16, torch.int32: I32, torch.int64: I64, torch.bool: BOOL,
                torch.uint8: BOOL}


class RelayError(RuntimeError):
    def __init__(self, status: int, text: str):
        self.status = status
        self.status_name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__(f"RELAY_{self.status_name}: {text}")


class TensorDesc(ctypes.Structure):
    _fields_ = [("data", ctypes.c_void_p), ("dtype", ctypes.c_int32), ("rank", ctypes.c_int32),
                ("shape", ctypes.c_int64 * MAX_RANK), ("layout", ctypes.c_int32), ("reserved", ctypes.c_int32)]


class Instr(ctypes.Structure):
    _fields_ = [("op", ctypes.c_int32), ("a", ctypes.c_int32), ("b", ctypes.c_int32), ("c", ctypes.c_int32),
                ("dtype", ctypes.c_int32), ("reserved", ctypes.c_int32), ("imm", ctypes.c_double)]


class EwiseProg(ctypes.Structure):
    _fields_ = [("n_instr", ctypes.c_int32), ("reserved", ctypes.c_int32), ("instr", ctypes.POINTER(Instr))]


class OutSpec(ctypes.Structure):
    _fields_ = [("value", ctypes.c_int32), ("red_op", ctypes.c_int32), ("axes_mask", ctypes.c_int32),
                ("keepdims", ctypes.c_int32)]


class Conv2dAttrs(ctypes.Structure):
    _fields_ = [("stride", ctypes.c_int32), ("pad", ctypes.c_int32), ("dilation", ctypes.c_int32),
                ("groups", ctypes.c_int32)]


_lib = None


class Pool2dAttrs(ctypes.Structure):
    _fields_ = [("kh", ctypes.c_int32), ("kw", ctypes.c_int32), ("sh", ctypes.c_int32), ("sw", ctypes.c_int32)]


def lib() -> ctypes.CDLL:
    """Loads the library; fails loudly if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_1810_00952_b200.build`; "
                              "there is no fallback path")
        L = ctypes.CDLL(LIB_PATH)
        L.relay_last_error.restype = ctypes.c_char_p
        L.relay_version.restype = ctypes.c_char_p
        L.relay_launch_count.restype = ctypes.c_int64
        for name in ("relay_workspace_bytes_dense_act", "relay_workspace_bytes_dense_act_grad",
                     "relay_workspace_bytes_conv2d_act", "relay_workspace_bytes_conv2d_act_grad",
                     "relay_workspace_bytes_reduce", "relay_workspace_bytes_lstm", "relay_workspace_bytes_lstm_grad"):
            getattr(L, name).restype = ctypes.c_size_t
        _lib = L
    return _lib


def _check(status: int):
    if status != 0:
        raise RelayError(status, lib().relay_last_error().decode())


# ---- descriptors ------------------------------------------------------------------------------------
def desc(t: Optional[torch.Tensor], layout: int = ROWMAJOR) -> Optional[TensorDesc]:
    """Descriptor of a contiguous torch tensor (device or host pointer is passed through as is)."""
    if t is None:
        return None
    if not t.is_contiguous():
        raise ValueError("tensors crossing the C-ABI must be contiguous")
    if t.dtype not in _TORCH2RELAY:
        raise ValueError(f"dtype {t.dtype} has no Relay base type here")
    d = TensorDesc()
    d.data = t.data_ptr() if t.numel() else (t.data_ptr() or None)
    d.dtype = _TORCH2RELAY[t.dtype]
    d.rank = t.dim()
    for i, s in enumerate(t.shape):
        d.shape[i] = s
    d.layout = layout
    return d


def desc_of_type(dtype: int, shape: Sequence[int], layout: int = ROWMAJOR, data: int = 0) -> TensorDesc:
    d = TensorDesc()
    d.data = data or None
    d.dtype = dtype
    d.rank = len(shape)
    for i, s in enumerate(shape):
        d.shape[i] = s
    d.layout = layout
    return d


def _ref(d):
    return ctypes.byref(d) if d is not None else None


def _shape(d: TensorDesc):
    return tuple(int(d.shape[i]) for i in range(d.rank))


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ws(ws: Optional[torch.Tensor]):
    if ws is None:
        return ctypes.c_void_p(None), ctypes.c_size_t(0)
    return ctypes.c_void_p(ws.data_ptr()), ctypes.c_size_t(ws.numel() * ws.element_size())


def make_prog(prog: dict):
    """prog: dict of lists op, a, b, c, dtype, imm (relay_workloads.program.Program.arrays())."""
    n = len(prog["op"])
    arr = (Instr * max(n, 1))()
    for j in range(n):
        arr[j].op, arr[j].a, arr[j].b, arr[j].c = prog["op"][j], prog["a"][j], prog["b"][j], prog["c"][j]
        arr[j].dtype, arr[j].imm = prog["dtype"][j], prog["imm"][j]
    p = EwiseProg()
    p.n_instr = n
    p.instr = ctypes.cast(arr, ctypes.POINTER(Instr))
    p._keep = arr
    return p


def _desc_array(descs):
    arr = (ctypes.POINTER(TensorDesc) * max(len(descs), 1))()
    for i, d in enumerate(descs):
        arr[i] = ctypes.pointer(d)
    return arr


# ---- type relations (host only) -----------------------------------------------------------------------
def relay_infer_dense(x: TensorDesc, w: TensorDesc) -> TensorDesc:
    out = TensorDesc()
    _check(lib().relay_infer_dense(_ref(x), _ref(w), ctypes.byref(out)))
    return out


def relay_infer_conv2d(x: TensorDesc, w: TensorDesc, stride: int, pad: int, dilation: int = 1, groups: int = 1) -> TensorDesc:
    out = TensorDesc()
    at = Conv2dAttrs(stride, pad, dilation, groups)
    _check(lib().relay_infer_conv2d(_ref(x), _ref(w), ctypes.byref(at), ctypes.byref(out)))
    return out


def relay_infer_broadcast(a: TensorDesc, b: TensorDesc) -> TensorDesc:
    out = TensorDesc()
    _check(lib().relay_infer_broadcast(_ref(a), _ref(b), ctypes.byref(out)))
    return out


def relay_infer_reduce(t: TensorDesc, red_op: int, axes_mask: int, keepdims: bool) -> TensorDesc:
    out = TensorDesc()
    _check(lib().relay_infer_reduce(_ref(t), red_op, axes_mask, int(keepdims), ctypes.byref(out)))
    return out


def relay_infer_stack(elem: TensorDesc, m: int) -> TensorDesc:
    out = TensorDesc()
    _check(lib().relay_infer_stack(_ref(elem), ctypes.c_int64(m), ctypes.byref(out)))
    return out


def relay_infer_lstm(x: TensorDesc, w_ih: TensorDesc, w_hh: TensorDesc):
    h, c = TensorDesc(), TensorDesc()
    _check(lib().relay_infer_lstm(_ref(x), _ref(w_ih), _ref(w_hh), ctypes.byref(h), ctypes.byref(c)))
    return h, c


def relay_infer_softmax_xent(scores: TensorDesc, targets: TensorDesc) -> TensorDesc:
    out = TensorDesc()
    _check(lib().relay_infer_softmax_xent(_ref(scores), _ref(targets), ctypes.byref(out)))
    return out


def relay_infer_max_pool2d(x: TensorDesc, kh: int, kw: int, sh: int, sw: int) -> TensorDesc:
    out = TensorDesc()
    at = Pool2dAttrs(kh, kw, sh, sw)
    _check(lib().relay_infer_max_pool2d(_ref(x), ctypes.byref(at), ctypes.byref(out)))
    return out


def relay_infer_ewise(prog: dict, inputs: Sequence[TensorDesc], value: int) -> TensorDesc:
    out = TensorDesc()
    p = make_prog(prog)
    _check(lib().relay_infer_ewise(ctypes.byref(p), _desc_array(list(inputs)), len(inputs), value, ctypes.byref(out)))
    return out


# ---- workspace queries ------------------------------------------------------------------------------
def relay_workspace_bytes_dense_act(x, w) -> int:
    return int(lib().relay_workspace_bytes_dense_act(_ref(desc(x)), _ref(desc(w))))


def relay_workspace_bytes_dense_act_grad(x, w) -> int:
    return int(lib().relay_workspace_bytes_dense_act_grad(_ref(desc(x)), _ref(desc(w))))


def relay_workspace_bytes_conv2d_act(x, w, stride, pad, layout=NCHW) -> int:
    at = Conv2dAttrs(stride, pad, 1, 1)
    return int(lib().relay_workspace_bytes_conv2d_act(_ref(desc(x, layout)), _ref(desc(w, OIHW)), ctypes.byref(at)))


def relay_workspace_bytes_conv2d_act_grad(x, w, stride, pad, layout=NCHW) -> int:
    at = Conv2dAttrs(stride, pad, 1, 1)
    return int(lib().relay_workspace_bytes_conv2d_act_grad(_ref(desc(x, layout)), _ref(desc(w, OIHW)), ctypes.byref(at)))


def relay_workspace_bytes_reduce(inputs, specs) -> int:
    ds = [desc(t) for t in inputs]
    sp = (OutSpec * len(specs))(*[OutSpec(*s) for s in specs])
    return int(lib().relay_workspace_bytes_reduce(_desc_array(ds), len(ds), sp, len(specs)))


def relay_workspace_bytes_lstm(x, w_ih, w_hh) -> int:
    return int(lib().relay_workspace_bytes_lstm(_ref(desc(x)), _ref(desc(w_ih)), _ref(desc(w_hh))))


# ---- compute entry points -----------------------------------------------------------------------------
def relay_fused_dense_act(x, w, b, act, y, ws=None):
    wp, wb = _ws(ws)
    _check(lib().relay_fused_dense_act(_ref(desc(x)), _ref(desc(w)), _ref(desc(b)), int(act), _ref(desc(y)), wp, wb, _stream()))


def relay_fused_dense_act_grad(x, w, y, dy, act, dx, dw, db, ws=None):
    wp, wb = _ws(ws)
    _check(lib().relay_fused_dense_act_grad(_ref(desc(x)), _ref(desc(w)), _ref(desc(y)), _ref(desc(dy)), int(act),
                                            _ref(desc(dx)), _ref(desc(dw)), _ref(desc(db)), wp, wb, _stream()))


def relay_contract_act(a, trans_a, b, trans_b, bias, act, c):
    _check(lib().relay_contract_act(_ref(desc(a)), int(bool(trans_a)), _ref(desc(b)), int(bool(trans_b)), _ref(desc(bias)), int(act),
                                    _ref(desc(c)), _stream()))


def relay_fused_conv2d_act(x, w, b, stride, pad, act, y, ws=None, layout=NCHW):
    """`layout` tags x and y: NCHW tensors of shape (N,C,H,W) or NHWC tensors of shape (N,H,W,C)."""
    wp, wb = _ws(ws)
    at = Conv2dAttrs(stride, pad, 1, 1)
    _check(lib().relay_fused_conv2d_act(_ref(desc(x, layout)), _ref(desc(w, OIHW)), _ref(desc(b)), ctypes.byref(at), int(act),
                                        _ref(desc(y, layout)), wp, wb, _stream()))


def relay_fused_conv2d_act_grad(x, w, y, dy, stride, pad, act, dx, dw, db, ws=None, layout=NCHW):
    wp, wb = _ws(ws)
    at = Conv2dAttrs(stride, pad, 1, 1)
    _check(lib().relay_fused_conv2d_act_grad(_ref(desc(x, layout)), _ref(desc(w, OIHW)), _ref(desc(y, layout)),
                                             _ref(desc(dy, layout)), ctypes.byref(at), int(act), _ref(desc(dx, layout)),
                                             _ref(desc(dw, OIHW)), _ref(desc(db)), wp, wb, _stream()))


def relay_fused_ewise(prog: dict, inputs, out_values, outputs, ws=None):
    wp, wb = _ws(ws)
    p = make_prog(prog)
    ins = [desc(t) for t in inputs]
    outs = [desc(t) for t in outputs]
    ov = (ctypes.c_int32 * max(len(out_values), 1))(*out_values)
    _check(lib().relay_fused_ewise(ctypes.byref(p), _desc_array(ins), len(ins), ov, _desc_array(outs), len(outs), wp, wb, _stream()))


def relay_fused_reduce(prog: Optional[dict], inputs, specs, outputs, ws=None):
    """specs: sequence of (value, red_op, axes_mask, keepdims)."""
    wp, wb = _ws(ws)
    p = make_prog(prog) if prog is not None else None
    ins = [desc(t) for t in inputs]
    outs = [desc(t) for t in outputs]
    sp = (OutSpec * max(len(specs), 1))(*[OutSpec(*s) for s in specs])
    _check(lib().relay_fused_reduce(ctypes.byref(p) if p is not None else None, _desc_array(ins), len(ins), sp,
                                    _desc_array(outs), len(outs), wp, wb, _stream()))


def relay_debug_group_route(prog: Optional[dict], inputs, specs) -> int:
    """Kernel tier a group would run on: 0 pre-compiled body, 1 vectorised tier (compiled at run time or interpreted), 2 scalar
    evaluator, 3 row reduction.
    specs as for relay_fused_reduce; (value, RED_NONE, 0, 0) entries describe a relay_fused_ewise call.  Host only."""
    p = make_prog(prog) if prog is not None else None
    ins = [desc(t) for t in inputs]
    sp = (OutSpec * max(len(specs), 1))(*[OutSpec(*s) for s in specs])
    r = int(lib().relay_debug_group_route(ctypes.byref(p) if p is not None else None, _desc_array(ins), len(ins), sp, len(specs)))
    if r < 0:
        raise RelayError(1, lib().relay_last_error().decode())
    return r


def relay_debug_jit_compile(prog: Optional[dict], inputs, specs, want_source: bool = False):
    """Host only: generates the body that would be compiled at run time for this group and compiles it for sm_100a.
    Returns the library's code (1 compiled, 0 not on that tier, -1 no run-time compiler), with the source text if asked;
    raises on a compile error or an ill-typed group."""
    p = make_prog(prog) if prog is not None else None
    ins = [desc(t) for t in inputs]
    sp = (OutSpec * max(len(specs), 1))(*[OutSpec(*s) for s in specs])
    cap = 1 << 16
    buf = ctypes.create_string_buffer(cap) if want_source else None
    r = int(lib().relay_debug_jit_compile(ctypes.byref(p) if p is not None else None, _desc_array(ins), len(ins), sp, len(specs), buf,
                                          ctypes.c_size_t(cap if want_source else 0)))
    if r <= -2:
        raise RelayError(1, lib().relay_last_error().decode())
    return (r, buf.value.decode()) if want_source else r


STATIC_SCRATCH_BYTES = 8 << 20


def relay_fused_reduce_static_scratch(prog: Optional[dict], inputs, specs, outputs):
    """relay_fused_reduce without a workspace argument: for callers that may not allocate device
    memory, the partial sums go to a fixed STATIC_SCRATCH_BYTES array inside the library.  Calls
    that overlap on one GPU race on that array; larger groups are rejected (ERR_WORKSPACE)."""
    p = make_prog(prog) if prog is not None else None
    ins = [desc(t) for t in inputs]
    outs = [desc(t) for t in outputs]
    sp = (OutSpec * max(len(specs), 1))(*[OutSpec(*s) for s in specs])
    _check(lib().relay_fused_reduce_static_scratch(ctypes.byref(p) if p is not None else None, _desc_array(ins), len(ins), sp,
                                                   _desc_array(outs), len(outs), _stream()))


def relay_debug_lstm_phase_cycles(x, w_ih, w_hh, b, h0, c0, h_all, c_final, ws, cycles):
    """relay_lstm_cell_seq that also fills `cycles` (device int64[8]) with per-phase cycle counts of the step loop."""
    wp, wb = _ws(ws)
    _check(lib().relay_debug_lstm_phase_cycles(_ref(desc(x)), _ref(desc(w_ih)), _ref(desc(w_hh)), _ref(desc(b)), _ref(desc(h0)), _ref(desc(c0)),
                                               _ref(desc(h_all)), _ref(desc(c_final)), wp, wb, ctypes.c_void_p(cycles.data_ptr()), _stream()))


def relay_lstm_cell_seq(x, w_ih, w_hh, b, h0, c0, h_all, c_final, ws=None):
    wp, wb = _ws(ws)
    _check(lib().relay_lstm_cell_seq(_ref(desc(x)), _ref(desc(w_ih)), _ref(desc(w_hh)), _ref(desc(b)), _ref(desc(h0)),
                                     _ref(desc(c0)), _ref(desc(h_all)), _ref(desc(c_final)), wp, wb, _stream()))


def relay_workspace_bytes_lstm_grad(x, w_ih, w_hh) -> int:
    return int(lib().relay_workspace_bytes_lstm_grad(_ref(desc(x)), _ref(desc(w_ih)), _ref(desc(w_hh))))


def relay_lstm_cell_seq_grad(x, w_ih, w_hh, b, h0, c0, h_all, dh_all, dc_final, dx, dw_ih, dw_hh, db, dh0, dc0, ws=None):
    wp, wb = _ws(ws)
    ts = [x, w_ih, w_hh, b, h0, c0, h_all, dh_all, dc_final, dx, dw_ih, dw_hh, db, dh0, dc0]
    _check(lib().relay_lstm_cell_seq_grad(*[_ref(desc(t)) for t in ts], wp, wb, _stream()))


def relay_softmax_xent(scores, targets, loss):
    _check(lib().relay_softmax_xent(_ref(desc(scores)), _ref(desc(targets)), _ref(desc(loss)), _stream()))


def relay_softmax_xent_grad(scores, targets, dloss, loss, dscores):
    _check(lib().relay_softmax_xent_grad(_ref(desc(scores)), _ref(desc(targets)), _ref(desc(dloss)), _ref(desc(loss)),
                                         _ref(desc(dscores)), _stream()))


def relay_max_pool2d(x, kh, kw, sh, sw, y, idx=None):
    at = Pool2dAttrs(kh, kw, sh, sw)
    _check(lib().relay_max_pool2d(_ref(desc(x, NCHW)), ctypes.byref(at), _ref(desc(y, NCHW)), _ref(desc(idx, NCHW)), _stream()))


def relay_max_pool2d_grad(idx, dy, kh, kw, sh, sw, dx):
    at = Pool2dAttrs(kh, kw, sh, sw)
    _check(lib().relay_max_pool2d_grad(_ref(desc(idx, NCHW)), _ref(desc(dy, NCHW)), ctypes.byref(at), _ref(desc(dx, NCHW)), _stream()))


def relay_sgd_update(params, grads, lr: float):
    pd, gd = [desc(p) for p in params], [desc(g) for g in grads]
    _check(lib().relay_sgd_update(_desc_array(pd), _desc_array(gd), len(pd), ctypes.c_float(lr), _stream()))


# ---- status helpers -----------------------------------------------------------------------------------
def relay_last_error() -> str:
    return lib().relay_last_error().decode()


def relay_poll_status():
    _check(lib().relay_poll_status(_stream()))


def relay_debug_set_jit(enabled: bool) -> bool:
    """Switches the run-time compiled elementwise bodies on or off for this process; returns the previous setting."""
    return bool(lib().relay_debug_set_jit(1 if enabled else 0))


def relay_debug_jit_compiled() -> int:
    """Bodies compiled at run time so far; -1 when compiled bodies cannot be used in this process (no compiler library, no driver)."""
    return int(lib().relay_debug_jit_compiled())


def relay_debug_bounds_probe():
    _check(lib().relay_debug_bounds_probe(_stream()))


def relay_debug_expire_wait(limit_us: int = 1000):
    _check(lib().relay_debug_expire_wait(int(limit_us), _stream()))


def relay_debug_plan_units(M: int, N: int, K: int, sms: int, max_units: int = 1024):
    """Unit plan of the two-SM contraction kernel as (row block, first chunk, width in chunks) triples, or None
    when the kernel would follow its fixed scheme."""
    buf = (ctypes.c_uint32 * max_units)()
    n = int(lib().relay_debug_plan_units(ctypes.c_int64(M), ctypes.c_int64(N), ctypes.c_int64(K), int(sms), buf, max_units))
    if n == -1:
        return None
    if n < 0:
        raise ValueError("relay_debug_plan_units: bad arguments")
    return [(int(e) & 0xFFF, (int(e) >> 12) & 0xFFF, int(e) >> 24) for e in buf[:n]]


def relay_launch_count() -> int:
    return int(lib().relay_launch_count())


def relay_version() -> str:
    return lib().relay_version().decode()
