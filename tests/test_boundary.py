"""Host-side boundary: the library loads, exports every declared symbol, and applies the type
relations (Fig. 4 kinding rules, Fig. 5 typing rules) to descriptors.  No GPU needed."""
import ctypes
import itertools
import os
import re

import pytest

import oracle
from paper_1810_00952_b200 import binding as B
from relay_workloads import program as P

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "relay_b200.h")


def T(dtype, shape, layout=B.ROWMAJOR):
    return B.desc_of_type(dtype, shape, layout)


def test_library_exports_every_declared_symbol():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = set(re.findall(r"\b(relay_[a-z0-9_]+)\s*\(", text))
    assert len(names) >= 20
    lib = B.lib()
    for n in sorted(names):
        assert hasattr(lib, n), f"{n} declared in the header but not exported"
    assert "sm_100a" in B.relay_version()


def test_code_tables_agree_between_header_builder_and_oracle():
    text = open(HEADER).read()
    def enum(prefix):
        return {m.group(1): int(m.group(2)) for m in re.finditer(prefix + r"([A-Z0-9]+)\s*=\s*(\d+)", text)}
    ops = enum("RELAY_OP_")
    for name, val in ops.items():
        assert getattr(P, "OP_" + name) == val
    oc = open(os.path.join(ROOT, "oracle", "relay_oracle.c")).read()
    for name, val in ops.items():
        assert re.search(r"ORC_OP_%s\s*=\s*%d\b" % (name, val), oc), name
    for name, val in enum("RELAY_RED_").items():
        assert getattr(P, "RED_" + name) == val and getattr(oracle, "RED_" + name) == val
    for name, val in enum("RELAY_ACT_").items():
        assert getattr(P, "ACT_" + name) == val and getattr(oracle, "ACT_" + name) == val
    dts = {m.group(1): int(m.group(2)) for m in re.finditer(r"RELAY_(F32|BF16|I32|I64|BOOL)\s*=\s*(\d+)", text)}
    for name, val in dts.items():
        assert getattr(P, name) == val and getattr(oracle, name) == val and getattr(B, name) == val


def test_struct_layouts_match_header_sizes():
    assert ctypes.sizeof(B.TensorDesc) == 8 + 4 + 4 + 6 * 8 + 4 + 4
    assert ctypes.sizeof(B.Instr) == 32 and ctypes.sizeof(B.OutSpec) == 16 and ctypes.sizeof(B.Conv2dAttrs) == 16


# ---- dense ------------------------------------------------------------------------------------------
def test_infer_dense_relation():
    for M, K, N in [(8, 64, 32), (1, 1, 1), (0, 5, 3), (4096, 4096, 4096)]:
        for dt in (B.F32, B.BF16):
            out = B.relay_infer_dense(T(dt, (M, K)), T(dt, (K, N)))
            assert B._shape(out) == (M, N) and out.dtype == dt and out.rank == 2
    # leading batch axes are carried through (batching adds a leading axis to every tensor, Section 5.2)
    for lead in [(3,), (2, 5), (1, 1, 1, 4)]:
        out = B.relay_infer_dense(T(B.BF16, lead + (7, 16)), T(B.BF16, (16, 24)))
        assert B._shape(out) == lead + (7, 24) and out.rank == len(lead) + 2


@pytest.mark.parametrize("x,w,status", [
    (T(B.F32, (8, 64)), T(B.F32, (63, 32)), "ERR_SHAPE"),
    (T(B.F32, (8, 64)), T(B.BF16, (64, 32)), "ERR_DTYPE"),
    (T(B.I32, (8, 64)), T(B.I32, (64, 32)), "ERR_DTYPE"),
    (T(B.F32, (8, 64, 1)), T(B.F32, (64, 32)), "ERR_SHAPE"),     # a batch of 8 with K = 1, not 64
    (T(B.F32, (64,)), T(B.F32, (64, 32)), "ERR_RANK"),
    (T(B.F32, (8, 64)), T(B.F32, (64,)), "ERR_RANK"),
    (T(B.F32, (8, 64), B.NCHW), T(B.F32, (64, 32)), "ERR_LAYOUT"),
    (T(B.F32, (8, -1)), T(B.F32, (64, 32)), "ERR_SHAPE"),
    (T(9, (8, 64)), T(B.F32, (64, 32)), "ERR_DTYPE"),
])
def test_infer_dense_rejections(x, w, status):
    with pytest.raises(B.RelayError) as e:
        B.relay_infer_dense(x, w)
    assert e.value.status_name == status and len(B.relay_last_error()) > 0


def test_rule_order_rank_before_dtype_before_shape():
    # everything wrong at once: rank is reported first, then dtype, then shape
    with pytest.raises(B.RelayError) as e:
        B.relay_infer_dense(T(B.F32, (8,)), T(B.BF16, (3, 3)))
    assert e.value.status_name == "ERR_RANK"
    with pytest.raises(B.RelayError) as e:
        B.relay_infer_dense(T(B.F32, (8, 4)), T(B.BF16, (3, 3)))
    assert e.value.status_name == "ERR_DTYPE"
    with pytest.raises(B.RelayError) as e:
        B.lib().relay_infer_dense(None, None, None) and None
        B._check(B.lib().relay_infer_dense(None, None, None))
    assert e.value.status_name == "ERR_NULL"


# ---- conv2d -----------------------------------------------------------------------------------------
def test_infer_conv2d_nhwc_tag_permutes_the_relation():
    """An NHWC-tagged x has shape (N,H,W,C); the result is NHWC with the same extents as the NCHW relation gives."""
    for H, W_, R, p, s in [(7, 6, 3, 1, 1), (9, 9, 3, 1, 2), (8, 5, 5, 0, 1), (56, 56, 3, 1, 1)]:
        a = B.relay_infer_conv2d(T(B.BF16, (2, 3, H, W_), B.NCHW), T(B.BF16, (5, 3, R, R), B.OIHW), s, p)
        b = B.relay_infer_conv2d(T(B.BF16, (2, H, W_, 3), B.NHWC), T(B.BF16, (5, 3, R, R), B.OIHW), s, p)
        n, o, pp, q = B._shape(a)
        assert B._shape(b) == (n, pp, q, o) and b.layout == B.NHWC and a.layout == B.NCHW
    with pytest.raises(B.RelayError) as e:          # channels are the LAST axis of an NHWC tensor
        B.relay_infer_conv2d(T(B.BF16, (2, 3, 7, 6), B.NHWC), T(B.BF16, (5, 3, 3, 3), B.OIHW), 1, 1)
    assert e.value.status_name == "ERR_SHAPE"
    with pytest.raises(B.RelayError) as e:
        B.relay_infer_conv2d(T(B.BF16, (2, 3, 7, 6), B.ROWMAJOR), T(B.BF16, (5, 3, 3, 3), B.OIHW), 1, 1)
    assert e.value.status_name == "ERR_LAYOUT"



def test_infer_conv2d_matches_window_counting():
    for H, W_, R, p, s in itertools.product(range(1, 7), (1, 4, 6), (1, 2, 3, 5), (0, 1, 2), (1, 2, 3)):
        x, w = T(B.BF16, (2, 3, H, W_), B.NCHW), T(B.BF16, (5, 3, R, R), B.OIHW)
        fits = H + 2 * p >= R and W_ + 2 * p >= R
        if not fits:
            with pytest.raises(B.RelayError) as e:
                B.relay_infer_conv2d(x, w, s, p)
            assert e.value.status_name == "ERR_SHAPE"
            continue
        out = B.relay_infer_conv2d(x, w, s, p)
        Pn = sum(1 for st in range(-p, H + p - R + 1, s))
        Qn = sum(1 for st in range(-p, W_ + p - R + 1, s))
        assert B._shape(out) == (2, 5, Pn, Qn) and out.layout == B.NCHW
        assert (Pn, Qn) == (oracle.conv2d_out_extent(H, R, s, p), oracle.conv2d_out_extent(W_, R, s, p))


def test_infer_conv2d_rejections():
    x, w = T(B.BF16, (2, 3, 8, 8), B.NCHW), T(B.BF16, (5, 3, 3, 3), B.OIHW)
    cases = [
        (T(B.BF16, (2, 4, 8, 8), B.NCHW), w, (1, 1, 1, 1), "ERR_SHAPE"),
        (T(B.BF16, (2, 3, 8, 8), B.ROWMAJOR), w, (1, 1, 1, 1), "ERR_LAYOUT"),
        (x, T(B.BF16, (5, 3, 3, 3), B.NCHW), (1, 1, 1, 1), "ERR_LAYOUT"),
        (x, T(B.F32, (5, 3, 3, 3), B.OIHW), (1, 1, 1, 1), "ERR_DTYPE"),
        (x, w, (0, 1, 1, 1), "ERR_ATTR"), (x, w, (1, -1, 1, 1), "ERR_ATTR"),
        (x, w, (1, 1, 2, 1), "ERR_ATTR"), (x, w, (1, 1, 1, 2), "ERR_ATTR"),
        (T(B.BF16, (2, 3, 8), B.NCHW), w, (1, 1, 1, 1), "ERR_RANK"),
    ]
    for xx, ww, (s, p, dil, grp), status in cases:
        with pytest.raises(B.RelayError) as e:
            B.relay_infer_conv2d(xx, ww, s, p, dil, grp)
        assert e.value.status_name == status, (status, str(e.value))


# ---- broadcast / ewise typing -------------------------------------------------------------------------
def test_infer_broadcast_brute_force_against_oracle_rule():
    shapes = [s for r in range(4) for s in itertools.product((1, 2, 3), repeat=r)]
    for sa in shapes:
        for sb in shapes:
            want = oracle.broadcast_shape(sa, sb)
            if want is None:
                with pytest.raises(B.RelayError) as e:
                    B.relay_infer_broadcast(T(B.F32, sa), T(B.F32, sb))
                assert e.value.status_name == "ERR_SHAPE"
            else:
                assert B._shape(B.relay_infer_broadcast(T(B.F32, sa), T(B.F32, sb))) == want


def test_infer_ewise_types_follow_fig5():
    p = P.Program([P.BF16, P.BF16])
    x32 = p.cast(0, P.F32); a32 = p.cast(1, P.F32)
    s = p.add(x32, a32); c = p.cmp(P.OP_GT, s, x32); sel = p.select(c, s, x32); out = p.cast(sel, P.BF16)
    ins = [T(B.BF16, (4, 1, 5)), T(B.BF16, (3, 1))]
    for vid, dt in ((0, B.BF16), (x32, B.F32), (s, B.F32), (c, B.BOOL), (sel, B.F32), (out, B.BF16)):
        t = B.relay_infer_ewise(p.arrays(), ins, vid)
        assert t.dtype == dt and B._shape(t) == (4, 3, 5)
    # literals: a float literal is a rank-0 f32 tensor (Type-Float-Literal); it broadcasts everywhere
    q = P.Program([P.F32]); k = q.const(2.0); r = q.mul(0, k)
    assert B._shape(B.relay_infer_ewise(q.arrays(), [T(B.F32, ())], r)) == ()


def test_infer_ewise_rejections():
    def bad(prog, ins, status, value=0):
        with pytest.raises(B.RelayError) as e:
            B.relay_infer_ewise(prog.arrays(), ins, value)
        assert e.value.status_name == status, str(e.value)
    f = [T(B.F32, (3,)), T(B.BF16, (3,))]
    p = P.Program([P.F32, P.BF16]); p.emit(P.OP_ADD, 0, 1, dtype=P.F32)
    bad(p, f, "ERR_DTYPE")                      # Type-Noncomp-BinaryOp: equal base types
    p = P.Program([P.F32, P.BF16]); p.emit(P.OP_LT, 0, 1, dtype=P.BOOL)
    bad(p, f, "ERR_DTYPE")                      # Type-Comp-BinaryOp: equal base types
    p = P.Program([P.F32, P.F32]); p.emit(P.OP_LT, 0, 1, dtype=P.F32)
    bad(p, [f[0], f[0]], "ERR_DTYPE")           # comparison yields Bool, not f32
    p = P.Program([P.F32]); p.emit(P.OP_SQ, 0, dtype=P.BF16)
    bad(p, [f[0]], "ERR_DTYPE")                 # Type-UnaryOp keeps the type
    p = P.Program([P.F32, P.F32]); p.emit(P.OP_SELECT, 0, 0, 1, dtype=P.F32)
    bad(p, [f[0], f[0]], "ERR_DTYPE")           # select condition must be Bool
    p = P.Program([P.F32]); p.emit(P.OP_ADD, 0, 3, dtype=P.F32)
    bad(p, [f[0]], "ERR_ATTR")                  # names a value that does not exist yet
    p = P.Program([P.F32]); p.emit(99, 0, dtype=P.F32)
    bad(p, [f[0]], "ERR_ATTR")
    p = P.Program([P.F32, P.F32]); p.add(0, 1)
    bad(p, [T(B.F32, (3, 2)), T(B.F32, (3,))], "ERR_SHAPE")   # (3,2) vs (3,) does not broadcast
    p = P.Program([P.I32, P.I32]); p.emit(P.OP_ADD, 0, 1, dtype=P.I32)
    bad(p, [T(B.I32, (3,)), T(B.I32, (3,))], "ERR_DTYPE")      # integer arithmetic not defined here
    p = P.Program([P.F32]); p.add(0, 0)
    bad(p, [f[0]], "ERR_ATTR", value=7)


# ---- reduce / stack / lstm ------------------------------------------------------------------------------
def test_infer_reduce_against_oracle_rule():
    shape = (4, 1, 6, 3)
    for mask in range(1, 16):
        axes = [d for d in range(4) if mask >> d & 1]
        for keep in (False, True):
            out = B.relay_infer_reduce(T(B.BF16, shape), B.RED_SUM, mask, keep)
            assert B._shape(out) == oracle.reduce_shape(shape, axes, keep) and out.dtype == B.F32
    assert B.relay_infer_reduce(T(B.BF16, shape), B.RED_ARGMAX, 8, False).dtype == B.I64
    assert B._shape(B.relay_infer_reduce(T(B.BF16, shape), B.RED_NONE, 0, False)) == shape
    for mask, status in ((0, "ERR_ATTR"), (16, "ERR_ATTR"), (-1, "ERR_ATTR")):
        with pytest.raises(B.RelayError) as e:
            B.relay_infer_reduce(T(B.BF16, shape), B.RED_SUM, mask, False)
        assert e.value.status_name == status
    with pytest.raises(B.RelayError) as e:
        B.relay_infer_reduce(T(B.BF16, (4, 0)), B.RED_MAX, 2, False)
    assert e.value.status_name == "ERR_SHAPE"


def test_infer_stack_tensor_literal_rule():
    # Type-Tensor-Literal: m tensors of Shape(d1..dn) -> Shape(m, d1..dn), same base type
    for m, s in itertools.product((1, 2, 7), [(), (3,), (2, 4), (1, 2, 3, 4, 5)]):
        out = B.relay_infer_stack(T(B.I32, s), m)
        assert B._shape(out) == (m,) + s and out.dtype == B.I32
    with pytest.raises(B.RelayError) as e:
        B.relay_infer_stack(T(B.F32, (1, 2, 3, 4, 5, 6)), 2)
    assert e.value.status_name == "ERR_RANK"
    with pytest.raises(B.RelayError) as e:
        B.relay_infer_stack(T(B.F32, (2,)), 0)
    assert e.value.status_name == "ERR_SHAPE"


def test_infer_lstm_relation():
    h, c = B.relay_infer_lstm(T(B.BF16, (128, 64, 1024)), T(B.BF16, (1024, 4096)), T(B.BF16, (1024, 4096)))
    assert B._shape(h) == (128, 64, 1024) and B._shape(c) == (64, 1024) and h.dtype == c.dtype == B.F32
    h, c = B.relay_infer_lstm(T(B.BF16, (5, 3, 20)), T(B.BF16, (20, 96)), T(B.BF16, (24, 96)))
    assert B._shape(h) == (5, 3, 24)
    bad = [((5, 3, 20), (21, 96), (24, 96), B.BF16, "ERR_SHAPE"), ((5, 3, 20), (20, 95), (24, 96), B.BF16, "ERR_SHAPE"),
           ((5, 3, 20), (20, 96), (24, 100), B.BF16, "ERR_SHAPE"), ((5, 3, 20), (20, 96), (24, 96), B.F32, "ERR_DTYPE"),
           ((3, 20), (20, 96), (24, 96), B.BF16, "ERR_RANK")]
    for xs, wi, wh, dt, status in bad:
        with pytest.raises(B.RelayError) as e:
            B.relay_infer_lstm(T(dt, xs), T(B.BF16, wi), T(B.BF16, wh))
        assert e.value.status_name == status


def test_workspace_queries_are_host_only():
    import torch
    x, w = torch.empty(8, 64), torch.empty(64, 32)
    assert B.relay_workspace_bytes_dense_act(x, w) == 0
    assert B.relay_workspace_bytes_dense_act_grad(x, w) >= 8 * 32 * 4
    xb = torch.empty(4, 2, 8, dtype=torch.bfloat16)
    assert B.relay_workspace_bytes_lstm(xb, torch.empty(8, 16, dtype=torch.bfloat16), torch.empty(4, 16, dtype=torch.bfloat16)) >= 4 * 2 * 16 * 4
    assert B.relay_workspace_bytes_dense_act_grad(x, torch.empty(63, 32)) == 0   # ill-typed -> 0


# ---- loss and parameter update ----------------------------------------------------------------------
def test_infer_softmax_xent_relation_and_rejections():
    for Bn, C in [(1, 10), (64, 1000), (0, 7), (8192, 8192)]:
        for zt, tt in [(B.F32, B.F32), (B.BF16, B.BF16), (B.BF16, B.F32)]:
            out = B.relay_infer_softmax_xent(T(zt, (Bn, C)), T(tt, (Bn, C)))
            assert out.dtype == B.F32 and B._shape(out) == (Bn,)
    cases = [(T(B.F32, (4, 10)), T(B.F32, (4, 9)), "ERR_SHAPE"), (T(B.F32, (4, 10)), T(B.F32, (5, 10)), "ERR_SHAPE"),
             (T(B.F32, (4, 10)), T(B.BF16, (4, 10)), "ERR_DTYPE"), (T(B.I32, (4, 10)), T(B.F32, (4, 10)), "ERR_DTYPE"),
             (T(B.F32, (4, 10, 1)), T(B.F32, (4, 10)), "ERR_RANK"), (T(B.F32, (4,)), T(B.F32, (4,)), "ERR_RANK"),
             (T(B.F32, (4, 0)), T(B.F32, (4, 0)), "ERR_SHAPE"), (T(B.F32, (4, 10), B.NCHW), T(B.F32, (4, 10)), "ERR_LAYOUT")]
    for z, t, status in cases:
        with pytest.raises(B.RelayError) as e:
            B.relay_infer_softmax_xent(z, t)
        assert e.value.status_name == status, str(e.value)


def test_sgd_update_descriptor_checks_run_before_any_launch():
    """Descriptor errors are found on the host (no GPU is touched): rank, then dtype, then shape."""
    lib = B.lib()

    def call(params, grads, lr=0.1):
        return lib.relay_sgd_update(B._desc_array(params), B._desc_array(grads), len(params), ctypes.c_float(lr), None)

    ok_p, ok_g = T(B.BF16, (4, 8)), T(B.F32, (4, 8))
    n0 = B.relay_launch_count()
    assert call([], []) == 0                                        # nothing to update
    def status_of(params, grads):
        st = call(params, grads)
        return B.RelayError(st, "").status_name
    assert status_of([ok_p, T(B.F32, (3,))], [ok_g, T(B.F32, (3, 1))]) == "ERR_RANK"
    assert status_of([T(B.I32, (3,))], [T(B.I32, (3,))]) == "ERR_DTYPE"
    assert status_of([T(B.F32, (3,))], [T(B.BF16, (3,))]) == "ERR_DTYPE"       # gradient narrower than the parameter
    assert status_of([ok_p], [T(B.F32, (4, 7))]) == "ERR_SHAPE"
    assert status_of([ok_p], [ok_g]) == "ERR_NULL"                                # descriptors without data
    assert B.relay_launch_count() == n0


def test_infer_max_pool2d_counts_windows_and_rejects_bad_windows():
    for H, W, kh, kw, sh, sw in itertools.product((1, 4, 7), (2, 5, 8), (1, 2, 3), (1, 2), (1, 2, 3), (1, 2)):
        x = T(B.BF16, (2, 3, H, W), B.NCHW)
        if kh > H or kw > W:
            with pytest.raises(B.RelayError) as e:
                B.relay_infer_max_pool2d(x, kh, kw, sh, sw)
            assert e.value.status_name == "ERR_ATTR"
            continue
        out = B.relay_infer_max_pool2d(x, kh, kw, sh, sw)
        P = len([p for p in range(H) if p * sh + kh <= H])
        Q = len([q for q in range(W) if q * sw + kw <= W])
        assert B._shape(out) == (2, 3, P, Q) and out.dtype == B.BF16
    for x, k, status in [(T(B.F32, (2, 3, 4)), (2, 2, 2, 2), "ERR_RANK"), (T(B.I32, (1, 1, 4, 4)), (2, 2, 2, 2), "ERR_DTYPE"),
                         (T(B.F32, (1, 1, 4, 4)), (0, 2, 2, 2), "ERR_ATTR"), (T(B.F32, (1, 1, 4, 4)), (2, 2, 2, -1), "ERR_ATTR")]:
        with pytest.raises(B.RelayError) as e:
            B.relay_infer_max_pool2d(x, *k)
        assert e.value.status_name == status
