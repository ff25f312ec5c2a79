"""GPU parity: conv2d anchor (+bias +activation) with its gradient group, and the LSTM sequence."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_1810_00952_b200 import binding as B
from relay_workloads import inputs as I

from parity import Guarded, assert_bf16, assert_f32, to_np, workspace

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
F64 = 5


def conv_fwd(x, w, b, stride, pad, act):
    d = B.relay_infer_conv2d(B.desc(x, B.NCHW), B.desc(w, B.OIHW), stride, pad)
    y = Guarded(B._shape(d), x.dtype, DEV)
    ws = workspace(B.relay_workspace_bytes_conv2d_act(x, w, stride, pad), DEV)
    B.relay_fused_conv2d_act(x.to(DEV), w.to(DEV), None if b is None else b.to(DEV), stride, pad, act, y.t, ws)
    torch.cuda.synchronize()
    return y.check()


def conv_grad(x, w, y, dy, stride, pad, act, want_dx=True, want_db=True):
    dx = Guarded(tuple(x.shape), x.dtype, DEV) if want_dx else None
    dw = Guarded(tuple(w.shape), x.dtype, DEV)
    db = Guarded((w.shape[0],), torch.float32, DEV) if want_db else None
    ws = workspace(B.relay_workspace_bytes_conv2d_act_grad(x, w, stride, pad), DEV)
    B.relay_fused_conv2d_act_grad(x.to(DEV), w.to(DEV), y.to(DEV), dy.to(DEV), stride, pad, act, dx.t if dx else None, dw.t,
                                  db.t if db else None, ws)
    torch.cuda.synchronize()
    return (dx.check() if dx else None), dw.check(), (db.check() if db else None)


@pytest.mark.parametrize("N,C,H,W,O,R,stride,pad", [(2, 3, 7, 6, 4, 3, 1, 1), (1, 5, 9, 9, 3, 3, 2, 1), (2, 2, 8, 5, 6, 5, 1, 0),
                                                     (1, 4, 6, 6, 2, 1, 1, 0), (3, 8, 10, 12, 16, 3, 2, 2), (1, 1, 1, 1, 1, 3, 1, 1),
                                                     # several tiles of the general tier along every GEMM axis, ragged tails, a split
                                                     # weight-gradient sum with a short last slice: 70 output channels (two tiles),
                                                     # LeNet's second conv (N*P*Q = 4096 over 37 slices), a 7x7 window at stride 3
                                                     (3, 7, 11, 13, 70, 3, 2, 1), (64, 20, 12, 12, 50, 5, 1, 0), (2, 4, 23, 19, 3, 7, 3, 3),
                                                     (5, 3, 33, 17, 5, 1, 1, 0)])
@pytest.mark.parametrize("tdt", [torch.float32, torch.bfloat16])
def test_conv_small_shapes_forward_and_gradient(N, C, H, W, O, R, stride, pad, tdt):
    t = I.cfg4_conv(N, C, H, W, O, R, R, dtype=tdt, salt=H)
    act = B.ACT_RELU
    y = conv_fwd(t["x"], t["w"], t["b"], stride, pad, act)
    xo, wo, bo = (I.as_f64(t[k]) for k in ("x", "w", "b"))
    want = oracle.conv2d_act(xo, wo, bo, stride, pad, act, F64)
    chk = assert_f32 if tdt == torch.float32 else assert_bf16
    chk(y, want, what="y")
    dy = I.normal(4, 3, tuple(y.shape), 1.0, tdt, salt=H)
    dx, dw, db = conv_grad(t["x"], t["w"], y, dy, stride, pad, act)
    odx, odw, odb = oracle.conv2d_act_grad(xo, wo, to_np(y), I.as_f64(dy), stride, pad, act, F64, F64, F64,
                                           dz_dtype=oracle.F32 if tdt == torch.float32 else oracle.BF16)
    chk(dx, odx, what="dx"); chk(dw, odw, what="dw")
    (assert_f32 if tdt == torch.float32 else (lambda g, o, what: assert_bf16(g, o, stored_bf16=False, what=what)))(db, odb, what="db")


@pytest.mark.parametrize("N,C,H,W,O", [(2, 64, 28, 28, 64), (2, 128, 16, 16, 128), (3, 128, 12, 24, 256), (1, 128, 56, 56, 128),
                                       (3, 256, 16, 16, 256)])
def test_conv_reduced_config_bf16_3x3(N, C, H, W, O):
    """Configuration 4's structure (3x3, stride 1, pad 1, NCHW/OIHW, bf16) at reduced sizes; the shapes
    with C and O multiples of 128 take the implicit-GEMM tensor-core kernels (several tiles, batch
    slices of unequal size), the first one the general SIMT tier."""
    t = I.cfg4_conv(N, C, H, W, O, salt=C + W)
    y = conv_fwd(t["x"], t["w"], t["b"], 1, 1, B.ACT_RELU)
    xo, wo, bo, dyo = (I.as_f64(t[k]) for k in ("x", "w", "b", "dy"))
    assert_bf16(y, oracle.conv2d_act(xo, wo, bo, 1, 1, B.ACT_RELU, F64), what="y")
    dx, dw, db = conv_grad(t["x"], t["w"], y, t["dy"], 1, 1, B.ACT_RELU)
    odx, odw, odb = oracle.conv2d_act_grad(xo, wo, to_np(y), dyo, 1, 1, B.ACT_RELU, F64, F64, F64, dz_dtype=oracle.BF16)
    assert_bf16(dx, odx, what="dx"); assert_bf16(dw, odw, what="dw"); assert_bf16(db, odb, stored_bf16=False, what="db")
    # tanh epilogue and no bias / no dx / no db through the same kernels
    y2 = conv_fwd(t["x"], t["w"], None, 1, 1, B.ACT_TANH)
    assert_bf16(y2, oracle.conv2d_act(xo, wo, None, 1, 1, B.ACT_TANH, F64), what="y tanh")
    _, dw2, _ = conv_grad(t["x"], t["w"], y2, t["dy"], 1, 1, B.ACT_TANH, want_dx=False, want_db=False)
    _, odw2, _ = oracle.conv2d_act_grad(xo, wo, to_np(y2), dyo, 1, 1, B.ACT_TANH, F64, F64, F64, want_dx=False, want_db=False,
                                        dz_dtype=oracle.BF16)
    assert_bf16(dw2, odw2, what="dw tanh")


@pytest.mark.parametrize("N,C,H,W,O,R,stride,pad,tdt", [(2, 3, 7, 6, 4, 3, 1, 1, torch.float32), (1, 5, 9, 9, 3, 3, 2, 1, torch.bfloat16),
                                                         (2, 128, 16, 16, 128, 3, 1, 1, torch.bfloat16),      # tensor-core instance
                                                         (3, 128, 12, 24, 256, 3, 1, 1, torch.bfloat16),
                                                         # two-SM kernel storing NHWC tiles itself: 3 and 1 blocks of 32 pixels
                                                         (76, 256, 12, 8, 256, 3, 1, 1, torch.bfloat16),
                                                         (80, 256, 4, 8, 256, 3, 1, 1, torch.bfloat16)])
def test_conv_nhwc_tagged_activations(N, C, H, W, O, R, stride, pad, tdt):
    """Layout-tagged activations: x, y, dy, dx are NHWC tensors of shape (N,H,W,C); the values are those of the NCHW
    definition (the oracle is given the same tensors permuted on the host)."""
    t = I.cfg4_conv(N, C, H, W, O, R, R, dtype=tdt, salt=H + 1)
    act = B.ACT_RELU
    x_nhwc = t["x"].permute(0, 2, 3, 1).contiguous()
    d = B.relay_infer_conv2d(B.desc(x_nhwc, B.NHWC), B.desc(t["w"], B.OIHW), stride, pad)
    assert d.layout == B.NHWC and B._shape(d)[3] == O
    y = Guarded(B._shape(d), tdt, DEV)
    ws = workspace(B.relay_workspace_bytes_conv2d_act(x_nhwc, t["w"], stride, pad, layout=B.NHWC), DEV)
    B.relay_fused_conv2d_act(x_nhwc.to(DEV), t["w"].to(DEV), t["b"].to(DEV), stride, pad, act, y.t, ws, layout=B.NHWC)
    torch.cuda.synchronize()
    yg = y.check()
    xo, wo, bo = (I.as_f64(t[k]) for k in ("x", "w", "b"))
    want = oracle.conv2d_act(xo, wo, bo, stride, pad, act, F64)                     # NCHW
    chk = assert_f32 if tdt == torch.float32 else assert_bf16
    chk(yg.permute(0, 3, 1, 2), want, what="y")
    dy = I.normal(4, 3, tuple(want.shape), 1.0, tdt, salt=H + 1)                      # NCHW values
    dy_nhwc = dy.permute(0, 2, 3, 1).contiguous()
    dx, dw, db = Guarded(tuple(x_nhwc.shape), tdt, DEV), Guarded(tuple(t["w"].shape), tdt, DEV), Guarded((O,), torch.float32, DEV)
    ws = workspace(B.relay_workspace_bytes_conv2d_act_grad(x_nhwc, t["w"], stride, pad, layout=B.NHWC), DEV)
    B.relay_fused_conv2d_act_grad(x_nhwc.to(DEV), t["w"].to(DEV), yg.to(DEV), dy_nhwc.to(DEV), stride, pad, act, dx.t, dw.t, db.t, ws,
                                  layout=B.NHWC)
    torch.cuda.synchronize()
    odx, odw, odb = oracle.conv2d_act_grad(xo, wo, to_np(yg.permute(0, 3, 1, 2)), I.as_f64(dy), stride, pad, act, F64, F64, F64,
                                           dz_dtype=oracle.F32 if tdt == torch.float32 else oracle.BF16)
    chk(dx.check().permute(0, 3, 1, 2), odx, what="dx"); chk(dw.check(), odw, what="dw")
    (assert_f32 if tdt == torch.float32 else (lambda g, o, what: assert_bf16(g, o, stored_bf16=False, what=what)))(db.check(), odb, what="db")
    # an NCHW-tagged y for an NHWC x is a layout error; nothing is written
    bad = torch.full(B._shape(d), 5.0, dtype=tdt, device=DEV)
    at = B.Conv2dAttrs(stride, pad, 1, 1)
    xd, wd, yd = B.desc(x_nhwc.to(DEV), B.NHWC), B.desc(t["w"].to(DEV), B.OIHW), B.desc(bad, B.NCHW)
    with pytest.raises(B.RelayError) as e:
        B._check(B.lib().relay_fused_conv2d_act(ctypes.byref(xd), ctypes.byref(wd), None, ctypes.byref(at), int(act), ctypes.byref(yd),
                                                 None, 0, None))
    assert e.value.status_name == "ERR_LAYOUT" and bool((bad == 5.0).all())


def test_conv_rejections():
    x = torch.zeros(2, 3, 8, 8, dtype=torch.bfloat16, device=DEV); w = torch.zeros(5, 3, 3, 3, dtype=torch.bfloat16, device=DEV)
    y = torch.zeros(2, 5, 8, 8, dtype=torch.bfloat16, device=DEV)
    n0 = B.relay_launch_count()
    with pytest.raises(B.RelayError) as e:
        B.relay_fused_conv2d_act(x, w, None, 1, 1, B.ACT_RELU, torch.zeros(2, 5, 8, 7, dtype=torch.bfloat16, device=DEV))
    assert e.value.status_name == "ERR_SHAPE"
    with pytest.raises(B.RelayError) as e:
        B.relay_fused_conv2d_act(x, w, torch.zeros(4, device=DEV), 1, 1, B.ACT_RELU, y)
    assert e.value.status_name == "ERR_SHAPE"
    with pytest.raises(B.RelayError) as e:
        B.relay_fused_conv2d_act(x, w.float(), None, 1, 1, B.ACT_RELU, y)
    assert e.value.status_name == "ERR_DTYPE"
    assert B.relay_launch_count() == n0


def test_conv_full_size_sampled():
    """Configuration 4 at full size.  The forward / dX kernels walk (image, band of rows) tiles in rounds over the SM
    pairs, the last round in another item shape, a schedule that exists only at this size: the oracle recomputes two
    random output rows (all channels) of EVERY image of y and dx plus images 0 and 31 whole, four 8 x 8 channel
    blocks of dW at the corners of its (o, c) range (all taps, all 32 images) and db of those channels, from the
    GPU's stored y; every output is also screened for elements that no tile wrote (Guarded)."""
    t = I.cfg4_conv()
    y = conv_fwd(t["x"], t["w"], t["b"], 1, 1, B.ACT_RELU)
    dx, dw, db = conv_grad(t["x"], t["w"], y, t["dy"], 1, 1, B.ACT_RELU)
    wo, bo = I.as_f64(t["w"]), I.as_f64(t["b"])
    for n in (0, 31):
        xo = I.as_f64(t["x"][n:n + 1])
        assert_bf16(y[n:n + 1], oracle.conv2d_act(xo, wo, bo, 1, 1, B.ACT_RELU, F64), what=f"y image {n}")
        odx, _, _ = oracle.conv2d_act_grad(xo, wo, to_np(y[n:n + 1]), I.as_f64(t["dy"][n:n + 1]), 1, 1, B.ACT_RELU, F64, F64, F64,
                                           want_dw=False, want_db=False)
        assert_bf16(dx[n:n + 1], odx, what=f"dx image {n}")
    # an output row depends on the three input rows around it: the oracle is run on that band (its zero padding is the
    # real one at the image's edge, elsewhere the band's outer rows are not used)
    rng = np.random.default_rng(17)
    H = t["x"].shape[2]
    got_y, want_y, got_dx, want_dx = [], [], [], []
    for n in range(t["x"].shape[0]):
        for h in {int(v) for v in rng.choice(H, 2, replace=False)} | ({0, H - 1} if n == 7 else set()):
            lo, hi = max(h - 1, 0), min(h + 2, H)
            xo = I.as_f64(t["x"][n:n + 1, :, lo:hi])
            want_y.append(oracle.conv2d_act(xo, wo, bo, 1, 1, B.ACT_RELU, F64)[0, :, h - lo]); got_y.append(to_np(y[n, :, h]))
            odx, _, _ = oracle.conv2d_act_grad(xo, wo, to_np(y[n:n + 1, :, lo:hi]), I.as_f64(t["dy"][n:n + 1, :, lo:hi]), 1, 1,
                                               B.ACT_RELU, F64, F64, F64, want_dw=False, want_db=False)
            want_dx.append(odx[0, :, h - lo]); got_dx.append(to_np(dx[n, :, h]))
    assert_bf16(np.stack(got_y), np.stack(want_y), what="y rows of every image")
    assert_bf16(np.stack(got_dx), np.stack(want_dx), what="dx rows of every image")
    for oc, ic in [(slice(0, 8), slice(0, 8)), (slice(0, 8), slice(248, 256)), (slice(248, 256), slice(0, 8)),
                   (slice(248, 256), slice(248, 256)), (slice(120, 128), slice(128, 136))]:
        _, odw, odb = oracle.conv2d_act_grad(I.as_f64(t["x"][:, ic]), wo[oc, ic], to_np(y[:, oc]), I.as_f64(t["dy"][:, oc]), 1, 1,
                                             B.ACT_RELU, F64, F64, F64, want_dx=False)
        assert_bf16(dw[oc, ic], odw, what=f"dw {oc} {ic}")
        assert_bf16(db[oc], odb, stored_bf16=False, what="db")
    # the same tensors tagged NHWC: the kernels store pixel-major tiles of the same accumulators, so y, dx and dw agree
    # bit for bit with the NCHW call; db is summed in another order
    nhwc = lambda a: a.permute(0, 2, 3, 1).contiguous().to(DEV)
    xh, dyh = nhwc(t["x"]), nhwc(t["dy"])
    wd, bd = t["w"].to(DEV), t["b"].to(DEV)
    yh = Guarded(tuple(dyh.shape), torch.bfloat16, DEV)
    B.relay_fused_conv2d_act(xh, wd, bd, 1, 1, B.ACT_RELU, yh.t, workspace(B.relay_workspace_bytes_conv2d_act(xh, wd, 1, 1, layout=B.NHWC), DEV),
                             layout=B.NHWC)
    torch.cuda.synchronize()
    assert torch.equal(yh.check().permute(0, 3, 1, 2), y)
    dxh, dwh, dbh = Guarded(tuple(xh.shape), torch.bfloat16, DEV), Guarded(tuple(wd.shape), torch.bfloat16, DEV), Guarded((wd.shape[0],), torch.float32, DEV)
    B.relay_fused_conv2d_act_grad(xh, wd, yh.t, dyh, 1, 1, B.ACT_RELU, dxh.t, dwh.t, dbh.t,
                                  workspace(B.relay_workspace_bytes_conv2d_act_grad(xh, wd, 1, 1, layout=B.NHWC), DEV), layout=B.NHWC)
    torch.cuda.synchronize()
    B.relay_poll_status()
    assert torch.equal(dxh.check().permute(0, 3, 1, 2), dx) and torch.equal(dwh.check(), dw)
    assert_bf16(dbh.check()[oc], odb, stored_bf16=False, what="db nhwc")


# ---- LSTM -------------------------------------------------------------------------------------------
def lstm(t):
    T_, Bn, _ = t["x"].shape
    H = t["w_hh"].shape[0]
    h_all = Guarded((T_, Bn, H), torch.float32, DEV)
    c_fin = Guarded((Bn, H), torch.float32, DEV)
    ws = workspace(B.relay_workspace_bytes_lstm(t["x"], t["w_ih"], t["w_hh"]), DEV)
    B.relay_lstm_cell_seq(*(t[k].to(DEV) for k in ("x", "w_ih", "w_hh", "b", "h0", "c0")), h_all.t, c_fin.t, ws)
    B.relay_poll_status()
    return h_all.check(), c_fin.check()


@pytest.mark.parametrize("T,Bn,In,H", [(1, 1, 8, 8), (5, 3, 20, 24), (8, 16, 128, 256), (3, 70, 40, 72), (12, 9, 64, 128)])
def test_lstm_small_shapes(T, Bn, In, H):
    t = I.cfg5_lstm(T, Bn, In, H, salt=T)
    g = torch.Generator().manual_seed(T)
    t["h0"] = torch.randn(Bn, H, generator=g) * 0.3
    t["c0"] = torch.randn(Bn, H, generator=g) * 0.3
    h_all, c_fin = lstm(t)
    oh, oc = oracle.lstm_cell_seq(*(I.as_f64(t[k]) for k in ("x", "w_ih", "w_hh", "b", "h0", "c0")))
    # bf16 GEMM inputs with fp32 accumulation and fp32 state: the bf16-path tolerance, results in f32
    assert_bf16(h_all, oh, stored_bf16=False, what="h_all"); assert_bf16(c_fin, oc, stored_bf16=False, what="c_final")
    assert bool((h_all.abs() < 1).all())


def test_lstm_full_size_sampled_batch_rows():
    """Configuration 5 at full size; batch rows are independent, so the oracle runs 3 of the 64
    rows through all 128 steps."""
    t = I.cfg5_lstm()
    h_all, c_fin = lstm(t)
    rows = [0, 31, 63]
    sub = {k: I.as_f64(t[k]) for k in ("w_ih", "w_hh", "b")}
    oh, oc = oracle.lstm_cell_seq(I.as_f64(t["x"][:, rows]), sub["w_ih"], sub["w_hh"], sub["b"], I.as_f64(t["h0"][rows]), I.as_f64(t["c0"][rows]))
    assert_bf16(h_all[:, rows], oh, stored_bf16=False, what="h_all"); assert_bf16(c_fin[rows], oc, stored_bf16=False, what="c_final")
    assert bool((h_all.abs() < 1).all()) and bool((c_fin.abs() <= 128).all())


def test_lstm_rejections():
    t = {k: v.to(DEV) for k, v in I.cfg5_lstm(2, 2, 8, 8).items()}
    h_all = torch.empty(2, 2, 8, device=DEV); c = torch.empty(2, 8, device=DEV)
    ws = workspace(B.relay_workspace_bytes_lstm(t["x"], t["w_ih"], t["w_hh"]), DEV)
    with pytest.raises(B.RelayError) as e:
        B.relay_lstm_cell_seq(t["x"], t["w_ih"], t["w_hh"], t["b"][:31].contiguous(), t["h0"], t["c0"], h_all, c, ws)
    assert e.value.status_name == "ERR_SHAPE"
    with pytest.raises(B.RelayError) as e:
        B.relay_lstm_cell_seq(t["x"], t["w_ih"], t["w_hh"], t["b"], t["h0"].bfloat16(), t["c0"], h_all, c, ws)
    assert e.value.status_name == "ERR_DTYPE"
    with pytest.raises(B.RelayError) as e:
        B.relay_lstm_cell_seq(t["x"], t["w_ih"], t["w_hh"], t["b"], t["h0"], t["c0"], h_all, c, None)
    assert e.value.status_name == "ERR_WORKSPACE"


def test_lstm_phase_cycle_report_leaves_results_unchanged():
    """The instrumented call returns the same h_all / c_final bit for bit and plausible counts (phases within the loop)."""
    t = I.cfg5_lstm(6, 16, 128, 256, salt=3)
    d = {k: v.to(DEV) for k, v in t.items()}
    h1, c1 = lstm(t)
    h2, c2 = torch.empty_like(h1), torch.empty_like(c1)
    ws = workspace(B.relay_workspace_bytes_lstm(d["x"], d["w_ih"], d["w_hh"]), DEV)
    cyc = torch.full((8,), -1, dtype=torch.int64, device=DEV)
    B.relay_debug_lstm_phase_cycles(d["x"], d["w_ih"], d["w_hh"], d["b"], d["h0"], d["c0"], h2, c2, ws, cyc)
    B.relay_poll_status()
    assert torch.equal(h1, h2) and torch.equal(c1, c2)
    c = cyc.cpu().tolist()
    assert c[7] == 6 and c[0] > 0 and all(0 <= v <= c[0] for v in c[1:7])
