"""GPU parity: dense anchor (+bias +activation) and its gradient group against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_1810_00952_b200 import binding as B
from relay_workloads import inputs as I

from parity import Guarded, assert_bf16, assert_f32, to_np, workspace

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
ACTS = (B.ACT_NONE, B.ACT_RELU, B.ACT_TANH, B.ACT_SIGMOID)
F64 = 5


def run_fwd(x, w, b, act):
    y = Guarded((x.shape[0], w.shape[1]), x.dtype, DEV)
    ws = workspace(B.relay_workspace_bytes_dense_act(x, w), DEV)
    B.relay_fused_dense_act(x.to(DEV), w.to(DEV), None if b is None else b.to(DEV), act, y.t, ws)
    torch.cuda.synchronize()
    return y.check()


def run_grad(x, w, y, dy, act, want_dx=True, want_db=True):
    M, K = x.shape
    N = w.shape[1]
    dx = Guarded((M, K), x.dtype, DEV) if want_dx else None
    dw = Guarded((K, N), x.dtype, DEV)
    db = Guarded((N,), torch.float32, DEV) if want_db else None
    ws = workspace(B.relay_workspace_bytes_dense_act_grad(x, w), DEV)
    B.relay_fused_dense_act_grad(x.to(DEV), w.to(DEV), y.to(DEV), dy.to(DEV), act, dx.t if dx else None, dw.t,
                                 db.t if db else None, ws)
    torch.cuda.synchronize()
    return (dx.check() if dx else None), dw.check(), (db.check() if db else None)


@pytest.mark.parametrize("act", ACTS)
def test_tiny_mlp_layer_fp32_forward_and_gradient(act):
    """Configuration 1: x[8,64] W[64,32] b[32] dy[8,32], fp32, max relative error <= 1e-4."""
    t = I.cfg1_tiny_mlp()
    y = run_fwd(t["x"], t["w"], t["b"], act)
    xo, wo, bo, dyo = (I.as_f64(t[k]) for k in ("x", "w", "b", "dy"))
    assert_f32(y, oracle.dense_act(xo, wo, bo, act, F64), what="y")
    if act == B.ACT_RELU:
        z = xo @ wo + bo
        assert bool((y.cpu()[torch.from_numpy(z < -1e-3)] == 0).all())      # exact zeros stay exact
    dx, dw, db = run_grad(t["x"], t["w"], y, t["dy"], act)
    odx, odw, odb = oracle.dense_act_grad(xo, wo, to_np(y), dyo, act, F64, F64, F64, dz_dtype=oracle.F32)   # the saved y decides the mask
    assert_f32(dx, odx, what="dx"); assert_f32(dw, odw, what="dw"); assert_f32(db, odb, what="db")


@pytest.mark.parametrize("M,K,N", [(1, 1, 1), (37, 53, 29), (130, 70, 200), (64, 64, 64), (5, 300, 8),
                                   (128, 64, 256), (200, 136, 264), (384, 512, 320), (72, 1032, 520),
                                   (1100, 24, 1100)])      # SIMT kernel with its 64-row tile (a grid that fills the SMs)
@pytest.mark.parametrize("tdt", [torch.float32, torch.bfloat16])
def test_odd_shapes_forward_and_gradient(M, K, N, tdt):
    t = I.cfg1_tiny_mlp(M, K, N, salt=M)
    x, w, b, dy = (t[k].to(tdt) for k in ("x", "w", "b", "dy"))
    w = (w / np.sqrt(K)).to(tdt)
    act = B.ACT_TANH
    y = run_fwd(x, w, b, act)
    xo, wo, bo, dyo = (v.double().numpy() for v in (x, w, b, dy))
    chk = assert_f32 if tdt == torch.float32 else assert_bf16
    chk(y, oracle.dense_act(xo, wo, bo, act, F64), what="y")
    dx, dw, db = run_grad(x, w, y, dy, act)
    # dZ is a value of the operand type (stored in bf16 / fp32 before the contractions read it)
    odx, odw, odb = oracle.dense_act_grad(xo, wo, to_np(y), dyo, act, F64, F64, F64,
                                          dz_dtype=oracle.F32 if tdt == torch.float32 else oracle.BF16)
    chk(dx, odx, what="dx"); chk(dw, odw, what="dw")
    if tdt == torch.float32:
        assert_f32(db, odb, what="db")
    else:
        assert_bf16(db, odb, stored_bf16=False, what="db")


def test_optional_outputs_no_bias_and_f32_bias():
    t = I.cfg3_mlp(batch=96, width=128, layers=1)
    x, w, dy = t["x"], t["w0"], t["dy"]
    y = run_fwd(x, w, None, B.ACT_RELU)
    xo, wo, dyo = (I.as_f64(v) for v in (x, w, dy))
    assert_bf16(y, oracle.dense_act(xo, wo, None, B.ACT_RELU, F64))
    bias32 = torch.linspace(-1, 1, 128)
    y2 = run_fwd(x, w, bias32, B.ACT_NONE)
    assert_bf16(y2, oracle.dense_act(xo, wo, bias32.double().numpy(), B.ACT_NONE, F64))
    dx, dw, db = run_grad(x, w, y, dy, B.ACT_RELU, want_dx=False, want_db=False)
    assert dx is None and db is None
    _, odw, _ = oracle.dense_act_grad(xo, wo, to_np(y), dyo, B.ACT_RELU, F64, F64, F64)
    assert_bf16(dw, odw)


@pytest.mark.parametrize("lead,M,K,N,tdt", [((3,), 8, 64, 32, torch.float32), ((2, 5), 24, 72, 40, torch.bfloat16),
                                            ((4,), 128, 256, 512, torch.bfloat16), ((0,), 8, 16, 8, torch.float32)])
def test_leading_batch_axes(lead, M, K, N, tdt):
    """Batching adds a leading axis to every tensor of the program (Section 5.2): the oracle runs the dense anchor
    and its gradient group once per batch element; the partials of the shared w and b add up over the batch."""
    nb = int(np.prod(lead))
    t = I.cfg1_tiny_mlp(max(nb * M, 1), K, N, salt=77)
    w, b = (t["w"] / np.sqrt(K)).to(tdt), t["b"].to(tdt)
    x = t["x"][:nb * M].to(tdt).reshape(lead + (M, K)); dy = t["dy"][:nb * M].to(tdt).reshape(lead + (M, N))
    y = Guarded(lead + (M, N), tdt, DEV)
    B.relay_fused_dense_act(x.to(DEV), w.to(DEV), b.to(DEV), B.ACT_TANH, y.t, None)
    dx, dw, db = Guarded(lead + (M, K), tdt, DEV), Guarded((K, N), tdt, DEV), Guarded((N,), torch.float32, DEV)
    ws = workspace(B.relay_workspace_bytes_dense_act_grad(x, w), DEV)
    B.relay_fused_dense_act_grad(x.to(DEV), w.to(DEV), y.t, dy.to(DEV), B.ACT_TANH, dx.t, dw.t, db.t, ws)
    torch.cuda.synchronize()
    yg, dxg, dwg, dbg = y.check(), dx.check(), dw.check(), db.check()
    wo, bo = w.double().numpy(), b.double().numpy()
    xe, dye, yge = x.reshape(nb, M, K), dy.reshape(nb, M, N), yg.reshape(nb, M, N)
    want_y, want_dx = np.zeros((nb, M, N)), np.zeros((nb, M, K))
    want_dw, want_db = np.zeros((K, N)), np.zeros(N)
    dzt = oracle.F32 if tdt == torch.float32 else oracle.BF16
    for e in range(nb):
        xo = xe[e].double().numpy()
        want_y[e] = oracle.dense_act(xo, wo, bo, B.ACT_TANH, F64)
        odx, odw, odb = oracle.dense_act_grad(xo, wo, to_np(yge[e]), dye[e].double().numpy(), B.ACT_TANH, F64, F64, F64, dz_dtype=dzt)
        want_dx[e] = odx; want_dw += odw; want_db += odb
    chk = assert_f32 if tdt == torch.float32 else assert_bf16
    if nb:
        chk(yg.reshape(nb, M, N), want_y, what="y"); chk(dxg.reshape(nb, M, K), want_dx, what="dx")
    chk(dwg, want_dw, what="dw")
    if tdt == torch.float32:
        assert_f32(dbg, want_db, what="db")
    else:
        assert_bf16(dbg, want_db, stored_bf16=False, what="db")
    # a batch axis on y that x does not have is a type error; nothing is written
    bad = torch.full((M, N), 5.0, dtype=tdt, device=DEV)
    if nb:
        with pytest.raises(B.RelayError) as e:
            B.relay_fused_dense_act(x.to(DEV), w.to(DEV), b.to(DEV), B.ACT_TANH, bad, None)
        assert e.value.status_name == "ERR_RANK" and bool((bad == 5.0).all())


def test_three_layer_mlp_chain_reduced_size_group_by_group():
    """Configuration 3's structure at width 256 / batch 192: every group is checked against the
    oracle fed with the GPU's stored inputs of that group (so relu masks are identical)."""
    t = I.cfg3_mlp(batch=192, width=256, layers=3)
    acts = [t["x"]]
    for l in range(3):
        y = run_fwd(acts[-1].to(DEV), t[f"w{l}"], t[f"b{l}"], B.ACT_RELU)
        assert_bf16(y, oracle.dense_act(to_np(acts[-1]), I.as_f64(t[f"w{l}"]), I.as_f64(t[f"b{l}"]), B.ACT_RELU, F64), what=f"y{l}")
        acts.append(y)
    g = t["dy"]
    for l in (2, 1, 0):
        dx, dw, db = run_grad(acts[l], t[f"w{l}"], acts[l + 1], g, B.ACT_RELU)
        odx, odw, odb = oracle.dense_act_grad(to_np(acts[l]), I.as_f64(t[f"w{l}"]), to_np(acts[l + 1]), to_np(g), B.ACT_RELU, F64, F64, F64)
        assert_bf16(dx, odx, what=f"dx{l}"); assert_bf16(dw, odw, what=f"dw{l}"); assert_bf16(db, odb, stored_bf16=False, what=f"db{l}")
        g = dx


def test_dense_rejections_leave_outputs_untouched():
    x = torch.zeros(8, 64, device=DEV); w = torch.zeros(64, 32, device=DEV); y = torch.full((8, 32), 5.0, device=DEV)
    n0 = B.relay_launch_count()
    cases = [(x, torch.zeros(63, 32, device=DEV), None, y, "ERR_SHAPE"), (x, w.bfloat16(), None, y, "ERR_DTYPE"),
             (x, w, torch.zeros(31, device=DEV), y, "ERR_SHAPE"), (x, w, None, torch.zeros(8, 31, device=DEV), "ERR_SHAPE"),
             (x, w, None, y.bfloat16(), "ERR_DTYPE"), (x, w, torch.zeros(32, dtype=torch.bfloat16, device=DEV), y, "ERR_DTYPE")]
    for xx, ww, bb, yy, status in cases:
        with pytest.raises(B.RelayError) as e:
            B.relay_fused_dense_act(xx, ww, bb, B.ACT_RELU, yy)
        assert e.value.status_name == status, str(e.value)
    with pytest.raises(B.RelayError) as e:
        B.relay_fused_dense_act(x, w, None, 9, y)
    assert e.value.status_name == "ERR_ATTR"
    with pytest.raises(B.RelayError) as e:     # gradient group without workspace
        B.relay_fused_dense_act_grad(x, w, y, y.clone(), B.ACT_RELU, torch.empty_like(x), torch.empty_like(w), None, None)
    assert e.value.status_name == "ERR_WORKSPACE"
    torch.cuda.synchronize()
    assert B.relay_launch_count() == n0 and bool((y == 5.0).all())


def test_full_size_mlp_layer_sampled_rows_and_columns():
    """Configuration 3 at full size (4096^3 per contraction, bf16, fp32 accumulate), all three
    layers forward and backward.  The work units of the contraction kernels are 256-row blocks cut into
    column ranges, a schedule that exists only at this size, so the oracle recomputes one row (all columns) in
    EVERY 128-row block of y and dx, one k-row (all columns) in every 128-row block of dW, the block-edge rows,
    and all of db, each from the GPU's stored inputs of that group; every output is also screened for
    elements that no unit wrote (Guarded)."""
    t = I.cfg3_mlp()
    rng = np.random.default_rng(5)
    rows = np.unique(np.concatenate([[0, 127, 128, 255, 256, 4095], np.arange(0, 4096, 128) + rng.integers(0, 128, 32)]))
    assert len(np.unique(rows // 128)) == 32
    acts = [t["x"].to(DEV)]
    for l in range(3):
        acts.append(run_fwd(acts[-1], t[f"w{l}"], t[f"b{l}"], B.ACT_RELU))
        want = oracle.dense_act(to_np(acts[l][rows]), I.as_f64(t[f"w{l}"]), I.as_f64(t[f"b{l}"]), B.ACT_RELU, F64)
        assert_bf16(acts[-1][rows], want, what=f"y{l}")
    g = t["dy"].to(DEV)
    for l in (2, 1, 0):
        dx, dw, db = run_grad(acts[l], t[f"w{l}"], acts[l + 1], g, B.ACT_RELU)
        wo = I.as_f64(t[f"w{l}"])
        odx, _, _ = oracle.dense_act_grad(to_np(acts[l][rows]), wo, to_np(acts[l + 1][rows]), to_np(g[rows]), B.ACT_RELU, F64, F64, F64,
                                          want_dw=False, want_db=False)
        assert_bf16(dx[rows], odx, what=f"dx{l}")
        # dW rows k in `krows`: needs x[:, krows] over the whole batch
        krows = np.unique(np.concatenate([[0, 127, 128, 4095], np.arange(0, 4096, 128) + rng.integers(0, 128, 32)]))
        _, odw, odb = oracle.dense_act_grad(to_np(acts[l][:, krows]), wo[krows], to_np(acts[l + 1]), to_np(g), B.ACT_RELU, F64, F64, F64,
                                            want_dx=False)
        assert_bf16(dw[krows], odw, what=f"dw{l}")
        assert_bf16(db, odb, stored_bf16=False, what=f"db{l}")
        g = dx


def test_two_sm_kernel_ragged_edges_and_half_width_tail_units():
    """A shape the two-SM kernel takes (more 256 x 256 tiles than SMs) with ragged M, N and K and a last
    round that is cut into half-width units; sampled rows (all columns) of y, dx and dW, and all of db."""
    M, K, N = 2600, 136, 3720
    t = I.cfg1_tiny_mlp(M, K, N, salt=77)
    x, w, b, dy = (t[k].bfloat16() for k in ("x", "w", "b", "dy"))
    w = (t["w"] / np.sqrt(K)).bfloat16()
    act = B.ACT_TANH
    y = run_fwd(x, w, b, act)
    xo, wo, bo, dyo = (v.double().numpy() for v in (x, w, b, dy))
    rng = np.random.default_rng(11)
    rows = np.unique(np.concatenate([[0, 127, 128, 255, 256, 2559, 2560, M - 1],
                                     np.minimum(np.arange(0, M, 128) + rng.integers(0, 128, (M + 127) // 128), M - 1)]))
    assert_bf16(y[rows], oracle.dense_act(xo[rows], wo, bo, act, F64), what="y")
    dx, dw, db = run_grad(x, w, y, dy, act)
    yo = to_np(y)
    odx, _, _ = oracle.dense_act_grad(xo[rows], wo, yo[rows], dyo[rows], act, F64, F64, F64, want_dw=False, want_db=False,
                                      dz_dtype=oracle.BF16)
    assert_bf16(dx[rows], odx, what="dx")
    krows = np.unique(np.concatenate([[0, 63, 64, 127, 128, K - 1], rng.integers(0, K, 6)]))
    _, odw, odb = oracle.dense_act_grad(xo[:, krows], wo[krows], yo, dyo, act, F64, F64, F64, want_dx=False, dz_dtype=oracle.BF16)
    assert_bf16(dw[krows], odw, what="dw")
    assert_bf16(db, odb, stored_bf16=False, what="db")


def test_two_sm_kernel_fixed_unit_scheme_on_a_large_ragged_output():
    """An output too large for the kernel's unit list (40 row blocks x 129 column chunks): the fixed scheme runs, whole
    rounds of 256 x 512 units and then 256 x 256 tiles with a split tail.  One sampled row in EVERY 256-row block (all
    columns), so that a unit that is skipped or computed twice with other data shows."""
    M, K, N = 10000, 2048, 16392
    assert B.relay_debug_plan_units(M, N, K, torch.cuda.get_device_properties(0).multi_processor_count) is None
    t = I.cfg1_tiny_mlp(M, K, N, salt=91)
    x, b = t["x"].bfloat16(), t["b"].bfloat16()
    w = (t["w"] / np.sqrt(K)).bfloat16()
    y = run_fwd(x, w, b, B.ACT_RELU)
    rng = np.random.default_rng(13)
    rows = np.unique(np.concatenate([np.arange(0, M, 256) + rng.integers(0, 16, (M + 255) // 256), [255, 256, M - 1]]))
    want = oracle.dense_act(x[rows].double().numpy(), w.double().numpy(), b.double().numpy(), B.ACT_RELU, F64)
    assert_bf16(y[rows], want, what="y")


@pytest.mark.parametrize("M,K,N", [(37, 53, 29), (256, 512, 384), (520, 264, 1032), (8, 64, 32), (1100, 40, 1090)])
@pytest.mark.parametrize("tdt", [torch.float32, torch.bfloat16])
def test_contraction_with_operands_read_transposed(M, K, N, tdt):
    """The contraction as a call of its own, in the three forms the dense groups use (plain, b transposed as in
    dx = dZ w^T, a transposed as in dw = x^T dZ) and with both transposed; results in the operand type and as the
    unrounded fp32 accumulator.  The oracle gets the transposed matrices materialised on the host."""
    t = I.cfg1_tiny_mlp(M, K, N, salt=K)
    a = t["x"].to(tdt)                                   # (M, K)
    b = (t["w"] / np.sqrt(K)).to(tdt)                    # (K, N)
    bias = t["b"].to(tdt)
    ao, bo, biaso = a.double().numpy(), b.double().numpy(), bias.double().numpy()
    chk = assert_f32 if tdt == torch.float32 else assert_bf16
    for ta, tb in ((0, 0), (0, 1), (1, 0), (1, 1)):
        ad = (a.t().contiguous() if ta else a).to(DEV)
        bd = (b.t().contiguous() if tb else b).to(DEV)
        for cdt, act, bb in ((tdt, B.ACT_TANH, bias), (torch.float32, B.ACT_NONE, None)):
            c = Guarded((M, N), cdt, DEV)
            B.relay_contract_act(ad, ta, bd, tb, None if bb is None else bb.to(DEV), act, c.t)
            torch.cuda.synchronize()
            want = oracle.dense_act(ao, bo, None if bb is None else biaso, act, F64)
            if cdt == torch.float32 and tdt == torch.bfloat16:
                assert_bf16(c.check(), want, stored_bf16=False, what=f"c f32 {ta}{tb}")
            else:
                chk(c.check(), want, what=f"c {ta}{tb}")
    # type errors: contraction lengths differ, operand types differ, result of a third type
    n0 = B.relay_launch_count()
    c = torch.full((M, N), 5.0, dtype=tdt, device=DEV)
    for args, status in [((a.to(DEV), 1, b.to(DEV), 0, None, B.ACT_NONE, c), "ERR_SHAPE" if M != K else None),
                         ((a.to(DEV), 0, b.to(DEV).to(torch.float32 if tdt == torch.bfloat16 else torch.bfloat16), 0, None, B.ACT_NONE, c), "ERR_DTYPE"),
                         ((a.to(DEV), 0, b.to(DEV), 0, None, 7, c), "ERR_ATTR"),
                         ((a.to(DEV), 0, b.to(DEV), 0, None, B.ACT_NONE, torch.empty(M, N, dtype=torch.int32, device=DEV)), "ERR_DTYPE")]:
        if status is None:
            continue
        with pytest.raises(B.RelayError) as e:
            B.relay_contract_act(*args)
        assert e.value.status_name == status, str(e.value)
    torch.cuda.synchronize()
    assert B.relay_launch_count() == n0 and bool((c == 5.0).all())
