"""Stream capture: every entry point only enqueues work on the caller's stream (no allocation, no synchronisation,
no work on another stream), so a sequence of calls can be captured into a CUDA graph and replayed.  Each case runs
the calls eagerly, captures the same calls, clears the results, replays the graph and compares bit for bit; the
eager results themselves are checked against the oracle by the parity tests of each group."""
import pytest
import torch

from paper_1810_00952_b200 import binding as B
from relay_workloads import inputs as I
from relay_workloads import program as P

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def dev(d):
    return {k: v.to(DEV) for k, v in d.items()}


def ws_of(*sizes):
    return torch.empty(max(16, *sizes), dtype=torch.uint8, device=DEV)


def capture_and_compare(fn, outs):
    fn()                                          # first use outside the capture (module load, kernel attributes)
    torch.cuda.synchronize()
    B.relay_poll_status()
    want = [o.clone() for o in outs]
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    n0 = B.relay_launch_count()
    with torch.cuda.graph(g, stream=s):
        fn()
    assert B.relay_launch_count() > n0            # the calls did enqueue kernels while capturing
    torch.cuda.synchronize()
    for rep in range(2):
        for o in outs:
            o.fill_(7)
        g.replay()
        torch.cuda.synchronize()
        B.relay_poll_status()
        for a, b in zip(want, outs):
            assert torch.equal(a, b), rep


def test_tiny_fp32_layer_forward_and_gradient():
    t = dev(I.cfg1_tiny_mlp())
    y, dx, dw, db = (torch.empty(s, device=DEV) for s in ((8, 32), (8, 64), (64, 32), (32,)))
    ws = ws_of(B.relay_workspace_bytes_dense_act_grad(t["x"], t["w"]))

    def fn():
        B.relay_fused_dense_act(t["x"], t["w"], t["b"], B.ACT_RELU, y, ws)
        B.relay_fused_dense_act_grad(t["x"], t["w"], y, t["dy"], B.ACT_RELU, dx, dw, db, ws)
    capture_and_compare(fn, [y, dx, dw, db])


def test_bf16_dense_layers_chain():
    t = dev(I.cfg3_mlp(512, 512))
    bf = torch.bfloat16
    ys = [torch.empty(512, 512, dtype=bf, device=DEV) for _ in range(3)]
    dxs = [torch.empty(512, 512, dtype=bf, device=DEV) for _ in range(3)]
    dws = [torch.empty(512, 512, dtype=bf, device=DEV) for _ in range(3)]
    dbs = [torch.empty(512, device=DEV) for _ in range(3)]
    ws = ws_of(B.relay_workspace_bytes_dense_act_grad(t["x"], t["w0"]))

    def fn():
        acts = [t["x"]] + ys
        for l in range(3):
            B.relay_fused_dense_act(acts[l], t[f"w{l}"], t[f"b{l}"], B.ACT_RELU, acts[l + 1], ws)
        g = t["dy"]
        for l in (2, 1, 0):
            B.relay_fused_dense_act_grad(acts[l], t[f"w{l}"], acts[l + 1], g, B.ACT_RELU, dxs[l], dws[l], dbs[l], ws)
            g = dxs[l]
    capture_and_compare(fn, ys + dxs + dws + dbs)


@pytest.mark.parametrize("layout", [B.NCHW, B.NHWC])
def test_conv_tensor_core_instance(layout):
    t = dev(I.cfg4_conv(2, 128, 16, 16, 128))
    if layout == B.NHWC:
        t["x"], t["dy"] = (t[k].permute(0, 2, 3, 1).contiguous() for k in ("x", "dy"))
    y, dx, dw, db = torch.empty_like(t["dy"]), torch.empty_like(t["x"]), torch.empty_like(t["w"]), torch.empty(128, device=DEV)
    ws = ws_of(B.relay_workspace_bytes_conv2d_act(t["x"], t["w"], 1, 1, layout=layout),
               B.relay_workspace_bytes_conv2d_act_grad(t["x"], t["w"], 1, 1, layout=layout))

    def fn():
        B.relay_fused_conv2d_act(t["x"], t["w"], t["b"], 1, 1, B.ACT_TANH, y, ws, layout=layout)
        B.relay_fused_conv2d_act_grad(t["x"], t["w"], y, t["dy"], 1, 1, B.ACT_TANH, dx, dw, db, ws, layout=layout)
    capture_and_compare(fn, [y, dx, dw, db])


def test_fused_elementwise_and_reduce_groups():
    t = dev(I.cfg2_ewise(512, 1024))
    out, dx = torch.empty_like(t["x"]), torch.empty_like(t["x"])
    da, db = torch.empty(1024, device=DEV), torch.empty(1, 1024, device=DEV)
    fwd_prog, fwd_outs = P.tanh_affine_residual_fwd(P.BF16)
    grad_prog, ids = P.tanh_affine_residual_grad(P.BF16)
    grad_specs = [(ids[0], B.RED_NONE, 0, 0), (ids[1], B.RED_SUM, 1, 0), (ids[2], B.RED_SUM, 1, 1)]
    ins = [t["dout"], t["x"], t["a"], t["b"]]
    ws = ws_of(B.relay_workspace_bytes_reduce(ins, grad_specs))

    def fn():
        B.relay_fused_ewise(fwd_prog.arrays(), [t["x"], t["a"], t["b"]], fwd_outs, [out])
        B.relay_fused_reduce(grad_prog.arrays(), ins, grad_specs, [dx, da, db], ws)
    capture_and_compare(fn, [out, dx, da, db])


def test_lstm_sequence_and_its_gradient_program():
    """Both persistent kernels are cooperative launches; they are captured as such."""
    T, Bn, In, H = 6, 16, 128, 256
    t = dev(I.cfg5_lstm(T, Bn, In, H))
    f32, bf = torch.float32, torch.bfloat16
    h_all, c = torch.empty(T, Bn, H, device=DEV), torch.empty(Bn, H, device=DEV)
    dh_all, dc_fin = I.normal(5, 8, (T, Bn, H), 1.0, f32).to(DEV), I.normal(5, 9, (Bn, H), 1.0, f32).to(DEV)
    dx, dw_ih, dw_hh = torch.empty(T, Bn, In, dtype=bf, device=DEV), torch.empty(In, 4 * H, dtype=bf, device=DEV), torch.empty(H, 4 * H, dtype=bf, device=DEV)
    db, dh0, dc0 = torch.empty(4 * H, device=DEV), torch.empty(Bn, H, device=DEV), torch.empty(Bn, H, device=DEV)
    ws = ws_of(B.relay_workspace_bytes_lstm(t["x"], t["w_ih"], t["w_hh"]), B.relay_workspace_bytes_lstm_grad(t["x"], t["w_ih"], t["w_hh"]))

    def fn():
        B.relay_lstm_cell_seq(t["x"], t["w_ih"], t["w_hh"], t["b"], t["h0"], t["c0"], h_all, c, ws)
        B.relay_lstm_cell_seq_grad(t["x"], t["w_ih"], t["w_hh"], t["b"], t["h0"], t["c0"], h_all, dh_all, dc_fin,
                                   dx, dw_ih, dw_hh, db, dh0, dc0, ws)
    capture_and_compare(fn, [h_all, c, dx, dw_ih, dw_hh, db, dh0, dc0])


def test_loss_update_and_pooling_groups():
    t = dev(I.loss_batch(256, 512))
    loss, dscores = torch.empty(256, device=DEV), torch.empty_like(t["scores"])
    ps, gs = I.param_set([(64, 96), (33,)], torch.bfloat16, torch.bfloat16)
    ps0 = [p.to(DEV) for p in ps]
    params, grads = [p.clone() for p in ps0], [g.to(DEV) for g in gs]
    x = I.pool_input(2, 8, 12, 16).to(DEV)
    y, idx = torch.empty(2, 8, 6, 8, dtype=torch.bfloat16, device=DEV), torch.empty(2, 8, 6, 8, dtype=torch.int32, device=DEV)
    dy, dxp = I.normal(8, 1, (2, 8, 6, 8), 1.0, torch.bfloat16).to(DEV), torch.empty_like(x)

    def fn():
        for p, p0 in zip(params, ps0):               # the update mutates its parameters: start every run from the same ones
            p.copy_(p0)
        B.relay_softmax_xent_grad(t["scores"], t["targets"], t["dloss"], loss, dscores)
        B.relay_sgd_update(params, grads, 1e-2)
        B.relay_max_pool2d(x, 2, 2, 2, 2, y, idx)
        B.relay_max_pool2d_grad(idx, dy, 2, 2, 2, 2, dxp)
    capture_and_compare(fn, [loss, dscores, y, idx, dxp] + params)
