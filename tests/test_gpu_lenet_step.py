"""GPU parity of one whole training step of the LeNet-shaped model of the paper's listing (Fig. 3):
conv 5x5 + tanh, max_pool 2x2, conv 5x5 + tanh, max_pool 2x2, flatten, linear + tanh, linear,
softmax_cross_entropy; the gradient program back to every parameter; update_model_params (SGD).
Every group is checked against the oracle fed with the GPU's stored inputs of that group."""
import numpy as np
import pytest
import torch

import oracle
from paper_1810_00952_b200 import binding as B
from relay_workloads import inputs as I

from parity import assert_f32, to_np

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
F64 = oracle.F64
TANH, NONE = B.ACT_TANH, B.ACT_NONE
K = (2, 2, 2, 2)


def ws_for(nbytes):
    return torch.empty(max(int(nbytes), 16), dtype=torch.uint8, device=DEV)


def E(*shape, dtype=torch.float32):
    return torch.empty(*shape, dtype=dtype, device=DEV)


def test_one_training_step_group_by_group():
    N, lr = 16, float(np.float32(0.002))
    t = {k: v.to(DEV) for k, v in I.lenet_batch(N).items()}
    x = t["x"]

    # ---- forward -------------------------------------------------------------------------------------
    c1 = E(N, 20, 24, 24); B.relay_fused_conv2d_act(x, t["w1"], t["b1"], 1, 0, TANH, c1, ws_for(B.relay_workspace_bytes_conv2d_act(x, t["w1"], 1, 0)))
    p1, i1 = E(N, 20, 12, 12), E(N, 20, 12, 12, dtype=torch.int32); B.relay_max_pool2d(c1, *K, p1, i1)
    c2 = E(N, 50, 8, 8); B.relay_fused_conv2d_act(p1, t["w2"], t["b2"], 1, 0, TANH, c2, ws_for(B.relay_workspace_bytes_conv2d_act(p1, t["w2"], 1, 0)))
    p2, i2 = E(N, 50, 4, 4), E(N, 50, 4, 4, dtype=torch.int32); B.relay_max_pool2d(c2, *K, p2, i2)
    flat = p2.view(N, 800)                                         # flatten_layer: the same bytes, another shape
    f1 = E(N, 500); B.relay_fused_dense_act(flat, t["w3"], t["b3"], TANH, f1)
    f2 = E(N, 10); B.relay_fused_dense_act(f1, t["w4"], t["b4"], NONE, f2)
    loss, dscores = E(N), E(N, 10)
    dloss = torch.full((N,), 1.0 / N, device=DEV)                  # the scalar being differentiated is the batch mean
    B.relay_softmax_xent_grad(f2, t["labels"], dloss, loss, dscores)
    torch.cuda.synchronize()

    n = to_np
    assert_f32(c1, oracle.conv2d_act(n(x), n(t["w1"]), n(t["b1"]), 1, 0, TANH, F64), "conv1")
    oy, oi = oracle.max_pool2d(n(c1), *K); assert np.array_equal(n(p1), oy) and np.array_equal(i1.cpu().numpy(), oi)
    assert_f32(c2, oracle.conv2d_act(n(p1), n(t["w2"]), n(t["b2"]), 1, 0, TANH, F64), "conv2")
    oy, oi = oracle.max_pool2d(n(c2), *K); assert np.array_equal(n(p2), oy) and np.array_equal(i2.cpu().numpy(), oi)
    assert_f32(f1, oracle.dense_act(n(flat), n(t["w3"]), n(t["b3"]), TANH, F64), "fc1")
    assert_f32(f2, oracle.dense_act(n(f1), n(t["w4"]), n(t["b4"]), NONE, F64), "fc2")
    ol, odz = oracle.softmax_xent_grad(n(f2), n(t["labels"]), n(dloss))
    assert_f32(loss, ol, "loss"); assert_f32(dscores, odz, "dscores")

    # ---- gradient program -------------------------------------------------------------------------------
    g = {k: torch.empty_like(t[k]) for k in ("w1", "b1", "w2", "b2", "w3", "b3", "w4", "b4")}
    d_f1 = E(N, 500)
    B.relay_fused_dense_act_grad(f1, t["w4"], f2, dscores, NONE, d_f1, g["w4"], g["b4"], ws_for(B.relay_workspace_bytes_dense_act_grad(f1, t["w4"])))
    d_flat = E(N, 800)
    B.relay_fused_dense_act_grad(flat, t["w3"], f1, d_f1, TANH, d_flat, g["w3"], g["b3"], ws_for(B.relay_workspace_bytes_dense_act_grad(flat, t["w3"])))
    d_c2 = E(N, 50, 8, 8); B.relay_max_pool2d_grad(i2, d_flat.view(N, 50, 4, 4), *K, d_c2)
    d_p1 = E(N, 20, 12, 12)
    B.relay_fused_conv2d_act_grad(p1, t["w2"], c2, d_c2, 1, 0, TANH, d_p1, g["w2"], g["b2"], ws_for(B.relay_workspace_bytes_conv2d_act_grad(p1, t["w2"], 1, 0)))
    d_c1 = E(N, 20, 24, 24); B.relay_max_pool2d_grad(i1, d_p1, *K, d_c1)
    B.relay_fused_conv2d_act_grad(x, t["w1"], c1, d_c1, 1, 0, TANH, None, g["w1"], g["b1"], ws_for(B.relay_workspace_bytes_conv2d_act_grad(x, t["w1"], 1, 0)))
    torch.cuda.synchronize()

    F32c = oracle.F32
    odx, odw, odb = oracle.dense_act_grad(n(f1), n(t["w4"]), n(f2), n(dscores), NONE, F64, F64, F64, dz_dtype=F32c)
    assert_f32(d_f1, odx, "d_fc1"); assert_f32(g["w4"], odw, "dw4"); assert_f32(g["b4"], odb, "db4")
    odx, odw, odb = oracle.dense_act_grad(n(flat), n(t["w3"]), n(f1), n(d_f1), TANH, F64, F64, F64, dz_dtype=F32c)
    assert_f32(d_flat, odx, "d_flat"); assert_f32(g["w3"], odw, "dw3"); assert_f32(g["b3"], odb, "db3")
    assert np.array_equal(n(d_c2), oracle.max_pool2d_grad(i2.cpu().numpy(), n(d_flat).reshape(N, 50, 4, 4), 8, 8))
    odx, odw, odb = oracle.conv2d_act_grad(n(p1), n(t["w2"]), n(c2), n(d_c2), 1, 0, TANH, F64, F64, F64, dz_dtype=F32c)
    assert_f32(d_p1, odx, "d_pool1"); assert_f32(g["w2"], odw, "dw2"); assert_f32(g["b2"], odb, "db2")
    assert np.array_equal(n(d_c1), oracle.max_pool2d_grad(i1.cpu().numpy(), n(d_p1), 24, 24))
    _, odw, odb = oracle.conv2d_act_grad(n(x), n(t["w1"]), n(c1), n(d_c1), 1, 0, TANH, F64, F64, F64, want_dx=False, dz_dtype=F32c)
    assert_f32(g["w1"], odw, "dw1"); assert_f32(g["b1"], odb, "db1")

    # ---- update_model_params: one launch for the eight parameters ------------------------------------------
    names = list(g)
    before = {k: n(t[k]) for k in names}
    n0 = B.relay_launch_count()
    B.relay_sgd_update([t[k] for k in names], [g[k] for k in names], lr)
    torch.cuda.synchronize()
    assert B.relay_launch_count() - n0 == 1
    for k in names:
        assert_f32(t[k], oracle.sgd_update(before[k], n(g[k]), lr, F64), k)

    # the step lowers the loss of this batch (oracle forward with the updated parameters, end to end)
    def oracle_loss(pr):
        a = oracle.conv2d_act(n(x), pr["w1"], pr["b1"], 1, 0, TANH, F64)
        a, _ = oracle.max_pool2d(a, *K)
        a = oracle.conv2d_act(a, pr["w2"], pr["b2"], 1, 0, TANH, F64)
        a, _ = oracle.max_pool2d(a, *K)
        a = oracle.dense_act(a.reshape(N, 800), pr["w3"], pr["b3"], TANH, F64)
        a = oracle.dense_act(a, pr["w4"], pr["b4"], NONE, F64)
        return oracle.softmax_xent(a, n(t["labels"])).mean()
    l0, l1 = oracle_loss(before), oracle_loss({k: n(t[k]) for k in names})
    assert abs(l0 - float(loss.mean())) < 1e-4 * max(l0, 1.0)
    assert l1 < l0
