"""GPU parity: gradient program of the LSTM sequence against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_1810_00952_b200 import binding as B
from relay_workloads import inputs as I

from parity import Guarded, assert_bf16, to_np, workspace

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
F32, BF16 = torch.float32, torch.bfloat16


def forward(d):
    T, Bn, _ = d["x"].shape
    H = d["w_hh"].shape[0]
    h_all, c = torch.empty(T, Bn, H, device=DEV), torch.empty(Bn, H, device=DEV)
    ws = workspace(B.relay_workspace_bytes_lstm(d["x"], d["w_ih"], d["w_hh"]), DEV)
    B.relay_lstm_cell_seq(d["x"], d["w_ih"], d["w_hh"], d["b"], d["h0"], d["c0"], h_all, c, ws)
    return h_all, c


def backward(d, h_all, dh_all, dc_fin, want=("dx", "db", "dh0", "dc0")):
    T, Bn, In = d["x"].shape
    H = d["w_hh"].shape[0]
    out = dict(dx=Guarded((T, Bn, In), BF16, DEV) if "dx" in want else None, dw_ih=Guarded((In, 4 * H), BF16, DEV),
               dw_hh=Guarded((H, 4 * H), BF16, DEV), db=Guarded((4 * H,), F32, DEV) if "db" in want else None,
               dh0=Guarded((Bn, H), F32, DEV) if "dh0" in want else None, dc0=Guarded((Bn, H), F32, DEV) if "dc0" in want else None)
    ws = workspace(B.relay_workspace_bytes_lstm_grad(d["x"], d["w_ih"], d["w_hh"]), DEV)
    g = lambda k: out[k].t if out[k] is not None else None
    B.relay_lstm_cell_seq_grad(d["x"], d["w_ih"], d["w_hh"], d["b"], d["h0"], d["c0"], h_all, dh_all, dc_fin, g("dx"), g("dw_ih"),
                               g("dw_hh"), g("db"), g("dh0"), g("dc0"), ws)
    torch.cuda.synchronize()
    B.relay_poll_status()
    return {k: (v.check() if v is not None else None) for k, v in out.items()}


def case(T, Bn, In, H, salt, h0_random=True):
    t = I.cfg5_lstm(T, Bn, In, H, salt=salt)
    if h0_random:
        t["h0"] = I.uniform(5, 6, (Bn, H), -0.5, 0.5, F32, salt)
        t["c0"] = I.uniform(5, 7, (Bn, H), -0.5, 0.5, F32, salt)
    dh_all = I.normal(5, 8, (T, Bn, H), 1.0, F32, salt)
    dc_fin = I.normal(5, 9, (Bn, H), 1.0, F32, salt)
    return t, dh_all, dc_fin


def oracle_grads(t, dh_all, dc_fin):
    names = ("x", "w_ih", "w_hh", "b", "h0", "c0")
    out = oracle.lstm_cell_seq_grad(*(I.as_f64(t[k]) for k in names), I.as_f64(dh_all), None if dc_fin is None else I.as_f64(dc_fin))
    return dict(zip(("dx", "dw_ih", "dw_hh", "db", "dh0", "dc0"), out))


def compare(got, want, keys=("dx", "dw_ih", "dw_hh", "db", "dh0", "dc0")):
    for k in keys:
        if got[k] is not None:
            assert_bf16(got[k], want[k], stored_bf16=k in ("dx", "dw_ih", "dw_hh"), what=k)


# cluster kernel (H a multiple of 64, B <= 128), per-step kernels otherwise.  The cluster kernel's variants: one, two or four
# MMA issuers (H / 64 odd, even, a multiple of four); a stage in one copy (rows of a group a multiple of 8) or tile by tile;
# 16 to 64 accumulator columns (rows of a group rounded up to 16), one or two (row, unit) pairs per thread; a last group
# with fewer rows than the others
@pytest.mark.parametrize("T,Bn,In,H", [(1, 8, 64, 64), (3, 8, 64, 64), (5, 40, 96, 128), (4, 16, 32, 20), (6, 3, 24, 72), (3, 16, 64, 1024),
                                       (2, 130, 64, 64), (2, 96, 64, 1024), (3, 20, 32, 128), (3, 24, 64, 192), (2, 100, 64, 1024),
                                       (2, 128, 32, 1024), (3, 44, 64, 256), (4, 20, 64, 512)])
def test_gradient_program(T, Bn, In, H):
    t, dh_all, dc_fin = case(T, Bn, In, H, salt=T * 100 + H)
    d = {k: v.to(DEV) for k, v in t.items()}
    h_all, _ = forward(d)
    got = backward(d, h_all, dh_all.to(DEV), dc_fin.to(DEV))
    compare(got, oracle_grads(t, dh_all, dc_fin))


def test_optional_inputs_and_outputs():
    t, dh_all, _ = case(3, 8, 64, 64, salt=9)
    d = {k: v.to(DEV) for k, v in t.items()}
    h_all, _ = forward(d)
    got = backward(d, h_all, dh_all.to(DEV), None, want=())
    assert got["dx"] is None and got["db"] is None and got["dh0"] is None and got["dc0"] is None
    want = oracle_grads(t, dh_all, None)
    compare(got, want, keys=("dw_ih", "dw_hh"))
    full = backward(d, h_all, dh_all.to(DEV), None)
    compare(full, want)
    assert torch.equal(full["dw_ih"], got["dw_ih"]) and torch.equal(full["dw_hh"], got["dw_hh"])    # deterministic


def test_empty_sequence_and_rejections():
    t, dh_all, dc_fin = case(2, 8, 64, 64, salt=3)
    d = {k: v.to(DEV) for k, v in t.items()}
    h_all, _ = forward(d)
    d0 = dict(d, x=torch.empty(0, 8, 64, dtype=BF16, device=DEV))
    got = backward(d0, torch.empty(0, 8, 64, device=DEV), torch.empty(0, 8, 64, device=DEV), dc_fin.to(DEV))
    assert not got["dw_ih"].any() and not got["dw_hh"].any() and not got["db"].any() and not got["dh0"].any()
    assert torch.equal(got["dc0"].cpu(), dc_fin)
    ws = workspace(B.relay_workspace_bytes_lstm_grad(d["x"], d["w_ih"], d["w_hh"]), DEV)
    dwi, dwh = torch.full((64, 256), 5.0, dtype=BF16, device=DEV), torch.full((64, 256), 5.0, dtype=BF16, device=DEV)
    args = lambda **kw: [kw.get(k, v) for k, v in dict(x=d["x"], w_ih=d["w_ih"], w_hh=d["w_hh"], b=d["b"], h0=d["h0"], c0=d["c0"], h_all=h_all,
                                                      dh_all=dh_all.to(DEV), dc_final=None, dx=None, dw_ih=dwi, dw_hh=dwh, db=None, dh0=None,
                                                      dc0=None).items()]
    n0 = B.relay_launch_count()
    for kw, status in [(dict(dh_all=dh_all[:1].to(DEV)), "ERR_SHAPE"), (dict(dw_ih=dwi.float()), "ERR_DTYPE"),
                       (dict(h_all=h_all.bfloat16()), "ERR_DTYPE"), (dict(db=torch.zeros(255, device=DEV)), "ERR_SHAPE"),
                       (dict(dw_hh=d["w_hh"]), "ERR_ATTR"), (dict(dc_final=torch.zeros(8, device=DEV)), "ERR_RANK")]:
        with pytest.raises(B.RelayError) as e:
            B.relay_lstm_cell_seq_grad(*args(**kw), ws)
        assert e.value.status_name == status, str(e.value)
    with pytest.raises(B.RelayError) as e:
        B.relay_lstm_cell_seq_grad(*args(), None)
    assert e.value.status_name == "ERR_WORKSPACE"
    torch.cuda.synchronize()
    assert B.relay_launch_count() == n0 and bool((dwi == 5.0).all())


def test_full_size_sampled_batch_rows():
    """Configuration 5 at full size (T=128, B=64, I=H=1024).  Batch rows are independent in dx, dh0 and dc0, so the
    oracle runs the whole program on 2 of the 64 rows; the weight partials (sums over all rows and steps) are compared
    at T = 128 with a batch the oracle can run whole in the next test."""
    t, dh_all, dc_fin = case(128, 64, 1024, 1024, salt=0, h0_random=False)
    d = {k: v.to(DEV) for k, v in t.items()}
    h_all, _ = forward(d)
    got = backward(d, h_all, dh_all.to(DEV), dc_fin.to(DEV))
    rows = [5, 63]
    sub = {k: (v[:, rows] if k == "x" else v[rows] if k in ("h0", "c0") else v) for k, v in t.items()}
    want = oracle_grads(sub, dh_all[:, rows], dc_fin[rows])
    assert_bf16(got["dx"][:, rows], want["dx"], what="dx")
    assert_bf16(got["dh0"][rows], want["dh0"], stored_bf16=False, what="dh0")
    assert_bf16(got["dc0"][rows], want["dc0"], stored_bf16=False, what="dc0")
    for k in ("dw_ih", "dw_hh", "db"):
        assert bool(torch.isfinite(got[k].float()).all())


def test_full_length_sequence_all_six_partials():
    """T = 128, I = H = 1024 as in configuration 5, with a batch of 8 rows so that the oracle can run the whole
    program: the weight and bias partials are sums over all 128 steps (and rows), which no shorter case reaches.
    (The two sides round dz to bf16 from an fp32 and an fp64 value; a differing last bit changes every later dz a
    little, so after a few steps their roundings are independent and each of the T*B terms of a weight partial differs
    by a fraction of a bf16 step of that term.  The error is 1.8e-3 of the RMS whatever T and B are, but its largest
    element over the 4.2 M of a weight partial depends on how heavy-tailed the sums are: with 4 rows one element
    reaches 1.05e-2 of the RMS beyond its storage rounding, with 8 rows 0.8e-2, inside the 1e-2 bound.)"""
    t, dh_all, dc_fin = case(128, 8, 1024, 1024, salt=41)
    d = {k: v.to(DEV) for k, v in t.items()}
    h_all, _ = forward(d)
    got = backward(d, h_all, dh_all.to(DEV), dc_fin.to(DEV))
    compare(got, oracle_grads(t, dh_all, dc_fin))


@pytest.mark.parametrize("T,Bn,In,H", [(128, 64, 1024, 1024), (32, 96, 128, 512)])
def test_reruns_are_bit_identical(T, Bn, In, H):
    """The persistent kernels exchange h / dz between blocks through L2 behind a grid barrier; a missed ordering there
    would show as run-to-run differences.  Forward and gradient program are rerun with other work in between."""
    t, dh_all, dc_fin = case(T, Bn, In, H, salt=7, h0_random=False)
    d = {k: v.to(DEV) for k, v in t.items()}
    dh_all, dc_fin = dh_all.to(DEV), dc_fin.to(DEV)
    ref = None
    for it in range(6):
        h_all, c = forward(d)
        got = backward(d, h_all, dh_all, dc_fin)
        cur = [h_all.cpu(), c.cpu()] + [got[k] for k in ("dx", "dw_ih", "dw_hh", "db", "dh0", "dc0")]
        if ref is None:
            ref = cur
        else:
            assert all(torch.equal(a.cpu(), b.cpu()) for a, b in zip(ref, cur)), it
        if it % 2 == 0:
            torch.zeros(1 << 24, device=DEV).sum().item()      # shifts the timing of the next launch
