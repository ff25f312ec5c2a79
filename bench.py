#!/usr/bin/env python
"""Benchmark of the fused operator groups on B200.

One "step" is one pass of the whole hot path over synthetic inputs shaped like the five
configurations: tiny fp32 MLP layer (forward + gradient), the bf16 broadcast-elementwise group
(forward + gradient group), the 3-layer bf16 MLP (forward + full backward), the 3x3 conv2d
(forward + dX + dW + db) and the LSTM sequence.  Every group is timed with CUDA events on the
launching stream; the line printed at the end carries the tensor-bound aggregate as `value`
(TFLOP/s over the dense + conv2d groups), the memory-bound aggregate (GB/s over the elementwise
groups), a per-group table, the roofline of the dominant kernel, the end-to-end figure with
host buffers, and the CPU oracle timed on a bounded sample.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--groups a,b,..]

With N > 1 (under torchrun) every rank runs an independent replica on its own GPU: the path
has no exchange step, so there is no collective on the data path.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

METRIC = "fused-group TFLOP/s (dense/conv) and HBM GB/s (ewise/reduce) on 1 B200 vs roofline"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL_PEAKS = {"hbm_gbs": 7700.0, "bf16_tflops": 2250.0}      # data-sheet figures (HGX B200, dense bf16), for context
ALL_GROUPS = ["cfg1", "cfg2", "cfg3", "cfg4", "cfg5", "next"]


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        d["source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["source"] = "fallback"
    return d


# ---------------------------------------------------------------------------------------------------
# clocks sampling (nvidia-smi in the background during the timed region)
# ---------------------------------------------------------------------------------------------------
class ClockSampler:
    Q = "clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown," \
        "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap"

    def __init__(self, index: int):
        self.index, self.rows, self.proc, self.t0 = index, [], None, None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "20"], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.monotonic(), [c.strip() for c in line.split(",")]))

    def begin(self):
        """Marks the start of the timed region: only samples that arrive from here on are reported (the tool is
        started earlier, during the warm-up, because it needs a few hundred milliseconds to deliver its first row)."""
        self.t0 = time.monotonic()

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        rows = [r for t, r in self.rows if self.t0 is None or t >= self.t0]
        for r in rows:
            try:
                sm.append(float(r[0])); mx = float(r[1])
            except Exception:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons), "samples": len(sm)}


# ---------------------------------------------------------------------------------------------------
# the groups
# ---------------------------------------------------------------------------------------------------
class Timer:
    """CUDA-event timing of labelled regions on the current stream."""

    def __init__(self):
        self.pending, self.ms, self.div = [], {}, {}

    def region(self, label, launches=1):
        """`launches` > 1: the region holds that many back-to-back launches of one kernel on DIFFERENT tensors (nothing a launch
        reads was touched by the launches before it); the recorded time is the region's divided by `launches`, i.e. the
        kernel's average duration without the few microseconds of event and launch latency that a lone short kernel carries."""
        t = self
        t.div[label] = launches

        class R:
            def __enter__(self_inner):
                self_inner.a = torch.cuda.Event(enable_timing=True); self_inner.b = torch.cuda.Event(enable_timing=True)
                self_inner.a.record()

            def __exit__(self_inner, *exc):
                self_inner.b.record()
                t.pending.append((label, self_inner.a, self_inner.b))
        return R()

    def collect(self):
        torch.cuda.synchronize()
        for label, a, b in self.pending:
            self.ms.setdefault(label, []).append(a.elapsed_time(b) / self.div.get(label, 1))
        self.pending = []


class LeNetStep:
    """One training step of the LeNet-shaped model of the paper's listing (Fig. 3), fp32: conv 5x5 + tanh, max_pool 2x2,
    conv 5x5 + tanh, max_pool 2x2, flatten, linear + tanh, linear, softmax_cross_entropy; the gradient program back to
    every parameter; one SGD update of the eight parameters.  All buffers are allocated once; `run` only enqueues."""

    def __init__(self, B, I, dev, N):
        self.B, self.N = B, N
        self.t = t = {k: v.to(dev) for k, v in I.lenet_batch(N).items()}
        self.p0 = {k: t[k].clone() for k in ("w1", "b1", "w2", "b2", "w3", "b3", "w4", "b4")}
        E = lambda *s, dt=torch.float32: torch.empty(*s, dtype=dt, device=dev)
        i32 = torch.int32
        self.c1, self.p1, self.i1 = E(N, 20, 24, 24), E(N, 20, 12, 12), E(N, 20, 12, 12, dt=i32)
        self.c2, self.p2, self.i2 = E(N, 50, 8, 8), E(N, 50, 4, 4), E(N, 50, 4, 4, dt=i32)
        self.f1, self.f2, self.loss, self.dscores = E(N, 500), E(N, 10), E(N), E(N, 10)
        self.dloss = torch.full((N,), 1.0 / N, device=dev)
        self.g = {k: torch.empty_like(v) for k, v in self.p0.items()}
        self.d_f1, self.d_flat, self.d_c2, self.d_p1, self.d_c1 = E(N, 500), E(N, 800), E(N, 50, 8, 8), E(N, 20, 12, 12), E(N, 20, 24, 24)
        flat = self.p2.view(N, 800)
        self.ws = torch.empty(max(16, B.relay_workspace_bytes_conv2d_act(t["x"], t["w1"], 1, 0), B.relay_workspace_bytes_conv2d_act(self.p1, t["w2"], 1, 0),
                                  B.relay_workspace_bytes_dense_act_grad(self.f1, t["w4"]), B.relay_workspace_bytes_dense_act_grad(flat, t["w3"]),
                                  B.relay_workspace_bytes_conv2d_act_grad(self.p1, t["w2"], 1, 0),
                                  B.relay_workspace_bytes_conv2d_act_grad(t["x"], t["w1"], 1, 0)), dtype=torch.uint8, device=dev)
        self.graph = None

    def flop(self):
        N = self.N
        conv1, conv2, fc1, fc2 = 2 * N * 20 * 24 * 24 * 25, 2 * N * 50 * 8 * 8 * 20 * 25, 2 * N * 800 * 500, 2 * N * 500 * 10
        return 3 * (conv2 + fc1 + fc2) + 2 * conv1        # forward + (dx, dW) of every layer; the first layer has no dx

    def run(self):
        B, t, g, ws, N = self.B, self.t, self.g, self.ws, self.N
        TANH, NONE, K = B.ACT_TANH, B.ACT_NONE, (2, 2, 2, 2)
        for k, v in self.p0.items():                       # every run starts from the same parameters
            t[k].copy_(v)
        B.relay_fused_conv2d_act(t["x"], t["w1"], t["b1"], 1, 0, TANH, self.c1, ws)
        B.relay_max_pool2d(self.c1, *K, self.p1, self.i1)
        B.relay_fused_conv2d_act(self.p1, t["w2"], t["b2"], 1, 0, TANH, self.c2, ws)
        B.relay_max_pool2d(self.c2, *K, self.p2, self.i2)
        flat = self.p2.view(N, 800)
        B.relay_fused_dense_act(flat, t["w3"], t["b3"], TANH, self.f1, ws)
        B.relay_fused_dense_act(self.f1, t["w4"], t["b4"], NONE, self.f2, ws)
        B.relay_softmax_xent_grad(self.f2, t["labels"], self.dloss, self.loss, self.dscores)
        B.relay_fused_dense_act_grad(self.f1, t["w4"], self.f2, self.dscores, NONE, self.d_f1, g["w4"], g["b4"], ws)
        B.relay_fused_dense_act_grad(flat, t["w3"], self.f1, self.d_f1, TANH, self.d_flat, g["w3"], g["b3"], ws)
        B.relay_max_pool2d_grad(self.i2, self.d_flat.view(N, 50, 4, 4), *K, self.d_c2)
        B.relay_fused_conv2d_act_grad(self.p1, t["w2"], self.c2, self.d_c2, 1, 0, TANH, self.d_p1, g["w2"], g["b2"], ws)
        B.relay_max_pool2d_grad(self.i1, self.d_p1, *K, self.d_c1)
        B.relay_fused_conv2d_act_grad(t["x"], t["w1"], self.c1, self.d_c1, 1, 0, TANH, None, g["w1"], g["b1"], ws)
        names = list(g)
        B.relay_sgd_update([t[k] for k in names], [g[k] for k in names], 0.002)

    def capture(self):
        self.graph, s = torch.cuda.CUDAGraph(), torch.cuda.Stream()
        s.wait_stream(torch.cuda.current_stream())
        with torch.cuda.graph(self.graph, stream=s):
            self.run()
        torch.cuda.current_stream().wait_stream(s)


class Workload:
    def __init__(self, dev, groups, small=False):
        from paper_1810_00952_b200 import binding as B
        from relay_workloads import inputs as I
        from relay_workloads import program as P
        self.B, self.I, self.P, self.dev, self.groups = B, I, P, dev, groups
        self.host, self.devt, self.out = {}, {}, {}
        ws_bytes = 16
        if "cfg1" in groups:
            self.host["cfg1"] = I.cfg1_tiny_mlp()
        if "cfg2" in groups:
            self.host["cfg2"] = I.cfg2_ewise(*((512, 1024) if small else (8192, 8192)))
        if "cfg3" in groups:
            self.host["cfg3"] = I.cfg3_mlp(*((256, 256) if small else (4096, 4096)))
        if "cfg4" in groups:
            self.host["cfg4"] = I.cfg4_conv(*((2, 32, 14, 14, 32) if small else (32, 256, 56, 56, 256)))
        if "cfg5" in groups:
            self.host["cfg5"] = I.cfg5_lstm(*((8, 8, 64, 64) if small else (128, 64, 1024, 1024)))
        if "next" in groups:       # loss group and parameter update (the rows that close a training step)
            self.host["next"] = I.loss_batch(*((256, 512) if small else (8192, 8192)))
        for g, d in self.host.items():
            self.host[g] = {k: v.pin_memory() for k, v in d.items()}
            self.devt[g] = {k: torch.empty_like(v, device=dev) for k, v in d.items()}
        E = lambda *s, dt=torch.bfloat16: torch.empty(*s, dtype=dt, device=dev)
        f32 = torch.float32
        if "cfg1" in groups:
            # a mid-size layer of the same fp32 tier (true fp32 FMA, no tensor cores), device-resident: its ALU roofline
            n32 = 128 if small else 1024
            t32 = I.cfg1_tiny_mlp(n32, n32, n32, salt=5)
            self.f32_mid = dict(x=t32["x"].to(dev), w=(t32["w"] / n32 ** 0.5).to(dev), b=t32["b"].to(dev), y=E(n32, n32, dt=f32))
            self.out["cfg1"] = dict(y=E(8, 32, dt=f32), dx=E(8, 64, dt=f32), dw=E(64, 32, dt=f32), db=E(32, dt=f32))
            ws_bytes = max(ws_bytes, B.relay_workspace_bytes_dense_act_grad(self.devt["cfg1"]["x"], self.devt["cfg1"]["w"]))
        if "cfg2" in groups:
            r, c = self.host["cfg2"]["x"].shape
            self.out["cfg2"] = dict(out=E(r, c), dx=E(r, c), da=E(c, dt=f32), db=E(1, c, dt=f32))
            self.fwd_prog, self.fwd_outs = P.tanh_affine_residual_fwd(P.BF16)
            self.grad_prog, ids = P.tanh_affine_residual_grad(P.BF16)
            self.grad_specs = [(ids[0], B.RED_NONE, 0, 0), (ids[1], B.RED_SUM, 1, 0), (ids[2], B.RED_SUM, 1, 1)]
            d = self.devt["cfg2"]
            ws_bytes = max(ws_bytes, B.relay_workspace_bytes_reduce([d["dout"], d["x"], d["a"], d["b"]], self.grad_specs))
        if "cfg2" in groups:
            # standalone reductions of the same [rows, cols] bf16 tensor: over the last axis (sum, max, argmax) and over axis 0
            r, c = self.host["cfg2"]["x"].shape
            self.red_prog = P.Program([P.BF16])
            self.red_out = dict(sum1=E(r, dt=f32), max1=E(r, dt=f32), arg1=E(r, dt=torch.int64), sum0=E(c, dt=f32))
            self.red_specs = dict(sum1=[(0, B.RED_SUM, 2, 0)], max1=[(0, B.RED_MAX, 2, 0)], arg1=[(0, B.RED_ARGMAX, 2, 0)],
                                  sum0=[(0, B.RED_SUM, 1, 0)])
            ws_bytes = max(ws_bytes, B.relay_workspace_bytes_reduce([self.devt["cfg2"]["x"]], self.red_specs["sum0"]))
            # two programs that have no pre-compiled body (they run on the vectorised evaluator): out = sigmoid(x*y) + relu(z)
            # with z constant down the rows, and its gradient group (dx, dy unreduced, dz summed over the rows)
            self.vm_fwd, self.vm_fwd_outs = P.sigmoid_product_relu_fwd(P.BF16)
            self.vm_grad, ids = P.sigmoid_product_relu_grad(P.BF16)
            self.vm_grad_specs = [(ids[0], B.RED_NONE, 0, 0), (ids[1], B.RED_NONE, 0, 0), (ids[2], B.RED_SUM, 1, 0)]
            self.vm_out = dict(out=E(r, c), dx=E(r, c), dy=E(r, c), dz=E(c, dt=f32))
            d = self.devt["cfg2"]
            ws_bytes = max(ws_bytes, B.relay_workspace_bytes_reduce([d["dout"], d["x"], d["dout"], d["a"]], self.vm_grad_specs))
        if "cfg3" in groups:
            m, k = self.host["cfg3"]["x"].shape
            o = dict()
            for l in range(3):
                o[f"y{l}"] = E(m, k); o[f"dx{l}"] = E(m, k); o[f"dw{l}"] = E(k, k); o[f"db{l}"] = E(k, dt=f32)
            self.out["cfg3"] = o
            ws_bytes = max(ws_bytes, B.relay_workspace_bytes_dense_act_grad(self.devt["cfg3"]["x"], self.devt["cfg3"]["w0"]))
        if "cfg4" in groups:
            d = self.devt["cfg4"]
            self.out["cfg4"] = dict(y=torch.empty_like(d["dy"]), dx=torch.empty_like(d["x"]), dw=torch.empty_like(d["w"]),
                                    db=E(d["w"].shape[0], dt=f32))
            ws_bytes = max(ws_bytes, B.relay_workspace_bytes_conv2d_act(d["x"], d["w"], 1, 1),
                           B.relay_workspace_bytes_conv2d_act_grad(d["x"], d["w"], 1, 1))
        if "cfg5" in groups:
            d = self.devt["cfg5"]
            T, Bn, _ = d["x"].shape
            H = d["w_hh"].shape[0]
            In = d["x"].shape[2]
            self.out["cfg5"] = dict(h_all=E(T, Bn, H, dt=f32), c=E(Bn, H, dt=f32), dx=E(T, Bn, In), dw_ih=E(In, 4 * H),
                                    dw_hh=E(H, 4 * H), db=E(4 * H, dt=f32), dh0=E(Bn, H, dt=f32), dc0=E(Bn, H, dt=f32))
            # upstream partials of the gradient program (device-resident, generated once)
            self.lstm_dh_all = I.normal(5, 8, (T, Bn, H), 1.0, f32).to(dev)
            self.lstm_dc_fin = I.normal(5, 9, (Bn, H), 1.0, f32).to(dev)
            self.lstm_zx = E(T * Bn, 4 * H, dt=f32)       # the batched input contraction alone (not a result of the step)
            ws_bytes = max(ws_bytes, B.relay_workspace_bytes_lstm(d["x"], d["w_ih"], d["w_hh"]),
                           B.relay_workspace_bytes_lstm_grad(d["x"], d["w_ih"], d["w_hh"]))
        if "next" in groups:
            d = self.devt["next"]
            self.out["next"] = dict(loss=E(d["scores"].shape[0], dt=f32), loss2=E(d["scores"].shape[0], dt=f32), dscores=torch.empty_like(d["scores"]))
            # parameters the update mutates: device-resident state of its own (three weight matrices), so the
            # other groups' inputs stay as generated; their gradients are generated once as well
            n = 256 if small else 4096
            ps, gs = I.param_set([(n, n)] * 3, torch.bfloat16, torch.bfloat16)
            self.sgd_params, self.sgd_grads = [p.to(dev) for p in ps], [g.to(dev) for g in gs]
            # max pooling 2x2 stride 2 of an activation of the conv configuration's shape (device-resident)
            shp = (2, 32, 14, 16) if small else (32, 256, 56, 56)
            self.pool_x = I.pool_input(*shp).to(dev)
            ps_ = (shp[0], shp[1], shp[2] // 2, shp[3] // 2)
            self.pool_y, self.pool_idx = E(*ps_), E(*ps_, dt=torch.int32)
            self.pool_dy, self.pool_dx = I.normal(8, 1, ps_, 1.0, torch.bfloat16).to(dev), torch.empty_like(self.pool_x)
            # four sets of tensors for four back-to-back launches (a launch's 90 MB are then not in L2 from the one before)
            self.pool_sets = [dict(x=self.pool_x, y=self.pool_y, idx=self.pool_idx, dy=self.pool_dy, dx=self.pool_dx)]
            for _ in range(0 if small else 3):
                self.pool_sets.append({k: v.clone() for k, v in self.pool_sets[0].items()})
            self.lenet = LeNetStep(B, I, dev, 4 if small else 64)
            # the conv configuration's tensors tagged NHWC (device-resident, permuted once): the layout-tagged calls
            c4 = self.devt["cfg4"] if "cfg4" in groups else {k: v.to(dev) for k, v in
                                                             I.cfg4_conv(*((2, 32, 14, 14, 32) if small else (32, 256, 56, 56, 256))).items()}
            nhwc = lambda a: a.permute(0, 2, 3, 1).contiguous()
            self.nhwc = dict(x=nhwc(c4["x"]), dy=nhwc(c4["dy"]), w=c4["w"], b=c4["b"])
            self.nhwc.update(y=torch.empty_like(self.nhwc["dy"]), dx=torch.empty_like(self.nhwc["x"]), dw=torch.empty_like(c4["w"]),
                             db=E(c4["w"].shape[0], dt=f32))
            ws_bytes = max(ws_bytes, B.relay_workspace_bytes_conv2d_act(self.nhwc["x"], c4["w"], 1, 1, layout=B.NHWC),
                           B.relay_workspace_bytes_conv2d_act_grad(self.nhwc["x"], c4["w"], 1, 1, layout=B.NHWC))
        self.ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
        self.flush_buf = torch.zeros(1024 * 1024 * 1024, dtype=torch.uint8, device=dev)
        self.pinned_out = {g: {k: torch.empty_like(v, device="cpu").pin_memory() for k, v in o.items()} for g, o in self.out.items()}
        self.upload()

    # -- data movement ---------------------------------------------------------------------------------
    def upload(self):
        n = 0
        for g, d in self.host.items():
            for k, v in d.items():
                self.devt[g][k].copy_(v, non_blocking=True)
                n += v.numel() * v.element_size()
        return n

    def download(self):
        n = 0
        for g, o in self.out.items():
            for k, v in o.items():
                self.pinned_out[g][k].copy_(v, non_blocking=True)
                n += v.numel() * v.element_size()
        return n

    def cfg1_sets(self, d, o):
        """Four sets of the tiny layer's tensors: the current ones and three copies (made once per buffer set)."""
        key = id(d)
        cache = self.__dict__.setdefault("_cfg1_sets", {})
        if key not in cache:
            cache[key] = [(d, o)] + [({k: v.clone() for k, v in d.items()}, {k: v.clone() for k, v in o.items()}) for _ in range(3)]
        return cache[key]

    def capture_cfg1(self):
        """Captures the tiny layer's forward + gradient group (five small launches, launch-bound when issued one by
        one) into a CUDA graph; `step` replays it as the group `cfg1.graph` while the captured buffers are current."""
        if "cfg1" not in self.groups:
            return
        B, d, o, ws = self.B, self.devt["cfg1"], self.out["cfg1"], self.ws
        g, s = torch.cuda.CUDAGraph(), torch.cuda.Stream()
        s.wait_stream(torch.cuda.current_stream())
        with torch.cuda.graph(g, stream=s):
            B.relay_fused_dense_act(d["x"], d["w"], d["b"], B.ACT_RELU, o["y"], ws)
            B.relay_fused_dense_act_grad(d["x"], d["w"], o["y"], d["dy"], B.ACT_RELU, o["dx"], o["dw"], o["db"], ws)
        torch.cuda.current_stream().wait_stream(s)
        self.cfg1_graph, self.cfg1_graph_bufs = g, d

    def capture_graphs(self):
        self.capture_cfg1()
        if "next" in self.groups:
            self.lenet.capture()

    def make_alternate(self):
        """Second set of device input and result buffers for the pipelined end-to-end loop."""
        self.alt = ({g: {k: torch.empty_like(v) for k, v in d.items()} for g, d in self.devt.items()},
                    {g: {k: torch.empty_like(v) for k, v in o.items()} for g, o in self.out.items()})

    def swap(self):
        (self.devt, self.out), self.alt = self.alt, (self.devt, self.out)

    def flush_l2(self):
        # 1 GiB read (a max-reduction): evicts the 126 MB L2 with CLEAN lines, so no write-back of the
        # flush itself overlaps the timed kernels, and keeps the GPU busy while the host queues the group
        self.flush_sink = self.flush_buf.view(torch.int32).max()

    # -- one pass of the hot path ------------------------------------------------------------------------
    def step(self, tm: Timer):
        B, ws = self.B, self.ws
        if "cfg1" in self.groups:
            d, o = self.devt["cfg1"], self.out["cfg1"]
            self.flush_l2()      # keeps the GPU busy while the host queues the calls: the events then time the device, not the host
            with tm.region("cfg1.fwd"):
                B.relay_fused_dense_act(d["x"], d["w"], d["b"], B.ACT_RELU, o["y"], ws)
            with tm.region("cfg1.grad"):
                B.relay_fused_dense_act_grad(d["x"], d["w"], o["y"], d["dy"], B.ACT_RELU, o["dx"], o["dw"], o["db"], ws)
            if getattr(self, "cfg1_graph", None) is not None and self.cfg1_graph_bufs is d:
                self.flush_l2()
                with tm.region("cfg1.graph"):
                    self.cfg1_graph.replay()
            # the same two calls as four back-to-back launches on four copies of the tensors (none in L2 after the flush): the
            # kernel's own duration, without the event and first-launch latency that a lone call of a few microseconds carries
            sets = self.cfg1_sets(d, o)
            self.flush_l2()
            with tm.region("cfg1.fwd.kernel", launches=len(sets)):
                for dd, oo in sets:
                    B.relay_fused_dense_act(dd["x"], dd["w"], dd["b"], B.ACT_RELU, oo["y"], ws)
            self.flush_l2()
            with tm.region("cfg1.grad.kernel", launches=len(sets)):
                for dd, oo in sets:
                    B.relay_fused_dense_act_grad(dd["x"], dd["w"], oo["y"], dd["dy"], B.ACT_RELU, oo["dx"], oo["dw"], oo["db"], ws)
            m = self.f32_mid
            with tm.region("cfg1.fp32_mid.fwd"):
                B.relay_fused_dense_act(m["x"], m["w"], m["b"], B.ACT_RELU, m["y"], ws)
        if "cfg2" in self.groups:
            d, o = self.devt["cfg2"], self.out["cfg2"]
            self.flush_l2()
            with tm.region("cfg2.fwd"):
                B.relay_fused_ewise(self.fwd_prog.arrays(), [d["x"], d["a"], d["b"]], self.fwd_outs, [o["out"]], ws)
            self.flush_l2()
            with tm.region("cfg2.grad"):
                B.relay_fused_reduce(self.grad_prog.arrays(), [d["dout"], d["x"], d["a"], d["b"]], self.grad_specs,
                                     [o["dx"], o["da"], o["db"]], ws)
            # a program without a pre-compiled body: as the library runs it (a body compiled at run time where the compiler
            # library is present), then on the in-kernel interpreter (the route without that library)
            for tag, compiled in (("jit", True), ("vm", False)):
                if compiled and B.relay_debug_jit_compiled() < 0:
                    continue
                before = B.relay_debug_set_jit(compiled)
                self.flush_l2()
                with tm.region(f"a6.{tag}_fwd"):
                    B.relay_fused_ewise(self.vm_fwd.arrays(), [d["x"], d["dout"], d["a"]], self.vm_fwd_outs, [self.vm_out["out"]], ws)
                self.flush_l2()
                with tm.region(f"a7.{tag}_grad"):
                    B.relay_fused_reduce(self.vm_grad.arrays(), [d["dout"], d["x"], o["out"], d["a"]], self.vm_grad_specs,
                                         [self.vm_out["dx"], self.vm_out["dy"], self.vm_out["dz"]], ws)
                B.relay_debug_set_jit(before)
            ra = self.red_prog.arrays()
            # four launches back to back, each on another 8192 x 8192 tensor (134 MB each, so none is still in L2)
            red_ins = [d["x"], d["dout"], o["out"], o["dx"]]
            for key in ("sum1", "max1", "arg1", "sum0"):
                self.flush_l2()
                with tm.region("a8." + key, launches=len(red_ins)):
                    for xin in red_ins:
                        B.relay_fused_reduce(ra, [xin], self.red_specs[key], [self.red_out[key]], ws)
        if "cfg3" in self.groups:
            d, o = self.devt["cfg3"], self.out["cfg3"]
            self.flush_l2()
            acts = [d["x"], o["y0"], o["y1"], o["y2"]]
            with tm.region("cfg3.fwd"):
                for l in range(3):
                    with tm.region("cfg3.fwd.layer"):
                        B.relay_fused_dense_act(acts[l], d[f"w{l}"], d[f"b{l}"], B.ACT_RELU, acts[l + 1], ws)
            with tm.region("cfg3.bwd"):
                g = d["dy"]
                for l in (2, 1, 0):
                    B.relay_fused_dense_act_grad(acts[l], d[f"w{l}"], acts[l + 1], g, B.ACT_RELU, o[f"dx{l}"], o[f"dw{l}"],
                                                 o[f"db{l}"], ws)
                    g = o[f"dx{l}"]
            # the two gradient contractions of one layer alone, each with its operand read transposed in place
            with tm.region("cfg3.bwd.gemm_dx"):
                B.relay_contract_act(d["dy"], 0, d["w2"], 1, None, B.ACT_NONE, o["dx2"])
            with tm.region("cfg3.bwd.gemm_dw"):
                B.relay_contract_act(acts[2], 1, d["dy"], 0, None, B.ACT_NONE, o["dw2"])
        if "cfg4" in self.groups:
            d, o = self.devt["cfg4"], self.out["cfg4"]
            self.flush_l2()
            with tm.region("cfg4.fwd"):
                B.relay_fused_conv2d_act(d["x"], d["w"], d["b"], 1, 1, B.ACT_RELU, o["y"], ws)
            self.flush_l2()
            with tm.region("cfg4.grad"):
                B.relay_fused_conv2d_act_grad(d["x"], d["w"], o["y"], d["dy"], 1, 1, B.ACT_RELU, o["dx"], o["dw"], o["db"], ws)
        if "cfg5" in self.groups:
            d, o = self.devt["cfg5"], self.out["cfg5"]
            self.flush_l2()
            with tm.region("cfg5.lstm"):
                B.relay_lstm_cell_seq(d["x"], d["w_ih"], d["w_hh"], d["b"], d["h0"], d["c0"], o["h_all"], o["c"], ws)
            T_, Bn_, In_ = d["x"].shape
            self.flush_l2()
            with tm.region("cfg5.lstm.zx_gemm"):
                B.relay_contract_act(d["x"].view(T_ * Bn_, In_), 0, d["w_ih"], 0, d["b"], B.ACT_NONE, self.lstm_zx)
            self.flush_l2()
            with tm.region("cfg5.lstm_grad"):
                B.relay_lstm_cell_seq_grad(d["x"], d["w_ih"], d["w_hh"], d["b"], d["h0"], d["c0"], o["h_all"], self.lstm_dh_all,
                                           self.lstm_dc_fin, o["dx"], o["dw_ih"], o["dw_hh"], o["db"], o["dh0"], o["dc0"], ws)

        if "next" in self.groups:
            d, o = self.devt["next"], self.out["next"]
            self.flush_l2()
            with tm.region("next.loss"):
                B.relay_softmax_xent(d["scores"], d["targets"], o["loss"])
            self.flush_l2()
            with tm.region("next.loss_grad"):
                B.relay_softmax_xent_grad(d["scores"], d["targets"], d["dloss"], o["loss2"], o["dscores"])
            self.flush_l2()
            with tm.region("next.sgd"):
                B.relay_sgd_update(self.sgd_params, self.sgd_grads, 1e-3)
            self.flush_l2()
            with tm.region("next.pool", launches=len(self.pool_sets)):
                for ps in self.pool_sets:
                    B.relay_max_pool2d(ps["x"], 2, 2, 2, 2, ps["y"], ps["idx"])
            self.flush_l2()
            with tm.region("next.pool_grad", launches=len(self.pool_sets)):
                for ps in self.pool_sets:
                    B.relay_max_pool2d_grad(ps["idx"], ps["dy"], 2, 2, 2, 2, ps["dx"])
            with tm.region("next.lenet"):
                self.lenet.run()
            if self.lenet.graph is not None:
                with tm.region("next.lenet_graph"):
                    self.lenet.graph.replay()
            h = self.nhwc
            self.flush_l2()
            with tm.region("next.conv_nhwc"):
                B.relay_fused_conv2d_act(h["x"], h["w"], h["b"], 1, 1, B.ACT_RELU, h["y"], ws, layout=B.NHWC)
            self.flush_l2()
            with tm.region("next.conv_nhwc_grad"):
                B.relay_fused_conv2d_act_grad(h["x"], h["w"], h["y"], h["dy"], 1, 1, B.ACT_RELU, h["dx"], h["dw"], h["db"], ws, layout=B.NHWC)

    # -- algorithmic work per step -------------------------------------------------------------------------
    def work(self):
        w = {}
        if "cfg1" in self.groups:
            w["cfg1.fwd"] = dict(flop=2 * 8 * 64 * 32); w["cfg1.grad"] = dict(flop=2 * 2 * 8 * 64 * 32 + 8 * 32 * 2)
            w["cfg1.graph"] = dict(flop=w["cfg1.fwd"]["flop"] + w["cfg1.grad"]["flop"])
            w["cfg1.fwd.kernel"] = dict(w["cfg1.fwd"]); w["cfg1.grad.kernel"] = dict(w["cfg1.grad"])
            w["cfg1.fp32_mid.fwd"] = dict(flop=2 * self.f32_mid["x"].shape[0] ** 3)
        if "cfg2" in self.groups:
            r, c = self.host["cfg2"]["x"].shape
            w["cfg2.fwd"] = dict(bytes=2 * r * c * 2 + 2 * c * 2)
            w["cfg2.grad"] = dict(bytes=3 * r * c * 2 + 2 * c * 2 + 2 * c * 4)
            for tag in ("jit", "vm"):
                w[f"a6.{tag}_fwd"] = dict(bytes=3 * r * c * 2 + c * 2); w[f"a7.{tag}_grad"] = dict(bytes=5 * r * c * 2 + c * 2 + c * 4)
            w["a8.sum1"] = dict(bytes=r * c * 2 + r * 4); w["a8.max1"] = dict(bytes=r * c * 2 + r * 4)
            w["a8.arg1"] = dict(bytes=r * c * 2 + r * 8); w["a8.sum0"] = dict(bytes=r * c * 2 + c * 4)
        if "cfg3" in self.groups:
            m, k = self.host["cfg3"]["x"].shape
            w["cfg3.fwd"] = dict(flop=3 * 2 * m * k * k); w["cfg3.bwd"] = dict(flop=6 * 2 * m * k * k)
            w["cfg3.fwd.layer"] = dict(flop=2 * m * k * k)
            w["cfg3.bwd.gemm_dx"] = dict(flop=2 * m * k * k); w["cfg3.bwd.gemm_dw"] = dict(flop=2 * m * k * k)
        if "cfg4" in self.groups:
            n, c, h, wd = self.host["cfg4"]["x"].shape
            o = self.host["cfg4"]["w"].shape[0]
            f = 2 * n * h * wd * o * c * 9
            w["cfg4.fwd"] = dict(flop=f); w["cfg4.grad"] = dict(flop=2 * f)
        if "cfg5" in self.groups:
            T, Bn, In = self.host["cfg5"]["x"].shape
            H = self.host["cfg5"]["w_hh"].shape[0]
            w["cfg5.lstm"] = dict(flop=2 * T * Bn * (In + H) * 4 * H)
            w["cfg5.lstm.zx_gemm"] = dict(flop=2 * T * Bn * In * 4 * H)
            # gradient program: gate recomputation (one forward's worth), dz w_hh^T per step, dx, dw_ih, dw_hh
            w["cfg5.lstm_grad"] = dict(flop=2 * T * Bn * (In + H) * 4 * H + 2 * T * Bn * 4 * H * (H + In) + 2 * T * Bn * 4 * H * (In + H))
        if "next" in self.groups:
            r, c = self.host["next"]["scores"].shape
            w["next.loss"] = dict(bytes=2 * r * c * 2 + r * 4)
            w["next.loss_grad"] = dict(bytes=3 * r * c * 2 + 2 * r * 4)
            w["next.sgd"] = dict(bytes=sum(3 * p.numel() * 2 for p in self.sgd_params))
            pool_bytes = self.pool_x.numel() * 2 + self.pool_y.numel() * (2 + 4)
            w["next.pool"] = dict(bytes=pool_bytes); w["next.pool_grad"] = dict(bytes=pool_bytes)
            n, h, wd, c = self.nhwc["x"].shape
            f = 2 * n * h * wd * self.nhwc["w"].shape[0] * c * 9
            w["next.conv_nhwc"] = dict(flop=f); w["next.conv_nhwc_grad"] = dict(flop=2 * f)
            w["next.lenet"] = dict(flop=self.lenet.flop()); w["next.lenet_graph"] = dict(flop=self.lenet.flop())
        return w


# ---------------------------------------------------------------------------------------------------
# CPU oracle on a bounded sample (single thread); also the `--impl reference` arm
# ---------------------------------------------------------------------------------------------------
def oracle_sample(rows3=192, rows2=1024, imgs4=1, rows5=2, reps1=200):
    """Times the fp64 oracle, as it stands, single-threaded, on slices of all five configurations along their
    independent dimension (batch rows / images; configuration 1 at full size).  Returns a dict: the aggregate rates
    over the sampled work (TFLOP/s over the dense + conv samples, GB/s of algorithmic bytes over the elementwise
    sample), the seconds spent, a description, and per configuration the sampled time with the full-size time it
    extrapolates to (linear in the sliced dimension)."""
    import oracle
    from relay_workloads import inputs as I
    from relay_workloads import program as P
    per = {}
    # configuration 1: full size, forward + gradient group, repeated (a single pass is microseconds)
    t1 = I.cfg1_tiny_mlp()
    x, w, b, dy = (I.as_f64(t1[k]) for k in ("x", "w", "b", "dy"))
    t0 = time.perf_counter()
    for _ in range(reps1):
        y = oracle.dense_act(x, w, b, oracle.ACT_RELU, oracle.F32)
        oracle.dense_act_grad(x, w, y, dy, oracle.ACT_RELU, oracle.F32, oracle.F32, oracle.F32)
    s1 = (time.perf_counter() - t0) / reps1
    per["cfg1"] = {"sample": "full size, forward + gradient group", "us_per_pass": s1 * 1e6, "flop": 3 * 2 * 8 * 64 * 32}
    # configuration 2: forward and gradient group on the first rows2 rows
    t2 = I.cfg2_ewise(rows=rows2)
    prog, outs = P.tanh_affine_residual_fwd(P.BF16)
    gprog, gids = P.tanh_affine_residual_grad(P.BF16)
    ins = [I.as_f64(t2[k]) for k in ("x", "a", "b")]
    gins = [I.as_f64(t2[k]) for k in ("dout", "x", "a", "b")]
    t0 = time.perf_counter()
    oracle.ewise(prog.arrays(), ins, outs)
    s2f = time.perf_counter() - t0
    t0 = time.perf_counter()
    oracle.reduce(gprog.arrays(), gins, [(gids[0], 0, (), False, oracle.BF16), (gids[1], 1, (0,), False, oracle.F32),
                                         (gids[2], 1, (0,), True, oracle.F32)])
    s2g = time.perf_counter() - t0
    bytes2 = (2 + 3) * rows2 * 8192 * 2
    per["cfg2"] = {"sample": f"first {rows2} of 8192 rows, forward + gradient group", "seconds": s2f + s2g,
                   "full_size_seconds_extrapolated": (s2f + s2g) * 8192 / rows2, "bytes": bytes2}
    # configuration 3: one layer forward + gradient group on the first rows3 batch rows
    t3 = I.cfg3_mlp(batch=rows3, layers=1)
    x, w, b, dy = (I.as_f64(t3[k]) for k in ("x", "w0", "b0", "dy"))
    t0 = time.perf_counter()
    y = oracle.dense_act(x, w, b, oracle.ACT_RELU, oracle.BF16)
    oracle.dense_act_grad(x, w, y, dy, oracle.ACT_RELU, oracle.BF16, oracle.BF16, oracle.F32)
    s3 = time.perf_counter() - t0
    flop3 = 3 * 2 * rows3 * 4096 * 4096
    per["cfg3"] = {"sample": f"one layer forward + gradient group on the first {rows3} of 4096 batch rows", "seconds": s3,
                   "full_size_seconds_extrapolated": s3 * 3 * 4096 / rows3, "flop": flop3}
    # configuration 4: forward + gradient group on the first imgs4 images
    t4 = I.cfg4_conv(N=imgs4)
    x, w, b, dy = (I.as_f64(t4[k]) for k in ("x", "w", "b", "dy"))
    t0 = time.perf_counter()
    y = oracle.conv2d_act(x, w, b, 1, 1, oracle.ACT_RELU, oracle.BF16)
    oracle.conv2d_act_grad(x, w, y, dy, 1, 1, oracle.ACT_RELU, oracle.BF16, oracle.BF16, oracle.F32)
    s4 = time.perf_counter() - t0
    flop4 = 3 * 2 * imgs4 * 56 * 56 * 256 * 256 * 9
    per["cfg4"] = {"sample": f"forward + dX + dW + db on the first {imgs4} of 32 images", "seconds": s4,
                   "full_size_seconds_extrapolated": s4 * 32 / imgs4, "flop": flop4}
    # configuration 5: the whole sequence (128 steps) for the first rows5 batch rows
    t5 = I.cfg5_lstm(B=rows5)
    a5 = [I.as_f64(t5[k]) for k in ("x", "w_ih", "w_hh", "b", "h0", "c0")]
    t0 = time.perf_counter()
    oracle.lstm_cell_seq(*a5)
    s5 = time.perf_counter() - t0
    flop5 = 2 * 128 * rows5 * 2048 * 4096
    per["cfg5"] = {"sample": f"all 128 steps for the first {rows5} of 64 batch rows (forward)", "seconds": s5,
                   "full_size_seconds_extrapolated": s5 * 64 / rows5, "flop": flop5}
    sec = s1 * reps1 + s2f + s2g + s3 + s4 + s5
    desc = (f"cfg1 full size x{reps1} ({s1 * 1e6:.0f} us per pass); cfg2 forward+gradient on the first {rows2} rows ({bytes2 / 1e6:.1f} MB, "
            f"{s2f + s2g:.1f} s); cfg3 one layer forward+gradient on the first {rows3} batch rows ({flop3 / 1e9:.1f} GFLOP, {s3:.1f} s); "
            f"cfg4 forward+gradient on the first {imgs4} image(s) ({flop4 / 1e9:.1f} GFLOP, {s4:.1f} s); cfg5 forward, 128 steps, "
            f"first {rows5} batch rows ({flop5 / 1e9:.1f} GFLOP, {s5:.1f} s); full-size times are extrapolated linearly")
    return {"tflops": (flop3 + flop4) / (s3 + s4) / 1e12, "gbs": bytes2 / (s2f + s2g) / 1e9, "seconds": sec, "desc": desc, "per_config": per}


def run_reference(args, rank, world):
    if rank != 0:
        return
    vals = []
    for i in range(args.warmup + args.steps):
        r = oracle_sample(rows3=16, rows2=64, imgs4=1, rows5=1, reps1=20)
        if i >= args.warmup:
            vals.append(r)
    tf = float(np.mean([v["tflops"] for v in vals])); gb = float(np.mean([v["gbs"] for v in vals])); sec = float(np.mean([v["seconds"] for v in vals]))
    desc = vals[-1]["desc"] if vals else ""
    line = {"impl": "reference", "metric": METRIC, "value": tf, "unit": "TFLOP/s", "hbm_gbs": gb, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": "all five configurations; each step = the oracle on a bounded sample: " + desc},
            "cpu_baseline": {"value": tf, "unit": "TFLOP/s", "cores": 1, "kind": "oracle", "sample": desc},
            "e2e": {"value": tf, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}, "gpu_launches": 0}
    print(json.dumps(line))


def max_over_ranks(value_ms: float, dist, device) -> float:
    """Multi-GPU numbers are the MAX over ranks of the device time (replicas run independently)."""
    t = torch.tensor([value_ms], dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job(per_rank_units: float, world: int, ms: float) -> float:
    """Weak scaling: every replica processes `per_rank_units` in `ms` (max over ranks)."""
    return world * per_rank_units / (ms * 1e-3) if ms else 0.0


# ---------------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--groups", default=",".join(ALL_GROUPS))
    ap.add_argument("--small", action="store_true", help="reduced shapes (for profiler captures and quick checks)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0")); world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        return run_reference(args, rank, world)
    if args.warmup < 3:
        args.warmup = 3 if not args.small else args.warmup

    from paper_1810_00952_b200 import binding as B
    B.lib()   # fails loudly if the CUDA library is missing
    assert torch.cuda.is_available(), "bench.py needs a CUDA device"
    dev = torch.device(f"cuda:{local}")
    torch.cuda.set_device(dev)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    groups = [g for g in args.groups.split(",") if g]
    wl = Workload(dev, groups, small=args.small)
    work = wl.work()
    peaks = load_peaks()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    tm = Timer()
    sampler = ClockSampler(local); sampler.start()
    wl.step(tm)                      # first use of every kernel, outside the capture
    torch.cuda.synchronize()
    wl.capture_graphs()
    for _ in range(args.warmup):
        wl.step(tm)
    tm.collect(); tm.ms = {}
    B.relay_poll_status()

    barrier()
    sampler.begin()
    n0 = B.relay_launch_count()
    t_all0 = torch.cuda.Event(enable_timing=True); t_all1 = torch.cuda.Event(enable_timing=True)
    t_all0.record()
    for _ in range(args.steps):
        wl.step(tm)
    t_all1.record()
    barrier()
    launches = (B.relay_launch_count() - n0) // max(args.steps, 1)
    tm.collect()
    clocks = sampler.stop()
    B.relay_poll_status()

    # per-group device time (sum of the groups' regions; L2 flushes between groups are not counted)
    top = [k for k in tm.ms if k.count(".") == 1]
    med = {k: float(np.median(v)) for k, v in tm.ms.items()}
    step_ms = sum(float(np.mean(tm.ms[k])) for k in top)
    step_ms_max = max_over_ranks(step_ms, dist, dev)

    tensor_keys = [k for k in top if k.startswith(("cfg3", "cfg4"))]
    hbm_keys = [k for k in top if k.startswith("cfg2")]
    t_ms = max_over_ranks(sum(float(np.mean(tm.ms[k])) for k in tensor_keys), dist, dev)
    h_ms = max_over_ranks(sum(float(np.mean(tm.ms[k])) for k in hbm_keys), dist, dev)
    tflops = whole_job(sum(work[k]["flop"] for k in tensor_keys), world, t_ms) / 1e12 if t_ms else None
    gbs = whole_job(sum(work[k]["bytes"] for k in hbm_keys), world, h_ms) / 1e9 if h_ms else None

    table = {}
    for k in sorted(tm.ms):
        ms = float(np.mean(tm.ms[k])) if k.count(".") == 1 else float(np.mean(tm.ms[k]))
        e = {"ms": round(ms, 5), "ms_median": round(med[k], 5), "ms_best": round(float(np.min(tm.ms[k])), 5)}
        if "flop" in work.get(k, {}):
            e["tflops"] = work[k]["flop"] / (ms * 1e-3) / 1e12
            e["frac_of_measured_bf16_peak"] = e["tflops"] / peaks["bf16_tflops"]
            e["frac_of_nominal_bf16_peak"] = e["tflops"] / NOMINAL_PEAKS["bf16_tflops"]
        if "bytes" in work.get(k, {}):
            e["gbs"] = work[k]["bytes"] / (ms * 1e-3) / 1e9
            e["frac_of_measured_hbm"] = e["gbs"] / peaks["hbm_gbs"]
            e["frac_of_nominal_hbm"] = e["gbs"] / NOMINAL_PEAKS["hbm_gbs"]
        table[k] = e

    # roofline of the dominant roofline-bound kernel: the tensor-core contraction (its three operand
    # layouts together are the largest tensor-bound share of the step); one forward layer call = one launch
    def traffic_of(kernel):
        """DRAM bytes per launch from the committed ncu capture, or None once the kernel source changed."""
        try:
            import hashlib
            t = json.load(open(os.path.join(ROOT, "profiles", "traffic.json")))[kernel]
            src = os.path.join(ROOT, t["source"])
            return t["dram_bytes_per_launch"] if hashlib.sha256(open(src, "rb").read()).hexdigest() == t["source_sha256"] else None
        except Exception:
            return None

    roofline, rooflines = None, {}
    if "cfg3.fwd" in table:
        # three launches back to back; the per-launch duration is the region's time / 3, so that the
        # overlap of one launch's set-up with the previous launch's tail is not counted twice
        a = table["cfg3.fwd"]["tflops"]
        rooflines["gemm_tc2_kernel (cfg3 forward, 3 launches of 4096^3)"] = {
            "bound": "tensor", "achieved": a, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": a / peaks["bf16_tflops"],
            "traffic": traffic_of("gemm_tc2_kernel"), "peak_source": peaks["source"] + " (burst, of measured)",
            "us_per_launch": table["cfg3.fwd"]["ms"] * 1e3 / 3,
            # the launches run inside a step of several milliseconds of device work: the sustained figure for context
            "frac_of_sustained_peak": a / peaks["bf16_tflops_sustained"] if peaks.get("bf16_tflops_sustained") else None}
    for key, name in (("cfg3.bwd.gemm_dx", "gemm_tc2_kernel, dx = dZ w^T (both operands K-major), one 4096^3 launch"),
                      ("cfg3.bwd.gemm_dw", "gemm_tc2_kernel, dw = x^T dZ (both operands MN-major), one 4096^3 launch"),
                      ("cfg5.lstm.zx_gemm", "gemm_tc2_kernel, zx = x W_ih + b for all T*B rows (8192 x 4096 x 1024, fp32 result)")):
        if key in table:
            a = table[key]["tflops"]
            rooflines[name] = {"bound": "tensor", "achieved": a, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": a / peaks["bf16_tflops"],
                               "traffic": None, "peak_source": peaks["source"] + " (burst, of measured)", "us_per_launch": table[key]["ms"] * 1e3}
    if "cfg4.fwd" in table:
        a = table["cfg4.fwd"]["tflops"]
        rooflines["conv2d forward group (repack + conv_fprop_tc_kernel)"] = {
            "bound": "tensor", "achieved": a, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": a / peaks["bf16_tflops"],
            "traffic": traffic_of("conv_fprop_tc2_kernel"), "peak_source": peaks["source"] + " (burst, of measured)"}
    for key, name in (("cfg4.grad", "conv2d gradient group (repacks + conv_fprop_tc_kernel on dZ + conv_wgrad_tc_kernel + reduce)"),
                      ("next.conv_nhwc", "conv2d forward group, NHWC-tagged tensors (conv_fprop_tc_kernel storing NHWC tiles)"),
                      ("next.conv_nhwc_grad", "conv2d gradient group, NHWC-tagged tensors")):
        if key in table:
            a = table[key]["tflops"]
            rooflines[name] = {"bound": "tensor", "achieved": a, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": a / peaks["bf16_tflops"],
                               "traffic": None, "peak_source": peaks["source"] + " (burst, of measured)"}
    for key, name in (("cfg2.fwd", "ewise2d_kernel<tanh_affine_residual_fwd>"), ("cfg2.grad", "ewise2d_kernel<tanh_affine_residual_grad> + finalize")):
        if key in table:
            a = table[key]["gbs"]
            rooflines[name] = {"bound": "hbm", "achieved": a, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": a / peaks["hbm_gbs"],
                               "traffic": traffic_of(key), "peak_source": peaks["source"] + " (of measured)"}
    for key, name in (("a6.jit_fwd", "relay_jit_kernel, out = sigmoid(x*y) + relu(z) (8192x8192 bf16, body compiled at run time)"),
                      ("a7.jit_grad", "relay_jit_kernel + finalize, gradient group of the same (dx, dy, column sum dz)"),
                      ("a6.vm_fwd", "ewise_vm_kernel, the same forward program on the in-kernel interpreter (run-time compiler switched off)"),
                      ("a7.vm_grad", "ewise_vm_kernel + finalize, the same gradient group on the interpreter"),
                      ("a8.sum1", "rowreduce_kernel<sum> (8192x8192 bf16 over the last axis)"),
                      ("a8.max1", "rowreduce_kernel<max> (8192x8192 bf16 over the last axis)"),
                      ("a8.arg1", "rowreduce_kernel<argmax> (8192x8192 bf16 over the last axis, int64 indices)"),
                      ("a8.sum0", "ewise2d_kernel<identity_colsum> + finalize (8192x8192 bf16 over axis 0)")):
        if key in table:
            a = table[key]["gbs"]
            rooflines[name] = {"bound": "hbm", "achieved": a, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": a / peaks["hbm_gbs"],
                               "traffic": traffic_of(key), "peak_source": peaks["source"] + " (of measured)"}
    for key, name in (("next.loss", "softmax_xent_kernel (loss)"), ("next.loss_grad", "softmax_xent_kernel (loss + partial)"),
                      ("next.sgd", "sgd_update_kernel (3 x 4096^2 bf16)"), ("next.pool", "max_pool_2x2_kernel (32x256x56x56 bf16)"),
                      ("next.pool_grad", "max_pool_2x2_grad_kernel (32x256x56x56 bf16)")):
        if key in table:
            a = table[key]["gbs"]
            rooflines[name] = {"bound": "hbm", "achieved": a, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": a / peaks["hbm_gbs"],
                               "traffic": traffic_of(key), "peak_source": peaks["source"] + " (of measured)"}
    # LSTM sequence and its gradient program: tensor-core work on a chain of T dependent steps; the fraction of the
    # tensor peak is reported for the record (the chain, not the tensor pipe, bounds them)
    for key, name in (("cfg5.lstm", "relay_lstm_cell_seq (zx contraction + lstm_persistent_kernel, T=128 dependent steps)"),
                      ("cfg5.lstm_grad", "relay_lstm_cell_seq_grad (recompute + lstm_grad_cluster_kernel + dx/dW contractions)")):
        if key in table:
            a = table[key]["tflops"]
            rooflines[name] = {"bound": "tensor", "achieved": a, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": a / peaks["bf16_tflops"],
                               "traffic": None, "peak_source": peaks["source"] + " (burst, of measured)",
                               "us_per_step": table[key]["ms"] * 1e3 / 128, "note": "latency chain of dependent steps"}
    if "cfg1.fp32_mid.fwd" in table:
        # ALU bound of the fp32 tier: every SM issues 128 fp32 FMA lanes per cycle = 256 FLOP per cycle and SM
        sms = torch.cuda.get_device_properties(dev).multi_processor_count
        mhz = clocks.get("sm_mhz") or 1965.0
        peak_alu = sms * 128 * 2 * mhz * 1e6 / 1e12
        a = table["cfg1.fp32_mid.fwd"]["tflops"]
        rooflines["gemm_simt_big_kernel (fp32 1024^3, true fp32 FMA with compensated run sums)"] = {
            "bound": "alu", "achieved": a, "peak": peak_alu, "unit": "TFLOP/s", "frac": a / peak_alu, "traffic": None,
            "peak_source": f"derived: {sms} SMs x 128 FMA lanes x 2 FLOP x {mhz:.0f} MHz (SM clock sampled during the run)"}
    for r_ in rooflines.values():
        if r_["bound"] == "alu":
            continue
        r_["frac_of_nominal"] = r_["achieved"] / NOMINAL_PEAKS["bf16_tflops" if r_["unit"] == "TFLOP/s" else "hbm_gbs"]
    if rooflines:
        first = next(iter(rooflines))
        roofline = dict(rooflines[first], kernel=first)

    # end to end: pinned host inputs -> device, the step, results -> pinned host, all inside the timed region
    e2e = None
    if not args.no_e2e:
        # Every step uploads its inputs from pinned host memory and reads all of its results back.  Three streams and two
        # sets of device buffers: while step i computes, the inputs of step i+1 upload into the other set and the results
        # of step i-1 are read back from it (the two directions of the link run concurrently).  A set's inputs are not
        # overwritten before the compute that read them has ended, nor its results before their read-back has.
        tm2 = Timer()
        h2d = d2h = 0
        main_s = torch.cuda.current_stream()
        up_s, d2h_s = torch.cuda.Stream(), torch.cuda.Stream()
        wl.make_alternate()
        comp_done, dl_done = [None, None], [None, None]

        def e2e_step(i):
            nonlocal h2d, d2h
            k = i & 1
            wl.swap()
            with torch.cuda.stream(up_s):
                if comp_done[k] is not None:
                    up_s.wait_event(comp_done[k])
                h2d = wl.upload()
                up_done = torch.cuda.Event(); up_done.record(up_s)
            main_s.wait_event(up_done)
            if dl_done[k] is not None:
                main_s.wait_event(dl_done[k])
            wl.step(tm2)
            comp_done[k] = torch.cuda.Event(); comp_done[k].record(main_s)
            with torch.cuda.stream(d2h_s):
                d2h_s.wait_event(comp_done[k])
                d2h = wl.download()
                dl_done[k] = torch.cuda.Event(); dl_done[k].record(d2h_s)

        def drain():
            for e in dl_done:
                if e is not None:
                    main_s.wait_event(e)

        for i in range(2):
            e2e_step(i)
        drain()
        barrier()
        a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
        n_e2e = 2 * max(1, min(args.steps, 20) // 2)
        a.record()
        up_s.wait_event(a)
        for i in range(n_e2e):
            e2e_step(i)
        drain()
        b.record()
        barrier()
        e_ms = max_over_ranks(a.elapsed_time(b) / n_e2e, dist, dev)
        flop_all = sum(work[k]["flop"] for k in tensor_keys)
        e2e = {"value": world * flop_all / (e_ms * 1e-3) / 1e12 if flop_all else None, "unit": "TFLOP/s", "ms_per_step": e_ms,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "note": "whole step incl. L2 flushes and all groups, inputs uploaded and all results read back every step "
                       "(pipelined over two buffer sets: upload of the next step and read-back of the previous one overlap the compute); "
                       "dense+conv FLOPs over that time"}

    # cfg5: where a step of the persistent kernel spends its time (one extra call, outside every timed region)
    lstm_phases = None
    if "cfg5" in groups and not args.small:
        try:
            d, o = wl.devt["cfg5"], wl.out["cfg5"]
            cyc = torch.zeros(8, dtype=torch.int64, device=dev)
            B.relay_debug_lstm_phase_cycles(d["x"], d["w_ih"], d["w_hh"], d["b"], d["h0"], d["c0"], o["h_all"], o["c"], wl.ws, cyc)
            torch.cuda.synchronize()
            c = [int(v) for v in cyc.cpu()]
            mhz = clocks.get("sm_mhz") or 1965.0
            T_ = max(c[7], 1)
            us = lambda v: v / T_ / mhz
            lstm_phases = {"us_per_step": us(c[0]), "loader_waits_for_grid_barrier_us": us(c[3]), "loader_issues_copies_us": us(c[4]),
                           "issuer_waits_for_first_stage_us": us(c[5]), "issuer_first_stage_to_last_commit_us": us(c[6]),
                           "epilogue_waits_for_product_us": us(c[1]), "epilogue_gates_and_publish_us": us(c[2]),
                           "note": "cycle counts of block 0 summed over the steps / T / sampled SM clock; the phases of the three warp roles overlap"}
        except Exception as e:      # the breakdown is a report, not a gate
            lstm_phases = {"error": str(e)}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        r = oracle_sample()
        cpu = {"value": r["tflops"], "unit": "TFLOP/s", "hbm_gbs": r["gbs"], "cores": 1, "kind": "oracle", "sample": r["desc"],
               "per_config": r["per_config"], "seconds": r["seconds"], "host_cores_available": os.cpu_count()}

    if rank == 0:
        line = {"metric": METRIC, "value": tflops if tflops is not None else gbs, "unit": "TFLOP/s" if tflops is not None else "GB/s",
                "hbm_gbs": gbs, "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_ms_max,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16 (fp32 accumulate); cfg1 f32",
                "data": "synthetic",
                "config": {"workload": ("reduced shapes" if args.small else "all five configurations at full size")
                           + ": step = cfg1 fwd+grad, cfg2 fwd+grad, an elementwise program and its gradient group on the vectorised evaluator, four standalone reductions of the cfg2 tensor (sum / max / argmax over the last axis, sum over axis 0), cfg3 3-layer fwd+bwd, cfg4 conv fwd+dX+dW+db, cfg5 LSTM forward + gradient program"
                           + ", then softmax cross-entropy loss / loss+partial on 8192x8192 bf16, SGD on three 4096^2 bf16 matrices and 2x2 max pooling"
                           + " forward + gradient on 32x256x56x56 bf16, one fp32 LeNet training step (batch 64) eager and replayed from a"
                           + " CUDA graph, the cfg4 conv with NHWC-tagged tensors; cfg1 is also replayed from a CUDA graph",
                           "value_covers": "dense + conv2d groups (cfg3 + cfg4) FLOPs / their device time; hbm_gbs covers cfg2 (the configuration's own two groups); a program without a pre-compiled body (a6.jit_fwd, a7.jit_grad: compiled at run time; a6.vm_fwd, a7.vm_grad: interpreted) and the standalone reductions (a8.*) are reported per group",
                           "groups": groups, "l2": "1 GiB streamed through L2 between groups (flush with clean lines); cfg2 inputs also exceed L2; the standalone reductions and "
                                 "the pooling kernels are timed as four back-to-back launches on four different sets of tensors (per-launch time = region / 4)",
                           "replicas": world},
                "groups": table, "roofline": roofline, "rooflines": rooflines, "cfg5_step_phases": lstm_phases, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": int(launches),
                "clocks": clocks, "peaks": dict({k: peaks.get(k) for k in ("hbm_gbs", "bf16_tflops", "bf16_tflops_sustained", "source")}, nominal=NOMINAL_PEAKS)}
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
