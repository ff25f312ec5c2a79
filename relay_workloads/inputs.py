"""Seeded synthetic inputs shaped like the benchmark configurations.

Only random tensors are made here -- none of the operators' arithmetic.  Every tensor is drawn
in fp64 from a counter-based generator (Philox, seeded per configuration and per tensor),
rounded once to its storage dtype, and returned as a CPU torch tensor; the CUDA path uploads
it and the CPU oracle reads its exact values as fp64.

The second argument of N(.,.) is a standard deviation throughout.
"""
from __future__ import annotations

import math
from typing import Dict

import numpy as np
import torch

SEED_BASE = 0x5EED0000


def _rng(cfg: int, tensor: int, salt: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=SEED_BASE + cfg * 16 + tensor + (salt << 32)))


def _store(a: np.ndarray, dtype: torch.dtype) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).to(dtype).contiguous()


def normal(cfg, tensor, shape, std, dtype, salt=0):
    return _store(_rng(cfg, tensor, salt).standard_normal(shape) * std, dtype)


def uniform(cfg, tensor, shape, lo, hi, dtype, salt=0):
    return _store(_rng(cfg, tensor, salt).uniform(lo, hi, shape), dtype)


def as_f64(t: torch.Tensor) -> np.ndarray:
    """Exact values of a stored tensor as fp64 (what the oracle consumes)."""
    return t.to(torch.float64).numpy()


def cfg1_tiny_mlp(M=8, K=64, N=32, salt=0) -> Dict[str, torch.Tensor]:
    """fp32 layer y = relu(x @ W + b) and upstream gradient dy, all ~ N(0,1)."""
    f = torch.float32
    return dict(x=normal(1, 0, (M, K), 1.0, f, salt), w=normal(1, 1, (K, N), 1.0, f, salt),
                b=normal(1, 2, (N,), 1.0, f, salt), dy=normal(1, 3, (M, N), 1.0, f, salt))


def cfg2_ewise(rows=8192, cols=8192, dtype=torch.bfloat16, salt=0) -> Dict[str, torch.Tensor]:
    """out = tanh(a*x+b)+x: x ~ N(0,1) [rows, cols]; a ~ U(0.5,1.5) [cols]; b ~ N(0,0.1) [1, cols];
    dout ~ N(0,1) [rows, cols]."""
    return dict(x=normal(2, 0, (rows, cols), 1.0, dtype, salt),
                a=uniform(2, 1, (cols,), 0.5, 1.5, dtype, salt),
                b=normal(2, 2, (1, cols), 0.1, dtype, salt),
                dout=normal(2, 3, (rows, cols), 1.0, dtype, salt))


def cfg3_mlp(batch=4096, width=4096, layers=3, dtype=torch.bfloat16, salt=0) -> Dict[str, torch.Tensor]:
    """relu MLP: x ~ N(0,1) [batch, width]; W_l ~ N(0, 1/sqrt(width)); b_l = 0; dy ~ N(0,1)."""
    d = dict(x=normal(3, 0, (batch, width), 1.0, dtype, salt),
             dy=normal(3, 1, (batch, width), 1.0, dtype, salt))
    for l in range(layers):
        d[f"w{l}"] = normal(3, 2 + l, (width, width), 1.0 / math.sqrt(width), dtype, salt)
        d[f"b{l}"] = torch.zeros(width, dtype=dtype)
    return d


def cfg4_conv(N=32, C=256, H=56, W=56, O=256, R=3, S=3, dtype=torch.bfloat16, salt=0) -> Dict[str, torch.Tensor]:
    """conv2d 3x3 s1 p1 NCHW/OIHW: x ~ U(0,1); Wt ~ N(0, sqrt(2/(R*S*C))); b ~ N(0, 0.01);
    dy ~ N(0,1) with the output's shape (stride 1, pad (R-1)/2)."""
    return dict(x=uniform(4, 0, (N, C, H, W), 0.0, 1.0, dtype, salt),
                w=normal(4, 1, (O, C, R, S), math.sqrt(2.0 / (R * S * C)), dtype, salt),
                b=normal(4, 2, (O,), 0.01, dtype, salt),
                dy=normal(4, 3, (N, O, H, W), 1.0, dtype, salt))


def cfg5_lstm(T=128, B=64, I=1024, H=1024, salt=0) -> Dict[str, torch.Tensor]:
    """LSTM over a sequence: x ~ N(0,1) bf16 [T,B,I]; W_ih [I,4H], W_hh [H,4H] ~ U(-k,k) bf16 with
    k = 1/sqrt(H); b ~ U(-k,k) fp32 [4H]; h0 = c0 = 0 fp32 [B,H]."""
    k = 1.0 / math.sqrt(H)
    bf, f = torch.bfloat16, torch.float32
    return dict(x=normal(5, 0, (T, B, I), 1.0, bf, salt),
                w_ih=uniform(5, 1, (I, 4 * H), -k, k, bf, salt),
                w_hh=uniform(5, 2, (H, 4 * H), -k, k, bf, salt),
                b=uniform(5, 3, (4 * H,), -k, k, f, salt),
                h0=torch.zeros(B, H, dtype=f), c0=torch.zeros(B, H, dtype=f))


def loss_batch(B=8192, C=8192, dtype=torch.bfloat16, target_dtype=None, one_hot=False, salt=0) -> Dict[str, torch.Tensor]:
    """Inputs of the loss group: scores ~ N(0,2) [B,C]; targets [B,C] either one-hot rows (class drawn
    uniformly) or U(0,1) weights; dloss ~ N(0,1) fp32 [B] (the upstream partial)."""
    target_dtype = target_dtype or dtype
    r = _rng(6, 1, salt)
    if one_hot:
        t = np.zeros((B, C))
        if B and C:
            t[np.arange(B), r.integers(0, C, B)] = 1.0
    else:
        t = r.uniform(0.0, 1.0, (B, C))
    return dict(scores=normal(6, 0, (B, C), 2.0, dtype, salt), targets=_store(t, target_dtype),
                dloss=normal(6, 2, (B,), 1.0, torch.float32, salt))


def param_set(shapes, dtype=torch.bfloat16, grad_dtype=None, salt=0):
    """Parameters ~ N(0, 0.05) and gradients ~ N(0, 1) of the given shapes (lists of CPU tensors)."""
    grad_dtype = grad_dtype or dtype
    ps = [normal(7, 2 * i, s, 0.05, dtype, salt) for i, s in enumerate(shapes)]
    gs = [normal(7, 2 * i + 1, s, 1.0, grad_dtype, salt) for i, s in enumerate(shapes)]
    return ps, gs


def pool_input(N=32, C=256, H=56, W=56, dtype=torch.bfloat16, levels=0, salt=0) -> torch.Tensor:
    """Activations to pool: N(0,1) values, or (levels > 0) integers in [0, levels) so that windows hold ties."""
    if levels:
        return _store(_rng(8, 0, salt).integers(0, levels, (N, C, H, W)).astype(np.float64), dtype)
    return normal(8, 0, (N, C, H, W), 1.0, dtype, salt)


def lenet_batch(N=16, dtype=torch.float32, salt=0) -> Dict[str, torch.Tensor]:
    """One batch for the LeNet-shaped model of the paper's listing: images U(0,1) [N,1,28,28], one-hot labels
    [N,10], parameters N(0, 0.1) (the listing initialises every parameter as a small Gaussian)."""
    r = _rng(9, 1, salt)
    labels = np.zeros((N, 10))
    labels[np.arange(N), r.integers(0, 10, N)] = 1.0
    shapes = dict(w1=(20, 1, 5, 5), b1=(20,), w2=(50, 20, 5, 5), b2=(50,), w3=(800, 500), b3=(500,), w4=(500, 10), b4=(10,))
    d = dict(x=uniform(9, 0, (N, 1, 28, 28), 0.0, 1.0, dtype, salt), labels=_store(labels, dtype))
    for i, (k, s) in enumerate(shapes.items()):
        d[k] = normal(9, 2 + i, s, 0.1, dtype, salt)
    return d
