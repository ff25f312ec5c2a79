"""Description format of a fused elementwise group: a let-list of typed instructions.

This module only *describes* programs (lists of integers and literals); it evaluates nothing.
Both the CUDA library (through its C-ABI) and the CPU oracle receive the same description, each
interprets it with code of its own.

Value ids: 0 .. n_in-1 name the group's inputs; n_in + j names the result of instruction j
(the paper's `let id = e in ...`, Fig. 1).  The opcode set is Fig. 1's BinOp / UnaryOp
productions, the cast production, and the elementwise library operators (tanh etc., Fig. 3).
"""
from __future__ import annotations

from typing import List, Sequence

# dtype codes of the C-ABI
F32, BF16, I32, I64, BOOL = 0, 1, 2, 3, 4

# opcodes of the C-ABI
(OP_ADD, OP_SUB, OP_MUL, OP_DIV, OP_NEG, OP_SQ, OP_NE, OP_EQ, OP_LT, OP_LE, OP_GT, OP_GE,
 OP_SELECT, OP_RELU, OP_TANH, OP_SIGMOID, OP_CAST, OP_CONST, OP_EXP, OP_LOG, OP_MAX,
 OP_MIN) = range(22)

# reduction codes of the C-ABI
RED_NONE, RED_SUM, RED_MAX, RED_MEAN, RED_ARGMAX = range(5)

ACT_NONE, ACT_RELU, ACT_TANH, ACT_SIGMOID = range(4)


class Program:
    """Builder for an instruction list.  Result dtypes follow Fig. 5: arithmetic keeps the
    operand type, comparisons give Bool, cast gives the named type."""

    def __init__(self, in_dtypes: Sequence[int]):
        self.in_dtypes = list(in_dtypes)
        self.op: List[int] = []
        self.a: List[int] = []
        self.b: List[int] = []
        self.c: List[int] = []
        self.imm: List[float] = []
        self.dtype: List[int] = []

    # -- bookkeeping -------------------------------------------------------------------------
    @property
    def n_in(self) -> int:
        return len(self.in_dtypes)

    def input(self, i: int) -> int:
        assert 0 <= i < self.n_in
        return i

    def dtype_of(self, vid: int) -> int:
        return self.in_dtypes[vid] if vid < self.n_in else self.dtype[vid - self.n_in]

    def emit(self, op: int, a: int = -1, b: int = -1, c: int = -1, imm: float = 0.0, dtype: int = F32) -> int:
        self.op.append(op); self.a.append(a); self.b.append(b); self.c.append(c)
        self.imm.append(float(imm)); self.dtype.append(dtype)
        return self.n_in + len(self.op) - 1

    def arrays(self) -> dict:
        return dict(op=list(self.op), a=list(self.a), b=list(self.b), c=list(self.c),
                    imm=list(self.imm), dtype=list(self.dtype), in_dtypes=list(self.in_dtypes))

    # -- instructions ------------------------------------------------------------------------
    def _bin(self, op, x, y):
        return self.emit(op, x, y, dtype=self.dtype_of(x))

    def add(self, x, y): return self._bin(OP_ADD, x, y)
    def sub(self, x, y): return self._bin(OP_SUB, x, y)
    def mul(self, x, y): return self._bin(OP_MUL, x, y)
    def div(self, x, y): return self._bin(OP_DIV, x, y)
    def max(self, x, y): return self._bin(OP_MAX, x, y)
    def min(self, x, y): return self._bin(OP_MIN, x, y)

    def _un(self, op, x):
        return self.emit(op, x, dtype=self.dtype_of(x))

    def neg(self, x): return self._un(OP_NEG, x)
    def sq(self, x): return self._un(OP_SQ, x)
    def relu(self, x): return self._un(OP_RELU, x)
    def tanh(self, x): return self._un(OP_TANH, x)
    def sigmoid(self, x): return self._un(OP_SIGMOID, x)
    def exp(self, x): return self._un(OP_EXP, x)
    def log(self, x): return self._un(OP_LOG, x)

    def cmp(self, op, x, y):
        assert OP_NE <= op <= OP_GE
        return self.emit(op, x, y, dtype=BOOL)

    def select(self, cond, x, y):
        return self.emit(OP_SELECT, cond, x, y, dtype=self.dtype_of(x))

    def cast(self, x, dtype):
        return self.emit(OP_CAST, x, dtype=dtype)

    def const(self, value, dtype=F32):
        return self.emit(OP_CONST, imm=value, dtype=dtype)


# -------------------------------------------------------------------------------------------------
# The groups of the benchmark configurations
# -------------------------------------------------------------------------------------------------
def tanh_affine_residual_fwd(storage=BF16, math=F32):
    """out = tanh(a * x + b) + x; inputs (x, a, b) in `storage`, arithmetic in `math`, out in
    `storage`."""
    p = Program([storage, storage, storage])
    x, a, b = (p.cast(i, math) for i in range(3))
    t = p.tanh(p.add(p.mul(a, x), b))
    out = p.cast(p.add(t, x), storage)
    return p, [out]


def tanh_affine_residual_grad(storage=BF16, math=F32):
    """Gradient program of out = tanh(a*x+b)+x for upstream dout; inputs (dout, x, a, b).
    With u = a*x+b, t = tanh u, s = 1 - t^2:
        dx  = dout * (a*s + 1)      (x is used twice: the two partials are summed)
        da  = sum over rows of dout * s * x
        db  = sum over rows of dout * s
    Returns (program, [dx_id, da_elem_id, db_elem_id]); the last two are the per-element
    summands that a reduce group sums over axis 0."""
    p = Program([storage] * 4)
    d, x, a, b = (p.cast(i, math) for i in range(4))
    t = p.tanh(p.add(p.mul(a, x), b))
    one = p.const(1.0, math)
    s = p.sub(one, p.sq(t))
    g = p.add(p.mul(a, s), one)
    dx = p.cast(p.mul(d, g), storage)
    ds = p.mul(d, s)
    dae = p.mul(ds, x)
    return p, [dx, dae, ds]


def sigmoid_product_relu_fwd(storage=BF16, math=F32):
    """out = sigmoid(x * y) + relu(z); inputs (x, y, z) in `storage` (z may be constant down the rows), arithmetic in
    `math`, out in `storage`."""
    p = Program([storage, storage, storage])
    x, y, z = (p.cast(i, math) for i in range(3))
    out = p.cast(p.add(p.sigmoid(p.mul(x, y)), p.relu(z)), storage)
    return p, [out]


def sigmoid_product_relu_grad(storage=BF16, math=F32):
    """Gradient program of out = sigmoid(x*y) + relu(z) for upstream dout; inputs (dout, x, y, z).
    With s = sigmoid(x*y), ds = dout * s * (1 - s):  dx = ds * y,  dy = ds * x,  dz = dout where z > 0 else 0.
    Returns (program, [dx_id, dy_id, dz_elem_id]); when z is constant down the rows its partial is the sum of the last
    value over the rows (a value used by every row collects every row's contribution)."""
    p = Program([storage] * 4)
    d, x, y, z = (p.cast(i, math) for i in range(4))
    s = p.sigmoid(p.mul(x, y))
    one = p.const(1.0, math)
    ds = p.mul(d, p.mul(s, p.sub(one, s)))
    dx = p.cast(p.mul(ds, y), storage)
    dy = p.cast(p.mul(ds, x), storage)
    zero = p.const(0.0, math)
    dz = p.select(p.cmp(OP_GT, z, zero), d, zero)
    return p, [dx, dy, dz]
