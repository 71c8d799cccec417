"""CPU oracle: a per-operator fp64 evaluator of a serialized computational graph.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what a
fused subgraph must compute.  It is used by the tests, by the smoke check and by
the benchmark's CPU-baseline leg, and by nothing else; the CUDA library neither
imports it nor shares any code, table or parser with it.

What it computes.  A graph G = (V, E, tau, sigma) (Definition 3.1 of the paper)
defines a function f_G from its input tensors to its output tensors.  Fusing the
graph into one kernel must leave f_G unchanged up to a numerical tolerance
(Definition 3.2, Eq. 1).  The oracle therefore *is* the definition of f_G: it
walks the nodes in the order the descriptor lists them and, for every node,
evaluates the operator over the whole tensor and materialises the result before
the next node runs.  Nothing is fused, tiled or reordered.

Arithmetic.  Floating-point tensors are held as float64 whatever their declared
dtype; integer and boolean tensors as exact int64.  A node whose declared output
dtype is a 16-bit float (bf16, f16) hands its *consumers* the value rounded to
that dtype (nearest, ties to even), because a graph that declares a narrow
intermediate asks for that rounding.  A node declared f32 is not rounded (f32 is
the compute type of the fused kernels; the oracle is the exact reference for
it).  Graph outputs are returned unrounded in float64, so that a kernel's single
final rounding is judged against the exact value.

Operator definitions follow the usual closed forms; the LayerNorm form (biased
variance, 1/sqrt(var + eps), (x - mean) * rstd * gamma + beta) is the one the
paper's fused add+LayerNorm kernel computes (Appendix H, case 1); its
masked-mean-pooling pattern (Appendix H, case 2: cast, mul, two sums over the
sequence dimension, clamp, div, a one-operand cat) is evaluated operator by
operator with the reductions over a leading dimension below.

Every function is pinned by tests/test_oracle_pins.py against closed forms,
invariants, brute force on tiny inputs and a third restatement; nothing here is
"parity unpinned".
"""
from __future__ import annotations

import math
import struct
from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence

import numpy as np

# ---------------------------------------------------------------------------
# descriptor format (own parser; numbers as fixed by the format, version 1)
# ---------------------------------------------------------------------------
_MAGIC = 0x31474E50
_DT_F32, _DT_F16, _DT_BF16, _DT_I8, _DT_BOOL, _DT_I32, _DT_I64 = range(7)
_FLOAT_DT = (_DT_F32, _DT_F16, _DT_BF16)
_IMM_BASE = 0xFFFFFFFE  # 0xFFFFFFFF -> imm[0], 0xFFFFFFFE -> imm[1]

_OP_NAMES = {
    1: "neg", 2: "abs", 3: "exp", 4: "log", 5: "sqrt", 6: "rsqrt", 7: "recip", 8: "tanh",
    9: "sigmoid", 10: "silu", 11: "gelu_tanh", 12: "gelu_erf", 13: "relu", 14: "cast",
    15: "square", 16: "erf",
    32: "add", 33: "sub", 34: "mul", 35: "div", 36: "max", 37: "min",
    38: "gt", 39: "ge", 40: "lt", 41: "le", 42: "eq", 43: "ne",
    64: "where", 65: "clamp", 66: "fma",
    96: "sum", 97: "mean", 98: "var", 99: "amax", 100: "amin", 101: "argmax", 102: "argmin",
    103: "logsumexp", 104: "sum_dim", 105: "mean_dim", 106: "amax_dim", 107: "amin_dim",
    128: "softmax", 129: "log_softmax", 130: "layer_norm", 131: "rms_norm",
    160: "roll", 161: "slice", 162: "view", 163: "cat", 164: "contiguous",
}


@dataclass
class TensorInfo:
    dtype: int
    is_input: bool
    is_output: bool
    dims: tuple


@dataclass
class NodeInfo:
    op: str
    ins: list          # tensor ids, or ("imm", value)
    outs: list
    imm: tuple
    attr: tuple


@dataclass
class GraphInfo:
    tensors: List[TensorInfo]
    nodes: List[NodeInfo]

    @property
    def input_ids(self):
        return [i for i, t in enumerate(self.tensors) if t.is_input]

    @property
    def output_ids(self):
        return [i for i, t in enumerate(self.tensors) if t.is_output]


def parse(desc: bytes) -> GraphInfo:
    """Decode a descriptor.  Raises ValueError on a malformed one."""
    if len(desc) < 16:
        raise ValueError("descriptor shorter than its header")
    magic, version, _r, n_t, n_n = struct.unpack_from("<IHHII", desc, 0)
    if magic != _MAGIC or version != 1:
        raise ValueError("bad magic or version")
    if len(desc) != 16 + 40 * n_t + 64 * n_n:
        raise ValueError("descriptor length does not match its tables")
    tensors, nodes = [], []
    off = 16
    for _ in range(n_t):
        dt, role, rank, _p, _q, d0, d1, d2, d3 = struct.unpack_from("<BBBBI4q", desc, off)
        off += 40
        if dt > _DT_I64 or rank > 4:
            raise ValueError("bad tensor record")
        tensors.append(TensorInfo(dt, bool(role & 1), bool(role & 2), (d0, d1, d2, d3)[:rank]))
    for _ in range(n_n):
        rec = struct.unpack_from("<HBB4I3I2d2q", desc, off)
        off += 64
        opc, n_in, n_out = rec[0], rec[1], rec[2]
        if opc not in _OP_NAMES or n_in > 4 or n_out > 3 or n_out < 1:
            raise ValueError("bad node record")
        imm = (rec[10], rec[11])
        ins = []
        for s in rec[3:3 + n_in]:
            if s >= _IMM_BASE:
                ins.append(("imm", imm[0xFFFFFFFF - s]))
            else:
                if s >= n_t:
                    raise ValueError("operand id out of range")
                ins.append(s)
        outs = list(rec[7:7 + n_out])
        if any(o >= n_t for o in outs):
            raise ValueError("output id out of range")
        nodes.append(NodeInfo(_OP_NAMES[opc], ins, outs, imm, (rec[12], rec[13])))
    return GraphInfo(tensors, nodes)


# ---------------------------------------------------------------------------
# storage <-> float64
# ---------------------------------------------------------------------------
def widen(arr: np.ndarray, dtype: int) -> np.ndarray:
    """Stored values -> exact float64 (float dtypes) or int64 (integer dtypes)."""
    if dtype == _DT_F32:
        return np.asarray(arr, dtype=np.float32).astype(np.float64)
    if dtype == _DT_F16:
        return np.asarray(arr, dtype=np.float16).astype(np.float64)
    if dtype == _DT_BF16:
        bits = np.asarray(arr, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
        return bits.view(np.float32).astype(np.float64)
    if dtype == _DT_BOOL:
        return (np.asarray(arr) != 0).astype(np.int64)
    return np.asarray(arr).astype(np.int64)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """float64 -> nearest bfloat16 value (ties to even), returned as float64.

    bf16 has an 8-bit exponent (bias 127) and 8 significant bits.  For a value
    with binary exponent e (clamped below at the subnormal exponent -126) the
    spacing of representable numbers is 2**(e-7); dividing by it is exact, and
    rint rounds half to even.
    """
    x = np.asarray(x, dtype=np.float64)
    out = x.copy()
    fin = np.isfinite(x) & (x != 0)
    if fin.any():
        v = x[fin]
        _, e = np.frexp(v)                    # v = m * 2**e with 0.5 <= |m| < 1
        e = np.maximum(e - 1, -126)           # exponent of the leading bit
        q = np.ldexp(1.0, e - 7)
        r = np.rint(v / q) * q
        r = np.where(np.abs(r) >= 2.0 ** 128, np.sign(r) * np.inf, r)
        out[fin] = r
    return out


def round_to_f16(x: np.ndarray) -> np.ndarray:
    with np.errstate(over="ignore"):
        return np.asarray(x, dtype=np.float64).astype(np.float16).astype(np.float64)


# ---------------------------------------------------------------------------
# operators (each loops over the whole tensor via one NumPy expression)
# ---------------------------------------------------------------------------
_SQRT_2_OVER_PI = math.sqrt(2.0 / math.pi)


def _f(x):
    return np.asarray(x, dtype=np.float64)


try:  # a vectorised libm-quality erf when SciPy is present
    from scipy.special import erf as _vec_erf
except Exception:  # pragma: no cover
    _vec_erf = np.vectorize(math.erf, otypes=[np.float64])


def _erf(x):
    return _vec_erf(_f(x))


def op_sigmoid(x):
    """sigmoid(x) = 1 / (1 + e^-x)."""
    return 1.0 / (1.0 + np.exp(-_f(x)))


def op_silu(x):
    """silu(x) = x * sigmoid(x)."""
    return _f(x) * op_sigmoid(x)


def op_gelu_tanh(x):
    """gelu_tanh(x) = 0.5 x (1 + tanh( sqrt(2/pi) (x + 0.044715 x^3) ))."""
    x = _f(x)
    return 0.5 * x * (1.0 + np.tanh(_SQRT_2_OVER_PI * (x + 0.044715 * x * x * x)))


def op_gelu_erf(x):
    """gelu_erf(x) = 0.5 x (1 + erf(x / sqrt 2))."""
    x = _f(x)
    return 0.5 * x * (1.0 + _erf(x / math.sqrt(2.0)))


_UNARY = {
    "neg": lambda x: -x,
    "abs": lambda x: np.abs(x),
    "exp": lambda x: np.exp(_f(x)),
    "log": lambda x: np.log(_f(x)),
    "sqrt": lambda x: np.sqrt(_f(x)),
    "rsqrt": lambda x: 1.0 / np.sqrt(_f(x)),
    "recip": lambda x: 1.0 / _f(x),
    "tanh": lambda x: np.tanh(_f(x)),
    "sigmoid": op_sigmoid,
    "silu": op_silu,
    "gelu_tanh": op_gelu_tanh,
    "gelu_erf": op_gelu_erf,
    "relu": lambda x: np.maximum(x, 0),          # NaN stays NaN
    "square": lambda x: x * x,
    "erf": lambda x: _erf(_f(x)),
}

_BINARY = {
    "add": lambda a, b: a + b,
    "sub": lambda a, b: a - b,
    "mul": lambda a, b: a * b,
    "div": lambda a, b: _f(a) / _f(b),
    # max/min propagate NaN, as the elementwise maximum/minimum of array libraries do
    "max": lambda a, b: np.maximum(a, b),
    "min": lambda a, b: np.minimum(a, b),
}

_COMPARE = {
    "gt": lambda a, b: a > b, "ge": lambda a, b: a >= b, "lt": lambda a, b: a < b,
    "le": lambda a, b: a <= b, "eq": lambda a, b: a == b, "ne": lambda a, b: a != b,
}


def red_sum(x):
    return _f(x).sum(axis=-1)


def red_mean(x):
    """mean = sum(x) / N."""
    x = _f(x)
    return x.sum(axis=-1) / x.shape[-1]


def red_var(x, correction: int):
    """Two-pass variance: sum((x - mean)^2) / (N - correction)."""
    x = _f(x)
    n = x.shape[-1]
    mean = x.sum(axis=-1, keepdims=True) / n
    d = x - mean
    return (d * d).sum(axis=-1) / (n - correction)


def red_amax(x):
    """Row maximum; a NaN anywhere in the row makes the result NaN."""
    return np.max(x, axis=-1)


def red_amin(x):
    return np.min(x, axis=-1)


def _arg_extreme(x, want_max: bool):
    """Smallest index attaining the row extreme; NaN counts as the extreme and the
    first NaN wins (the convention of the common array libraries)."""
    x = np.asarray(x)
    rows = x.reshape(-1, x.shape[-1])
    out = np.empty(rows.shape[0], dtype=np.int64)
    for i, row in enumerate(rows):
        nan = np.isnan(row) if row.dtype.kind == "f" else np.zeros(row.shape, bool)
        if nan.any():
            out[i] = int(np.flatnonzero(nan)[0])
        else:
            ext = row.max() if want_max else row.min()
            out[i] = int(np.flatnonzero(row == ext)[0])
    return out.reshape(x.shape[:-1])


def red_argmax(x):
    return _arg_extreme(x, True)


def red_argmin(x):
    return _arg_extreme(x, False)


def red_logsumexp(x):
    """logsumexp(x) = m + log(sum_k e^(x_k - m)), m the row maximum;
    m = -inf gives -inf and m = +inf gives +inf."""
    x = _f(x)
    m = np.max(x, axis=-1, keepdims=True)
    with np.errstate(invalid="ignore", divide="ignore", over="ignore"):
        shift = np.where(np.isfinite(m), m, 0.0)
        s = np.exp(x - shift).sum(axis=-1, keepdims=True)
        out = np.where(np.isfinite(m), shift + np.log(s), m)
        out = np.where(np.isnan(x).any(axis=-1, keepdims=True), np.nan, out)
    return out[..., 0]


def red_over_dim(kind: str, x, dim: int):
    """Reduction over one dimension `dim` of x, that dimension dropped from the result:
    sum_k x[.., k, ..]; mean = that sum / D; amax / amin = the extreme (a NaN along the
    dimension makes the result NaN).  This is what the paper's masked-mean-pooling pattern
    uses twice (Appendix H, case 2: sum(hidden * mask, 1) and sum(mask, 1) over the sequence
    dimension of [B, S, D] tensors)."""
    x = _f(x)
    if not 0 <= dim < x.ndim:
        raise ValueError("reduced dimension outside the tensor")
    if kind == "sum_dim":
        return x.sum(axis=dim)
    if kind == "mean_dim":
        return x.sum(axis=dim) / x.shape[dim]
    if kind == "amax_dim":
        return np.max(x, axis=dim)
    if kind == "amin_dim":
        return np.min(x, axis=dim)
    raise ValueError(kind)


def op_cat(parts, dim: int):
    """Concatenation of the operands along `dim` (one operand: the operand itself)."""
    return np.concatenate([np.asarray(p) for p in parts], axis=dim)


def comp_softmax(x):
    """softmax(x)_j = e^(x_j - m) / sum_k e^(x_k - m), m the row maximum.
    A row that is -inf throughout yields NaN (inf - inf), as IEEE arithmetic does."""
    x = _f(x)
    with np.errstate(invalid="ignore", over="ignore"):
        m = np.max(x, axis=-1, keepdims=True)
        e = np.exp(x - m)
        return e / e.sum(axis=-1, keepdims=True)


def comp_log_softmax(x):
    """log_softmax(x)_j = x_j - logsumexp(x)."""
    x = _f(x)
    with np.errstate(invalid="ignore"):
        return x - red_logsumexp(x)[..., None]


def comp_layer_norm(x, gamma, beta, eps: float):
    """mean = sum(x)/N; var = sum((x-mean)^2)/N (biased); rstd = 1/sqrt(var + eps);
    y = (x - mean) * rstd * gamma + beta.  Returns (y, mean, rstd)."""
    x = _f(x)
    n = x.shape[-1]
    mean = x.sum(axis=-1, keepdims=True) / n
    d = x - mean
    var = (d * d).sum(axis=-1, keepdims=True) / n
    rstd = 1.0 / np.sqrt(var + eps)
    y = d * rstd
    if gamma is not None:
        y = y * _f(gamma)
    if beta is not None:
        y = y + _f(beta)
    return y, mean[..., 0], rstd[..., 0]


def comp_rms_norm(x, gamma, eps: float):
    """y = x / sqrt(mean(x^2) + eps) * gamma."""
    x = _f(x)
    ms = (x * x).sum(axis=-1, keepdims=True) / x.shape[-1]
    y = x * (1.0 / np.sqrt(ms + eps))
    if gamma is not None:
        y = y * _f(gamma)
    return y


def op_roll(x, dim: int, shift: int):
    """y[..., i, ...] = x[..., (i - shift) mod D, ...] along `dim`: the circular shift that the
    paper's fused kernel replaces by index arithmetic, idx = (S + i - shift) mod S (Section 4.4)."""
    x = np.asarray(x)
    d = x.shape[dim]
    idx = (np.arange(d) - shift) % d
    return np.take(x, idx, axis=dim)


def op_slice(x, dim: int, start: int, length: int):
    """y[..., i, ...] = x[..., start + i, ...] for i < length along `dim`."""
    x = np.asarray(x)
    if start < 0 or start + length > x.shape[dim]:
        raise ValueError("slice outside the tensor")
    sl = [slice(None)] * x.ndim
    sl[dim] = slice(start, start + length)
    return x[tuple(sl)]


def op_view(x, dims):
    """Same elements in the same row-major order under another shape."""
    return np.ascontiguousarray(x).reshape(dims)


def op_contiguous(x):
    """The same values, laid out densely in row-major order: as every tensor of a descriptor is
    dense already, the identity on values (the paper's first case study keeps such a node after its
    rolls and slices, Section 4.4)."""
    return np.ascontiguousarray(x)


def op_cast(x, dst_dtype: int):
    """Value conversion.  Float -> integer truncates toward zero; anything -> bool
    tests for non-zero; to a float type the value is kept (narrow-float rounding is
    applied by the caller when consumers read the tensor)."""
    x = np.asarray(x)
    if dst_dtype in _FLOAT_DT:
        return x.astype(np.float64)
    if dst_dtype == _DT_BOOL:
        return (x != 0).astype(np.int64)
    if x.dtype.kind == "f":
        return np.trunc(x).astype(np.int64)
    return x.astype(np.int64)


# ---------------------------------------------------------------------------
# the evaluator
# ---------------------------------------------------------------------------
def _consumer_view(val: np.ndarray, dtype: int) -> np.ndarray:
    if dtype == _DT_BF16:
        return round_to_bf16(val)
    if dtype == _DT_F16:
        return round_to_f16(val)
    return val


def evaluate(desc: bytes, inputs: Sequence[np.ndarray],
             keep_intermediates: Optional[Dict[int, np.ndarray]] = None) -> List[np.ndarray]:
    """Evaluate f_G (Definition 3.1) node by node.

    ``inputs`` are the stored arrays in descriptor input order (bf16 as uint16
    bit patterns).  Returns the graph outputs in descriptor output order: float64
    arrays for float outputs (unrounded), int64 arrays for integer / boolean
    outputs, each shaped as its tensor record says.  If ``keep_intermediates`` is
    a dict, every tensor's value is also left there by id.
    """
    g = parse(desc)
    if len(inputs) != len(g.input_ids):
        raise ValueError("wrong number of inputs")
    exact: Dict[int, np.ndarray] = {}     # value as computed
    seen: Dict[int, np.ndarray] = {}      # value as consumers read it
    last_use: Dict[int, int] = {}
    for ni, n in enumerate(g.nodes):
        for s in n.ins:
            if not isinstance(s, tuple):
                last_use[s] = ni
    for tid, arr in zip(g.input_ids, inputs):
        t = g.tensors[tid]
        if tuple(np.shape(arr)) != tuple(t.dims):
            raise ValueError(f"input {tid}: shape {np.shape(arr)} != {t.dims}")
        exact[tid] = seen[tid] = widen(arr, t.dtype)

    def operand(s):
        if isinstance(s, tuple):
            return np.float64(s[1])
        if s not in seen:
            raise ValueError(f"tensor {s} read before it is produced")
        return seen[s]

    for ni, n in enumerate(g.nodes):
        a = [operand(s) for s in n.ins]
        out_t = [g.tensors[o] for o in n.outs]
        with np.errstate(all="ignore"):
            if n.op in _UNARY:
                res = [_UNARY[n.op](a[0])]
            elif n.op == "cast":
                res = [op_cast(a[0], out_t[0].dtype)]
            elif n.op in _BINARY:
                res = [_BINARY[n.op](a[0], a[1])]
            elif n.op in _COMPARE:
                res = [_COMPARE[n.op](a[0], a[1]).astype(np.int64)]
            elif n.op == "where":
                res = [np.where(np.asarray(a[0]) != 0, a[1], a[2])]
            elif n.op == "clamp":
                res = [np.minimum(np.maximum(a[0], a[1]), a[2])]
            elif n.op == "fma":
                res = [a[0] * a[1] + a[2]]
            elif n.op == "roll":      # (dim, shift) in attr; optionally a second dimension as imm = (1 + dim, shift)
                res = [op_roll(a[0], int(n.attr[0]), int(n.attr[1]))]
                if n.imm[0] != 0:
                    res = [op_roll(res[0], int(n.imm[0]) - 1, int(n.imm[1]))]
            elif n.op == "slice":     # (dim, start) in attr, the length from the output shape; optionally a second dimension in imm
                res = [op_slice(a[0], int(n.attr[0]), int(n.attr[1]), int(out_t[0].dims[int(n.attr[0])]))]
                if n.imm[0] != 0:
                    res = [op_slice(res[0], int(n.imm[0]) - 1, int(n.imm[1]), int(out_t[0].dims[int(n.imm[0]) - 1]))]
            elif n.op == "view":
                res = [op_view(a[0], tuple(out_t[0].dims))]
            elif n.op in ("sum_dim", "mean_dim", "amax_dim", "amin_dim"):
                res = [red_over_dim(n.op, a[0], int(n.attr[0]))]
            elif n.op == "cat":
                res = [op_cat(a, int(n.attr[0]))]
            elif n.op == "contiguous":
                res = [op_contiguous(a[0])]
            elif n.op == "sum":
                res = [red_sum(a[0])]
            elif n.op == "mean":
                res = [red_mean(a[0])]
            elif n.op == "var":
                res = [red_var(a[0], int(n.attr[0]))]
            elif n.op == "amax":
                res = [red_amax(a[0])]
            elif n.op == "amin":
                res = [red_amin(a[0])]
            elif n.op == "argmax":
                res = [red_argmax(a[0])]
            elif n.op == "argmin":
                res = [red_argmin(a[0])]
            elif n.op == "logsumexp":
                res = [red_logsumexp(a[0])]
            elif n.op == "softmax":
                res = [comp_softmax(a[0])]
            elif n.op == "log_softmax":
                res = [comp_log_softmax(a[0])]
            elif n.op == "layer_norm":
                gamma = a[1] if len(a) > 1 else None
                beta = a[2] if len(a) > 2 else None
                res = list(comp_layer_norm(a[0], gamma, beta, float(n.imm[0])))[:len(n.outs)]
            elif n.op == "rms_norm":
                res = [comp_rms_norm(a[0], a[1] if len(a) > 1 else None, float(n.imm[0]))]
            else:  # pragma: no cover
                raise ValueError(n.op)
        for o, t, r in zip(n.outs, out_t, res):
            r = np.asarray(r)
            if t.dtype in _FLOAT_DT:
                r = r.astype(np.float64)
            else:
                r = op_cast(r, t.dtype) if r.dtype.kind == "f" else r.astype(np.int64)
            want = tuple(t.dims)
            if r.shape != want:
                if int(np.prod(r.shape, dtype=np.int64)) == int(np.prod(want, dtype=np.int64)) \
                        and tuple(d for d in r.shape if d != 1) == tuple(d for d in want if d != 1):
                    r = r.reshape(want)       # kept vs dropped size-1 dims only
                else:
                    r = np.broadcast_to(r, want).copy() if _broadcastable(r.shape, want) else _bad(o, r.shape, want)
            exact[o] = r
            seen[o] = _consumer_view(r, t.dtype)
        # free what nobody reads any more (every intermediate was still materialised)
        if keep_intermediates is None:
            for s in list(seen):
                t = g.tensors[s]
                if last_use.get(s, -1) <= ni and not t.is_output and s in seen:
                    del seen[s]
                    exact.pop(s, None)
    if keep_intermediates is not None:
        keep_intermediates.update(exact)
    missing = [o for o in g.output_ids if o not in exact]
    if missing:
        raise ValueError(f"outputs never produced: {missing}")
    return [exact[o] for o in g.output_ids]


def _broadcastable(src, dst) -> bool:
    try:
        return np.broadcast_shapes(src, dst) == tuple(dst)
    except ValueError:
        return False


def _bad(o, got, want):
    raise ValueError(f"tensor {o}: computed shape {got} does not fit declared {want}")


# ---------------------------------------------------------------------------
# the validity rule (Eq. 1 read in allclose form with the per-dtype tolerances)
# ---------------------------------------------------------------------------
TOLERANCES = {
    _DT_F32: (1e-5, 1e-6),      # rtol, atol for fp32 outputs
    _DT_BF16: (1.6e-2, 1e-3),   # bf16 outputs, fp32 accumulation
    _DT_F16: (1e-3, 1e-5),      # the paper's t = -5 row for float16
}


# smallest magnitude that rounds to infinity (largest finite value plus half a unit in the last place)
_OVERFLOW_AT = {
    _DT_F32: (2.0 - 2.0 ** -24) * 2.0 ** 127,
    _DT_BF16: (2.0 - 2.0 ** -8) * 2.0 ** 127,
    _DT_F16: 65520.0,
}


def compare(got: np.ndarray, ref: np.ndarray, dtype: int) -> dict:
    """err(f_G(x), f_pi(G)(x)) <= t, elementwise: |got - ref| <= atol + rtol*|ref| for
    float outputs; infinities must agree exactly and NaN must sit where NaN sits;
    integer and boolean outputs must be identical (tolerance 0)."""
    got = np.asarray(got)
    ref = np.asarray(ref)
    if got.shape != ref.shape:
        return {"ok": False, "violations": -1, "reason": f"shape {got.shape} vs {ref.shape}"}
    if dtype not in _FLOAT_DT:
        bad = int((got.astype(np.int64) != ref.astype(np.int64)).sum())
        return {"ok": bad == 0, "violations": bad, "max_abs": float(bad != 0), "max_rel": 0.0}
    rtol, atol = TOLERANCES[dtype]
    g = got.astype(np.float64)
    r = ref.astype(np.float64)
    # The reference is unrounded; the output is stored in `dtype`.  A value at or beyond the
    # point where round-to-nearest overflows that type is, correctly stored, an infinity.
    lim = _OVERFLOW_AT[dtype]
    with np.errstate(invalid="ignore"):
        r = np.where(np.abs(r) >= lim, np.sign(r) * np.inf, r)
    fin = np.isfinite(r)
    with np.errstate(invalid="ignore"):
        bad_special = (~fin) & ~((np.isnan(r) & np.isnan(g)) | (g == r))
        diff = np.abs(np.where(fin, g - r, 0.0))
        bad_fin = fin & ~(diff <= atol + rtol * np.abs(np.where(fin, r, 0.0)))
    diff_f = diff[fin]
    max_abs = float(np.nanmax(diff_f)) if diff_f.size else 0.0
    with np.errstate(divide="ignore", invalid="ignore"):
        rel = diff_f / np.abs(r[fin])
        rel = rel[np.isfinite(rel)]
    bad = int(bad_special.sum() + bad_fin.sum())
    return {"ok": bad == 0, "violations": bad, "max_abs": max_abs,
            "max_rel": float(rel.max()) if rel.size else 0.0}
