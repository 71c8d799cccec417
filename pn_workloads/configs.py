"""Seeded synthetic workloads: the five benchmark subgraphs and their inputs.

Each ``cN(...)`` function returns a :class:`Workload`: the serialized graph,
the input arrays, and bookkeeping (names, shapes, dtypes, compulsory bytes).
The default arguments are the full benchmark sizes; smaller sizes of the same
graph serve the parity tests.

The shapes follow the long-tail fusible subgraphs the paper describes (2-35
operators, pointwise + last-dim reduction + normalisation, fp32 / bf16,
Section 3.3); the inputs are synthetic and stand in for the paper's benchmark
suite, none of whose items are reproduced here.

Storage conventions for host arrays: f32 -> float32, f16 -> float16,
bf16 -> uint16 bit patterns, i8 -> int8, bool -> uint8, i32/i64 -> int32/int64.

Nothing in this module evaluates an operator of the graph: it draws random
numbers, rounds them to their storage type and writes descriptors.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Tuple

import numpy as np

from . import descriptor as D
from .descriptor import GraphBuilder, Imm

NP_STORAGE = {D.F32: np.float32, D.F16: np.float16, D.BF16: np.uint16, D.I8: np.int8,
              D.BOOL: np.uint8, D.I32: np.int32, D.I64: np.int64}


@dataclass
class Workload:
    name: str
    desc: bytes
    inputs: List[np.ndarray]
    input_names: List[str]
    input_meta: List[Tuple[int, tuple]]    # (dtype code, dims)
    output_names: List[str]
    output_meta: List[Tuple[int, tuple]]
    n_nodes: int
    notes: Dict[str, object] = field(default_factory=dict)

    @property
    def compulsory_bytes(self) -> int:
        """Every graph input read once plus every graph output written once."""
        tot = 0
        for dt, dims in self.input_meta + self.output_meta:
            tot += D.DTYPE_BYTES[dt] * int(np.prod(dims, dtype=np.int64)) if dims else D.DTYPE_BYTES[dt]
        return tot


# ---------------------------------------------------------------------------
# storage rounding helpers (data preparation only)
# ---------------------------------------------------------------------------
def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float values to bfloat16 (nearest, ties to even); returns uint16 bits.
    Finite inputs only."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (b + (np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1)))) >> np.uint32(16)
    return r.astype(np.uint16)


def _rng(seed: int, cfg: int, tensor: int) -> np.random.Generator:
    return np.random.default_rng([seed, cfg, tensor])


def _draw(rng, kind: str, shape, a: float, b: float, chunk: int = 1 << 24) -> np.ndarray:
    """Draw float64 values in bounded chunks and hand them back as float32.
    kind 'normal': mean a, std b; kind 'uniform': on [a, b)."""
    n = int(np.prod(shape, dtype=np.int64))
    out = np.empty(n, dtype=np.float32)
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        if kind == "normal":
            v = rng.standard_normal(hi - lo) * b + a
        else:
            v = rng.random(hi - lo) * (b - a) + a
        out[lo:hi] = v
    return out.reshape(shape)


def _store(x32: np.ndarray, dtype: int) -> np.ndarray:
    if dtype == D.F32:
        return x32
    if dtype == D.BF16:
        return to_bf16_bits(x32)
    if dtype == D.F16:
        return x32.astype(np.float16)
    raise ValueError(dtype)


def _finish(name, g: GraphBuilder, in_names, out_names, inputs, notes=None) -> Workload:
    ins = g.input_ids()
    outs = g.output_ids()
    assert len(ins) == len(inputs) == len(in_names) and len(outs) == len(out_names)
    for tid, arr in zip(ins, inputs):
        dt, dims = g.tensor_meta(tid)
        assert tuple(arr.shape) == tuple(dims) and arr.dtype == NP_STORAGE[dt], (name, tid)
    return Workload(name, g.build(), [np.ascontiguousarray(a) for a in inputs], list(in_names),
                    [g.tensor_meta(t) for t in ins], list(out_names),
                    [g.tensor_meta(t) for t in outs], len(g._nodes), notes or {})


# ---------------------------------------------------------------------------
# C1: pointwise chain  y = gelu_tanh(x*w + b) + r
# ---------------------------------------------------------------------------
def c1(M: int = 1024, N: int = 1024, seed: int = 0, dtype: int = D.F32) -> Workload:
    g = GraphBuilder()
    x = g.input(dtype, (M, N))
    w = g.input(dtype, (N,))
    b = g.input(dtype, (N,))
    r = g.input(dtype, (M, N))
    if dtype == D.F32:
        t0 = g.op("mul", [x, w], D.F32, (M, N))
        t1 = g.op("add", [t0, b], D.F32, (M, N))
        t2 = g.op("gelu_tanh", [t1], D.F32, (M, N))
        y = g.op("add", [t2, r], D.F32, (M, N))
    else:  # 16-bit storage, fp32 math, one rounding at the end
        xf, wf, bf, rf = (g.op("cast", [t], D.F32, dm) for t, dm in
                          ((x, (M, N)), (w, (N,)), (b, (N,)), (r, (M, N))))
        t0 = g.op("mul", [xf, wf], D.F32, (M, N))
        t1 = g.op("add", [t0, bf], D.F32, (M, N))
        t2 = g.op("gelu_tanh", [t1], D.F32, (M, N))
        t3 = g.op("add", [t2, rf], D.F32, (M, N))
        y = g.op("cast", [t3], dtype, (M, N))
    g.mark_output(y)
    xs = _store(_draw(_rng(seed, 1, 0), "normal", (M, N), 0.0, 1.0), dtype)
    ws = _store(_draw(_rng(seed, 1, 1), "uniform", (N,), -1.0, 1.0), dtype)
    bs = _store(_draw(_rng(seed, 1, 2), "uniform", (N,), -1.0, 1.0), dtype)
    rs = _store(_draw(_rng(seed, 1, 3), "normal", (M, N), 0.0, 1.0), dtype)
    return _finish("c1_pointwise_chain", g, ["x", "w", "b", "r"], ["y"], [xs, ws, bs, rs])


# ---------------------------------------------------------------------------
# C2: masked scaled softmax, bf16 in/out with fp32 math
# ---------------------------------------------------------------------------
def c2(B: int = 512, Q: int = 512, K: int = 512, seed: int = 0, dtype: int = D.BF16,
       head_dim: int = 64) -> Workload:
    g = GraphBuilder()
    s = g.input(dtype, (B, Q, K))
    m = g.input(D.I8, (Q, K))
    t0 = g.op("cast", [s], D.F32, (B, Q, K)) if dtype != D.F32 else s
    t1 = g.op("mul", [t0, Imm(1.0 / math.sqrt(head_dim))], D.F32, (B, Q, K))
    t2 = g.op("where", [m, t1, Imm(-math.inf)], D.F32, (B, Q, K))
    t3 = g.op("softmax", [t2], D.F32, (B, Q, K))
    y = g.op("cast", [t3], dtype, (B, Q, K)) if dtype != D.F32 else t3
    g.mark_output(y)
    scores = _store(_draw(_rng(seed, 2, 0), "normal", (B, Q, K), 0.0, math.sqrt(2.0)), dtype)
    mask = np.tril(np.ones((Q, K), dtype=np.int8))  # mask[q, k] = 1 iff k <= q
    return _finish("c2_masked_scaled_softmax", g, ["scores", "mask"], ["y"], [scores, mask])


# ---------------------------------------------------------------------------
# C3: residual + LayerNorm + cast; outputs y, mean, rstd
# ---------------------------------------------------------------------------
def c3(M: int = 16384, N: int = 4096, seed: int = 0, dtype: int = D.BF16, eps: float = 1e-5,
       also_output_sum: bool = False) -> Workload:
    g = GraphBuilder()
    x = g.input(dtype, (M, N))
    res = g.input(dtype, (M, N))
    gamma = g.input(D.F32, (N,))
    beta = g.input(D.F32, (N,))
    t0 = g.op("cast", [x], D.F32, (M, N)) if dtype != D.F32 else x
    t1 = g.op("cast", [res], D.F32, (M, N)) if dtype != D.F32 else res
    h = g.op("add", [t0, t1], D.F32, (M, N))
    n, mean, rstd = g.node("layer_norm", [h, gamma, beta], [D.F32, D.F32, D.F32],
                           [(M, N), (M,), (M,)], extra_imm=[eps])
    y = g.op("cast", [n], dtype, (M, N)) if dtype != D.F32 else n
    names = {y: "y", mean: "mean", rstd: "rstd"}
    if also_output_sum:  # the paper's fused add+LayerNorm kernel also returns the sum
        hb = g.op("cast", [h], dtype, (M, N)) if dtype != D.F32 else h
        names[hb] = "h"
    for t in names:
        g.mark_output(t)
    out_names = [names[i] for i in g.output_ids()]   # table order decides output order
    xs = _store(_draw(_rng(seed, 3, 0), "normal", (M, N), 0.0, 1.0), dtype)
    rs = _store(_draw(_rng(seed, 3, 1), "normal", (M, N), 0.0, 1.0), dtype)
    ga = _draw(_rng(seed, 3, 2), "uniform", (N,), 0.5, 1.5)
    be = _draw(_rng(seed, 3, 3), "normal", (N,), 0.0, 0.1)
    return _finish("c3_residual_layernorm", g, ["x", "residual", "gamma", "beta"], out_names,
                   [xs, rs, ga, be], {"eps": eps})


# ---------------------------------------------------------------------------
# C4: long-row reduction: logsumexp (f32) and argmax (i64)
# ---------------------------------------------------------------------------
def c4(M: int = 64, N: int = 262144, seed: int = 0, spike_p: float = 0.01,
       spike: float = 30.0, dtype: int = D.F32) -> Workload:
    g = GraphBuilder()
    x = g.input(dtype, (M, N))
    xf = g.op("cast", [x], D.F32, (M, N)) if dtype != D.F32 else x
    lse = g.op("logsumexp", [xf], D.F32, (M,))
    idx = g.op("argmax", [xf], D.I64, (M,))
    g.mark_output(lse); g.mark_output(idx)
    rng = _rng(seed, 4, 0)
    xs = _draw(rng, "normal", (M, N), 0.0, 2.0)          # variance 4
    hit = _draw(rng, "uniform", (M, N), 0.0, 1.0) < spike_p
    xs[hit] = np.float32(spike)
    per_row = hit.sum(axis=1)
    xs = _store(xs, dtype)
    return _finish("c4_long_row_reduction", g, ["x"], ["logsumexp", "argmax"], [xs],
                   {"spikes_per_row_min": int(per_row.min()), "spike": spike})


# ---------------------------------------------------------------------------
# C5: multi-output gated DAG
# ---------------------------------------------------------------------------
def c5(M: int = 8192, N: int = 14336, seed: int = 0, dtype: int = D.BF16) -> Workload:
    g = GraphBuilder()
    a = g.input(dtype, (M, N))
    gt = g.input(dtype, (M, N))
    col = g.input(dtype, (1, N))
    row = g.input(dtype, (M, 1))
    cast = (lambda t, dm: g.op("cast", [t], D.F32, dm)) if dtype != D.F32 else (lambda t, dm: t)
    t0 = cast(a, (M, N))
    t1 = cast(gt, (M, N))
    t2 = g.op("sigmoid", [t1], D.F32, (M, N))
    t3 = g.op("mul", [t0, t2], D.F32, (M, N))
    t4 = g.op("mul", [t3, cast(col, (1, N))], D.F32, (M, N))
    h = g.op("mul", [t4, cast(row, (M, 1))], D.F32, (M, N))
    hb = g.op("cast", [h], dtype, (M, N)) if dtype != D.F32 else h
    pos = g.op("gt", [h, Imm(0.0)], D.BOOL, (M, N))
    msk = g.op("cast", [pos], D.I8, (M, N))
    mean = g.op("mean", [h], D.F32, (M,))
    var = g.op("var", [h], D.F32, (M,), attr=[0, 0])       # population variance
    for t in (hb, msk, mean, var):
        g.mark_output(t)
    av = _store(_draw(_rng(seed, 5, 0), "normal", (M, N), 0.0, 1.0), dtype)
    gv = _store(_draw(_rng(seed, 5, 1), "normal", (M, N), 0.0, 1.0), dtype)
    cv = _store(_draw(_rng(seed, 5, 2), "uniform", (1, N), 0.9, 1.1), dtype)
    rv = _store(_draw(_rng(seed, 5, 3), "uniform", (M, 1), 0.5, 2.0), dtype)
    return _finish("c5_gated_multi_output", g, ["a", "g", "col_scale", "row_scale"],
                   ["h", "mask", "mean", "var"], [av, gv, cv, rv])


# ---------------------------------------------------------------------------
# N1: roll + slice + add + LayerNorm with two outputs (the operator sequence of the paper's
# first case study: contiguous, view, roll, slice, contiguous, view, add, layer_norm)
# ---------------------------------------------------------------------------
def n1(S: int = 133, SC: int = 128, Cc: int = 96, shift: int = 3, seed: int = 0, dtype: int = D.BF16,
       eps: float = 1e-5) -> Workload:
    g = GraphBuilder()
    x = g.input(dtype, (1, S * S, Cc))           # the window-partitioned feature map, flat
    res = g.input(dtype, (1, SC * SC, Cc))
    gamma = g.input(dtype, (Cc,))
    beta = g.input(dtype, (Cc,))
    # the eight operators of the case study: contiguous, view, roll (both window axes at once), slice
    # (both), contiguous, view, add, layer_norm
    c0 = g.op("contiguous", [x], dtype, (1, S * S, Cc))
    v = g.op("view", [c0], dtype, (S, S, Cc))
    r = g.op("roll", [v], dtype, (S, S, Cc), attr=[0, shift], extra_imm=[1 + 1, shift])
    sl = g.op("slice", [r], dtype, (SC, SC, Cc), attr=[0, 0], extra_imm=[1 + 1, 0])
    c1 = g.op("contiguous", [sl], dtype, (SC, SC, Cc))
    w = g.op("view", [c1], dtype, (1, SC * SC, Cc))
    cast = (lambda t, dm: g.op("cast", [t], D.F32, dm)) if dtype != D.F32 else (lambda t, dm: t)
    h = g.op("add", [cast(res, (1, SC * SC, Cc)), cast(w, (1, SC * SC, Cc))], D.F32, (1, SC * SC, Cc))
    y = g.node("layer_norm", [h, cast(gamma, (Cc,)), cast(beta, (Cc,))], [D.F32], [(1, SC * SC, Cc)], extra_imm=[eps])[0]
    out_add = g.op("cast", [h], dtype, (1, SC * SC, Cc)) if dtype != D.F32 else h
    out_ln = g.op("cast", [y], dtype, (1, SC * SC, Cc)) if dtype != D.F32 else y
    names = {out_add: "add", out_ln: "layer_norm"}
    for t in names:
        g.mark_output(t)
    xs = _store(_draw(_rng(seed, 6, 0), "normal", (1, S * S, Cc), 0.0, 1.0), dtype)
    rs = _store(_draw(_rng(seed, 6, 1), "normal", (1, SC * SC, Cc), 0.0, 1.0), dtype)
    ga = _store(_draw(_rng(seed, 6, 2), "uniform", (Cc,), 0.5, 1.5), dtype)
    be = _store(_draw(_rng(seed, 6, 3), "normal", (Cc,), 0.0, 0.1), dtype)
    return _finish("n1_roll_slice_add_layernorm", g, ["x", "residual", "gamma", "beta"],
                   [names[i] for i in g.output_ids()], [xs, rs, ga, be],
                   {"eps": eps, "shift": shift,
                    # only the SC x SC window of x is ever read
                    "touched_bytes": D.DTYPE_BYTES[dtype] * (4 * SC * SC * Cc + 2 * Cc)})


# ---------------------------------------------------------------------------
# N2: masked mean pooling (the operator sequence of the paper's second case study: cast, mul,
# sum, sum, clamp, div, cat): both sums run over the sequence dimension S of [B, S, D]
# ---------------------------------------------------------------------------
def n2(B: int = 256, S: int = 512, Dh: int = 1024, seed: int = 0, dtype: int = D.BF16,
       mask_dtype: int = D.I64, dense_mask: bool = False, floor: float = 1e-9) -> Workload:
    g = GraphBuilder()
    mshape = (B, S, Dh) if dense_mask else (B, S, 1)     # an expanded mask is a stride-0 view
    cshape = (B, Dh) if dense_mask else (B, 1)
    mask = g.input(mask_dtype, mshape)
    hidden = g.input(dtype, (B, S, Dh))
    m = g.op("cast", [mask], D.F32, mshape)
    prod = g.op("mul", [hidden, m], D.F32, (B, S, Dh))
    num = g.op("sum_dim", [prod], D.F32, (B, Dh), attr=[1, 0])
    cnt = g.op("sum_dim", [m], D.F32, cshape, attr=[1, 0])
    den = g.op("clamp", [cnt, Imm(floor), Imm(math.inf)], D.F32, cshape)
    q = g.op("div", [num, den], D.F32, (B, Dh))
    out = g.op("cat", [q], D.F32, (B, Dh), attr=[1, 0])
    g.mark_output(out)
    hs = _store(_draw(_rng(seed, 7, 0), "normal", (B, S, Dh), 0.0, 1.0), dtype)
    # a padded batch: sequence b keeps its first L_b positions, L_b uniform on [S/4, S]
    lens = _rng(seed, 7, 1).integers(max(1, S // 4), S + 1, size=B)
    keep = (np.arange(S)[None, :] < lens[:, None])
    mv = np.broadcast_to(keep[:, :, None], mshape)
    if mask_dtype in (D.F32, D.BF16, D.F16):
        ms = _store(np.ascontiguousarray(mv, dtype=np.float32), mask_dtype)
    else:
        ms = np.ascontiguousarray(mv).astype(NP_STORAGE[mask_dtype])
    return _finish("n2_masked_mean_pooling", g, ["mask", "hidden"], ["pooled"], [ms, hs],
                   {"floor": floor, "lengths_min": int(lens.min()), "lengths_max": int(lens.max())})


# ---------------------------------------------------------------------------
# A gated activation read from the two halves of one tensor: y = x[..., :N] * silu(x[..., N:]).
# Two slices of the last dimension of one input (index-remapped loads, Section 3.2): a
# supplementary shape for the benchmark sweep and the parity tests, not one of the named configs.
# ---------------------------------------------------------------------------
def gated_halves(M: int = 8192, N: int = 14336, seed: int = 0, dtype: int = D.BF16) -> Workload:
    g = GraphBuilder()
    x = g.input(dtype, (M, 2 * N))
    a = g.op("slice", [x], dtype, (M, N), attr=[1, 0])
    b = g.op("slice", [x], dtype, (M, N), attr=[1, N])
    cast = (lambda t: g.op("cast", [t], D.F32, (M, N))) if dtype != D.F32 else (lambda t: t)
    h = g.op("mul", [cast(a), g.op("silu", [cast(b)], D.F32, (M, N))], D.F32, (M, N))
    g.mark_output(g.op("cast", [h], dtype, (M, N)) if dtype != D.F32 else h)
    xv = _store(_draw(_rng(seed, 8, 0), "normal", (M, 2 * N), 0.0, 1.0), dtype)
    return _finish("gated_halves", g, ["x"], ["y"], [xv])


CONFIGS = {"c1": c1, "c2": c2, "c3": c3, "c4": c4, "c5": c5}
# subgraphs beyond the five benchmark ones (index-remapped loads; a reduction over a leading dimension)
EXTENDED = {"n1": n1, "n2": n2}

# Reduced sizes of the same graphs: several tiles plus a ragged tail each, small enough
# for the CPU oracle to finish in well under a second.
SMALL = {
    "c1": dict(M=37, N=1000),
    "c2": dict(B=3, Q=40, K=200),
    "c3": dict(M=33, N=1000),
    "c4": dict(M=5, N=10007),
    "c5": dict(M=19, N=1432),
    "n1": dict(S=21, SC=16, Cc=96),
    "n2": dict(B=3, S=37, Dh=200),
}
