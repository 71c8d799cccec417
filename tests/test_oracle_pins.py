"""Pins for the CPU oracle: it is checked here against things other than itself --
values the paper prints, textbook constants, invariants, brute force in pure Python
on tiny inputs, and special cases that reduce to a library routine.  CPU only."""
import math
import os
import struct

import numpy as np
import pytest

from oracle import evaluator as E
from pn_workloads import configs as C
from pn_workloads import descriptor as D
from pn_workloads.descriptor import GraphBuilder, Imm

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _gold(name):
    rows = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


def run1(op, arrays, dtypes, out_dtype, out_dims, imms=(), attr=(0, 0), extra_imm=()):
    """Evaluate a one-node graph through the oracle's public entry point."""
    g = GraphBuilder()
    ids = [g.input(dt, a.shape) for a, dt in zip(arrays, dtypes)]
    ins = list(ids) + [Imm(v) for v in imms]
    o = g.op(op, ins, out_dtype, out_dims, attr=attr, extra_imm=extra_imm)
    g.mark_output(o)
    return E.evaluate(g.build(), arrays)[0]


def f32(*v):
    return np.array(v, dtype=np.float32)


# ---------------------------------------------------------------------------
# descriptor format
# ---------------------------------------------------------------------------
def test_parser_reads_what_the_writer_wrote():
    w = C.c5(M=3, N=8)
    g = E.parse(w.desc)
    assert [g.tensors[i].dims for i in g.input_ids] == [(3, 8), (3, 8), (1, 8), (3, 1)]
    assert [n.op for n in g.nodes][-4:] == ["gt", "cast", "mean", "var"]
    gt = [n for n in g.nodes if n.op == "gt"][0]
    assert gt.ins[1] == ("imm", 0.0)
    # hand-assembled bytes for a one-node graph: neg(f32[2]) -> f32[2]
    raw = struct.pack("<IHHII", 0x31474E50, 1, 0, 2, 1)
    raw += struct.pack("<BBBBI4q", 0, 1, 1, 0, 0, 2, 0, 0, 0)
    raw += struct.pack("<BBBBI4q", 0, 2, 1, 0, 0, 2, 0, 0, 0)
    raw += struct.pack("<HBB4I3I2d2q", 1, 1, 1, 0, 0, 0, 0, 1, 0, 0, 0.0, 0.0, 0, 0)
    out = E.evaluate(raw, [f32(1.5, -2.0)])[0]
    assert out.tolist() == [-1.5, 2.0]


@pytest.mark.parametrize("mutate", ["short", "magic", "length", "opcode", "operand"])
def test_parser_rejects_malformed(mutate):
    good = bytearray(C.c1(M=2, N=4).desc)
    if mutate == "short":
        bad = good[:10]
    elif mutate == "magic":
        bad = good[:]; bad[0] ^= 0xFF
    elif mutate == "length":
        bad = good + b"\0"
    elif mutate == "opcode":
        bad = good[:]; struct.pack_into("<H", bad, 16 + 40 * 8, 999)
    else:
        bad = good[:]; struct.pack_into("<I", bad, 16 + 40 * 8 + 4, 77)
    with pytest.raises(ValueError):
        E.evaluate(bytes(bad), C.c1(M=2, N=4).inputs)


# ---------------------------------------------------------------------------
# activations: textbook constants, symmetries, libm
# ---------------------------------------------------------------------------
def test_activation_known_points():
    x = f32(0.0, 1.0, -1.0, 2.0)
    ge = run1("gelu_erf", [x], [D.F32], D.F32, (4,))
    # gelu_erf(1) = Phi(1), the standard normal CDF at one standard deviation
    assert ge[0] == 0.0 and abs(ge[1] - 0.8413447460685429) < 1e-15
    assert abs(ge[2] - (-(1 - 0.8413447460685429))) < 1e-15
    gt = run1("gelu_tanh", [x], [D.F32], D.F32, (4,))
    assert gt[0] == 0.0
    assert abs(gt[1] - 0.8411919906082768) < 1e-15
    assert abs(gt[2] + 0.15880800939172324) < 1e-15
    assert abs(gt[3] - 1.954597694087775) < 1e-15
    si = run1("silu", [x], [D.F32], D.F32, (4,))
    # silu(1) = 1/(1+1/e)
    assert si[0] == 0.0 and abs(si[1] - 0.7310585786300049) < 1e-15
    assert abs(si[2] + 0.2689414213699951) < 1e-15
    sg = run1("sigmoid", [x], [D.F32], D.F32, (4,))
    assert sg[0] == 0.5 and abs(sg[1] - 0.7310585786300049) < 1e-15


def test_activation_symmetries():
    rng = np.random.default_rng(1)
    x = rng.standard_normal(257).astype(np.float32) * 3
    xm = (-x).astype(np.float32)
    for op in ("gelu_tanh", "gelu_erf", "silu"):
        a = run1(op, [x], [D.F32], D.F32, x.shape)
        b = run1(op, [xm], [D.F32], D.F32, x.shape)
        # f(x) = x * s(x) with s(x) + s(-x) = 1  =>  f(x) - f(-x) = x
        np.testing.assert_allclose(a - b, x.astype(np.float64), rtol=0, atol=1e-14)
    s = run1("sigmoid", [x], [D.F32], D.F32, x.shape) + run1("sigmoid", [xm], [D.F32], D.F32, x.shape)
    np.testing.assert_allclose(s, 1.0, atol=1e-15)
    # gelu_erf through the complementary error function of libm
    ge = run1("gelu_erf", [x], [D.F32], D.F32, x.shape)
    ref = [0.5 * float(v) * math.erfc(-float(v) / math.sqrt(2)) for v in x]
    np.testing.assert_allclose(ge, ref, rtol=1e-13, atol=1e-15)
    # tanh through exponentials
    th = run1("tanh", [x], [D.F32], D.F32, x.shape)
    ref = [(math.exp(2 * float(v)) - 1) / (math.exp(2 * float(v)) + 1) for v in x]
    np.testing.assert_allclose(th, ref, rtol=1e-13, atol=1e-15)


def test_unary_binary_against_libm_scalars():
    x = f32(0.25, 1.0, 2.5, 9.0)
    table = {"exp": math.exp, "log": math.log, "sqrt": math.sqrt, "neg": lambda v: -v,
             "recip": lambda v: 1 / v, "rsqrt": lambda v: 1 / math.sqrt(v), "abs": abs,
             "square": lambda v: v * v, "erf": math.erf, "relu": lambda v: max(v, 0.0)}
    for op, fn in table.items():
        for arr in (x, (-x).astype(np.float32)) if op in ("neg", "abs", "relu", "erf", "square") else (x,):
            got = run1(op, [arr], [D.F32], D.F32, arr.shape)
            np.testing.assert_allclose(got, [fn(float(v)) for v in arr], rtol=1e-15)
    a, b = f32(3.0, -2.0, 0.5, 7.0), f32(2.0, 4.0, -0.5, 7.0)
    bt = {"add": lambda p, q: p + q, "sub": lambda p, q: p - q, "mul": lambda p, q: p * q,
          "div": lambda p, q: p / q, "max": max, "min": min}
    for op, fn in bt.items():
        got = run1(op, [a, b], [D.F32, D.F32], D.F32, (4,))
        assert got.tolist() == [fn(float(p), float(q)) for p, q in zip(a, b)]
    ct = {"gt": [1, 0, 1, 0], "ge": [1, 0, 1, 1], "lt": [0, 1, 0, 0], "le": [0, 1, 0, 1],
          "eq": [0, 0, 0, 1], "ne": [1, 1, 1, 0]}
    for op, want in ct.items():
        got = run1(op, [a, b], [D.F32, D.F32], D.BOOL, (4,))
        assert got.dtype == np.int64 and got.tolist() == want
    # sub is not commutative, div neither: operand order matters
    assert run1("sub", [a], [D.F32], D.F32, (4,), imms=[1.0]).tolist() == [2.0, -3.0, -0.5, 6.0]
    assert run1("fma", [a, b, a], [D.F32] * 3, D.F32, (4,)).tolist() == [9.0, -10.0, 0.25, 56.0]
    assert run1("clamp", [a], [D.F32], D.F32, (4,), imms=[0.0, 3.0]).tolist() == [3.0, 0.0, 0.5, 3.0]


def test_where_and_signed_zero():
    c = np.array([1, 0, -3, 0], dtype=np.int8)
    a, b = f32(1, 2, 3, 4), f32(-1, -2, -3, -4)
    assert run1("where", [c, a, b], [D.I8, D.F32, D.F32], D.F32, (4,)).tolist() == [1, -2, 3, -4]
    z = f32(-0.0, 0.0, 1e-30, -1e-30)
    assert run1("gt", [z], [D.F32], D.BOOL, (4,), imms=[0.0]).tolist() == [0, 0, 1, 0]


# ---------------------------------------------------------------------------
# reductions and composites
# ---------------------------------------------------------------------------
def test_softmax_invariants_and_brute_force():
    rng = np.random.default_rng(2)
    x = (np.rint(rng.standard_normal((7, 33)) * 2 * 1024) / 1024).astype(np.float32)   # multiples of 2^-10
    y = run1("softmax", [x], [D.F32], D.F32, x.shape)
    np.testing.assert_allclose(y.sum(-1), 1.0, atol=1e-12)
    assert (y >= 0).all() and (y <= 1).all()
    # brute force without the max shift (inputs are well scaled)
    for i in range(x.shape[0]):
        ex = [math.exp(float(v)) for v in x[i]]
        tot = math.fsum(ex)
        np.testing.assert_allclose(y[i], [e / tot for e in ex], rtol=1e-13)
    # shift invariance, with a shift that is exact in fp32 for these magnitudes
    xs = (x + np.float32(8.0)).astype(np.float32)
    assert np.array_equal(xs.astype(np.float64) - 8.0, x.astype(np.float64))
    np.testing.assert_allclose(run1("softmax", [xs], [D.F32], D.F32, x.shape), y, rtol=1e-12)
    # the row maximum is subtracted first: inputs near 1000 would overflow e^x otherwise
    xb = (x + np.float32(1000.0)).astype(np.float32)
    assert np.array_equal(xb.astype(np.float64) - 1000.0, x.astype(np.float64))
    np.testing.assert_allclose(run1("softmax", [xb], [D.F32], D.F32, x.shape), y, rtol=1e-12)
    # masked entries are exactly zero; a fully masked row is NaN
    xm = x.copy(); xm[:, 5:] = -np.inf; xm[3, :] = -np.inf
    ym = run1("softmax", [xm], [D.F32], D.F32, x.shape)
    assert (ym[[0, 1, 2, 4, 5, 6], 5:] == 0).all() and np.isnan(ym[3]).all()
    np.testing.assert_allclose(ym[0, :5].sum(), 1.0, atol=1e-13)


def test_c2_structure():
    w = C.c2(B=2, Q=9, K=9)
    y = E.evaluate(w.desc, w.inputs)[0]
    for q in range(9):
        assert (np.count_nonzero(y[:, q, :], axis=-1) == q + 1).all()   # causal: k <= q
        assert (y[:, q, q + 1:] == 0).all()
    assert (y[:, 0, 0] == 1.0).all()
    np.testing.assert_allclose(y.sum(-1), 1.0, atol=1e-12)
    # row q = 1: two survivors, closed form 1/(1+e^{(s1-s0)/8})
    s = E.widen(w.inputs[0], D.BF16)
    want = 1.0 / (1.0 + np.exp((s[:, 1, 1] - s[:, 1, 0]) * 0.125))
    np.testing.assert_allclose(y[:, 1, 0], want, rtol=1e-13)


def test_logsumexp_pins():
    rng = np.random.default_rng(3)
    x = (np.rint(rng.standard_normal((5, 41)) * 3 * 1024) / 1024).astype(np.float32)   # multiples of 2^-10
    l = run1("logsumexp", [x], [D.F32], D.F32, (5,))
    for i in range(5):
        m = max(float(v) for v in x[i])
        ref = m + math.log(math.fsum(math.exp(float(v) - m) for v in x[i]))
        assert abs(l[i] - ref) < 1e-13
        assert m <= l[i] <= m + math.log(41)
    c = np.full((2, 16), 1.25, dtype=np.float32)
    np.testing.assert_allclose(run1("logsumexp", [c], [D.F32], D.F32, (2,)), 1.25 + math.log(16), rtol=1e-15)
    xs = (x + np.float32(4.0)).astype(np.float32)
    assert np.array_equal(xs.astype(np.float64) - 4.0, x.astype(np.float64))
    np.testing.assert_allclose(run1("logsumexp", [xs], [D.F32], D.F32, (5,)), l + 4.0, rtol=1e-13)
    inf = np.full((1, 4), -np.inf, dtype=np.float32)
    assert run1("logsumexp", [inf], [D.F32], D.F32, (1,))[0] == -np.inf
    inf[0, 2] = np.inf
    assert run1("logsumexp", [inf], [D.F32], D.F32, (1,))[0] == np.inf
    # keepdim form of the declared shape is honoured
    assert run1("logsumexp", [x], [D.F32], D.F32, (5, 1)).shape == (5, 1)
    # relation to softmax: log(softmax) = x - lse
    ls = run1("log_softmax", [x], [D.F32], D.F32, x.shape)
    sm = run1("softmax", [x], [D.F32], D.F32, x.shape)
    np.testing.assert_allclose(ls, np.log(sm), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(ls, x.astype(np.float64) - l[:, None], rtol=1e-13, atol=1e-13)


def test_c4_closed_form():
    w = C.c4(M=4, N=50000)
    x = w.inputs[0]
    lse, idx = E.evaluate(w.desc, w.inputs)
    assert idx.dtype == np.int64
    for i in range(4):
        hits = [j for j in range(x.shape[1]) if x[i, j] == np.float32(30.0)]
        assert len(hits) >= 2                       # ties exist; lowest index must win
        assert idx[i] == hits[0]
        # the other entries are N(0, var 4): they add less than 1e-6 to the sum
        assert 0 <= lse[i] - (30.0 + math.log(len(hits))) < 1e-6 / len(hits) * 50


def test_argmax_argmin_brute_force_and_nan():
    rng = np.random.default_rng(4)
    x = rng.integers(-3, 4, size=(20, 17)).astype(np.float32)      # many ties
    am = run1("argmax", [x], [D.F32], D.I64, (20,))
    an = run1("argmin", [x], [D.F32], D.I64, (20,))
    for i in range(20):
        best = 0
        worst = 0
        for j in range(17):
            if x[i, j] > x[i, best]:
                best = j
            if x[i, j] < x[i, worst]:
                worst = j
        assert am[i] == best and an[i] == worst
    xn = x.copy(); xn[2, 9] = np.nan; xn[2, 12] = np.nan
    assert run1("argmax", [xn], [D.F32], D.I64, (20,))[2] == 9
    assert run1("argmin", [xn], [D.F32], D.I64, (20,))[2] == 9
    assert np.isnan(run1("amax", [xn], [D.F32], D.F32, (20,))[2])
    assert run1("amax", [x], [D.F32], D.F32, (20,)).tolist() == [float(max(r)) for r in x]
    assert run1("amin", [x], [D.F32], D.F32, (20,)).tolist() == [float(min(r)) for r in x]


def test_mean_var_pins():
    v = np.arange(1, 9, dtype=np.float32)[None, :]               # 1..8: mean 4.5, var 5.25 / 6
    assert run1("mean", [v], [D.F32], D.F32, (1,))[0] == 4.5
    assert run1("sum", [v], [D.F32], D.F32, (1,))[0] == 36.0
    assert run1("var", [v], [D.F32], D.F32, (1,), attr=(0, 0))[0] == 5.25
    assert run1("var", [v], [D.F32], D.F32, (1,), attr=(1, 0))[0] == 6.0
    c = np.full((3, 10), -2.5, dtype=np.float32)
    assert (run1("var", [c], [D.F32], D.F32, (3,))[...] == 0).all()
    rng = np.random.default_rng(5)
    x = rng.standard_normal((6, 29)).astype(np.float32)
    var = run1("var", [x], [D.F32], D.F32, (6,))
    for i in range(6):
        xs = [float(t) for t in x[i]]
        ex2 = math.fsum(t * t for t in xs) / 29
        ex = math.fsum(xs) / 29
        assert abs(var[i] - (ex2 - ex * ex)) < 1e-13


def test_layer_norm_pins():
    gold = dict((k, float(v)) for k, v in _gold("layernorm_case.txt"))
    v = np.arange(1, 9, dtype=np.float32)[None, :]
    g = GraphBuilder()
    x = g.input(D.F32, (1, 8)); ga = g.input(D.F32, (8,)); be = g.input(D.F32, (8,))
    y, mean, rstd = g.node("layer_norm", [x, ga, be], [D.F32] * 3, [(1, 8), (1,), (1,)],
                           extra_imm=[gold["eps"]])
    for t in (y, mean, rstd):
        g.mark_output(t)
    yo, mo, ro = E.evaluate(g.build(), [v, np.full(8, 2, np.float32), np.full(8, -1, np.float32)])
    assert mo[0] == gold["mean"]
    assert abs(1.0 / ro[0] ** 2 - (gold["biased_var"] + gold["eps"])) < 1e-12
    want = [(j - 4.5) / math.sqrt(5.25 + 1e-5) * 2 - 1 for j in range(1, 9)]
    np.testing.assert_allclose(yo[0], want, rtol=1e-14)
    # invariants on random rows with gamma = 1, beta = 0
    rng = np.random.default_rng(6)
    xr = (rng.standard_normal((9, 64)) * 1.5 + 0.3).astype(np.float32)
    g = GraphBuilder(); x = g.input(D.F32, (9, 64))
    y, mean, rstd = g.node("layer_norm", [x], [D.F32] * 3, [(9, 64), (9,), (9,)], extra_imm=[1e-5])
    for t in (y, mean, rstd):
        g.mark_output(t)
    yo, mo, ro = E.evaluate(g.build(), [xr])
    np.testing.assert_allclose(yo.mean(-1), 0, atol=1e-12)
    var = xr.astype(np.float64).var(-1)
    np.testing.assert_allclose(yo.var(-1), var / (var + 1e-5), rtol=1e-12)      # "1" up to eps
    np.testing.assert_allclose(ro ** 2 * (var + 1e-5), 1.0, rtol=1e-13)
    # affine part
    ga = rng.uniform(0.5, 1.5, 64).astype(np.float32); be = rng.standard_normal(64).astype(np.float32)
    g = GraphBuilder(); x = g.input(D.F32, (9, 64)); a = g.input(D.F32, (64,)); b = g.input(D.F32, (64,))
    g.mark_output(g.node("layer_norm", [x, a, b], [D.F32], [(9, 64)], extra_imm=[1e-5])[0])
    np.testing.assert_allclose(E.evaluate(g.build(), [xr, ga, be])[0],
                               yo * ga.astype(np.float64) + be.astype(np.float64), rtol=1e-14, atol=1e-15)
    # rms_norm: unit gamma gives rows whose mean square is ms/(ms+eps)
    yr = run1("rms_norm", [xr], [D.F32], D.F32, xr.shape, extra_imm=[1e-6])
    ms = (xr.astype(np.float64) ** 2).mean(-1)
    np.testing.assert_allclose((yr ** 2).mean(-1), ms / (ms + 1e-6), rtol=1e-12)
    assert np.sign(yr[0, 0]) == np.sign(xr[0, 0])


def test_clamped_divide_of_masked_mean_pooling():
    # out = sum(h*m) / max(sum(m), 1e-9): the epilogue of the paper's pooling kernel
    floor = dict((k, float(v)) for k, v in _gold("layernorm_case.txt"))["clamp_floor"]
    h = f32(1, 2, 3, 4, 5, 6).reshape(2, 3)
    m = f32(1, 0, 1, 0, 0, 0).reshape(2, 3)
    g = GraphBuilder()
    hi = g.input(D.F32, (2, 3)); mi = g.input(D.F32, (2, 3))
    p = g.op("mul", [hi, mi], D.F32, (2, 3))
    s = g.op("sum", [p], D.F32, (2, 1)); c = g.op("sum", [mi], D.F32, (2, 1))
    cc = g.op("clamp", [c, Imm(floor), Imm(math.inf)], D.F32, (2, 1))
    g.mark_output(g.op("div", [s, cc], D.F32, (2, 1)))
    assert E.evaluate(g.build(), [h, m])[0].ravel().tolist() == [2.0, 0.0]


# ---------------------------------------------------------------------------
# broadcasting and casts
# ---------------------------------------------------------------------------
def test_broadcasting_matches_explicit_materialisation():
    rng = np.random.default_rng(7)
    a = rng.standard_normal((2, 3, 1, 5)).astype(np.float32)
    b = rng.standard_normal((3, 4, 1)).astype(np.float32)
    got = run1("mul", [a, b], [D.F32, D.F32], D.F32, (2, 3, 4, 5))
    full_a = np.empty((2, 3, 4, 5)); full_b = np.empty((2, 3, 4, 5))
    for i in range(2):
        for j in range(3):
            for k in range(4):
                for l in range(5):
                    full_a[i, j, k, l] = a[i, j, 0, l]; full_b[i, j, k, l] = b[j, k, 0]
    assert np.array_equal(got, full_a * full_b)


def test_bf16_widen_exhaustive_and_narrow_ties():
    bits = np.arange(65536, dtype=np.uint16)
    got = E.widen(bits, D.BF16)
    ref = np.array([struct.unpack("<f", struct.pack("<I", int(b) << 16))[0] for b in bits])
    assert np.array_equal(got[~np.isnan(ref)], ref[~np.isnan(ref)]) and np.isnan(got[np.isnan(ref)]).all()
    # every bf16 value rounds to itself
    fin = np.isfinite(ref)
    assert np.array_equal(E.round_to_bf16(ref[fin]), ref[fin])
    # ties to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7 -> 1; 1 + 3*2^-8 -> 1 + 2^-6
    r = E.round_to_bf16(np.array([1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8, 1 + 2.0 ** -8 + 2.0 ** -30,
                                  -(1 + 2.0 ** -8), 3.4e38, 2.0 ** -133 * 1.5, 1e-45]))
    assert r.tolist() == [1.0, 1 + 2.0 ** -6, 1 + 2.0 ** -7, -1.0, np.inf, 2.0 ** -132, 0.0]
    # the midpoint of two neighbours always lands on the one with the even mantissa
    pos = np.sort(ref[fin & (ref > 0)])
    mids = (pos[:-1] + pos[1:]) / 2
    rm = E.round_to_bf16(mids)
    lo_bits = np.arange(1, len(pos))            # bit pattern of pos[k] is k+1
    want = np.where(lo_bits % 2 == 0, pos[:-1], pos[1:])
    assert np.array_equal(rm, want)
    # Table 2's accepted bf16 "max diff" is one spacing of bf16 in [4, 8)
    name, printed, lo, hi = _gold("sparkle_max_diff.txt")[0]
    sp = E.round_to_bf16(np.array([float(lo) + 1e-9 + 2.0 ** -6])) - float(lo)
    assert sp[0] == 2.0 ** -5 and round(float(sp[0]), 3) == float(printed)
    # fp16 narrowing agrees with the IEEE half type
    assert E.round_to_f16(np.array([1 + 2.0 ** -11, 65520.0])).tolist() == [1.0, np.inf]


def test_declared_narrow_intermediate_is_rounded_for_consumers_only():
    x = f32(1.00390625 * 3)                      # 3.01171875 is not a bf16 value
    g = GraphBuilder()
    xi = g.input(D.F32, (1,))
    nb = g.op("cast", [xi], D.BF16, (1,))        # declared bf16, consumed below
    d = g.op("sub", [nb, xi], D.F32, (1,))
    g.mark_output(nb); g.mark_output(d)
    out_nb, out_d = E.evaluate(g.build(), [x])
    assert out_nb[0] == float(x[0])              # outputs are reported unrounded
    assert out_d[0] == 3.015625 - float(x[0])    # the consumer saw the rounded value
    # float -> int truncates toward zero; int8 -> float is exact
    assert run1("cast", [f32(2.9, -2.9)], [D.F32], D.I32, (2,)).tolist() == [2, -2]
    assert run1("cast", [np.array([-128, 127], np.int8)], [D.I8], D.F32, (2,)).tolist() == [-128.0, 127.0]


# ---------------------------------------------------------------------------
# whole graphs: a third restatement in pure Python on tiny shapes
# ---------------------------------------------------------------------------
def _bf(a):
    return E.widen(a, D.BF16)


def test_c1_restated():
    w = C.c1(M=3, N=5)
    x, ww, b, r = [a.astype(np.float64) for a in w.inputs]
    y = E.evaluate(w.desc, w.inputs)[0]
    for i in range(3):
        for j in range(5):
            u = x[i, j] * ww[j] + b[j]
            ref = 0.5 * u * (1 + math.tanh(math.sqrt(2 / math.pi) * (u + 0.044715 * u ** 3))) + r[i, j]
            assert abs(y[i, j] - ref) < 1e-14


def test_c3_restated():
    w = C.c3(M=4, N=12, also_output_sum=True)
    x, res = _bf(w.inputs[0]), _bf(w.inputs[1])
    ga, be = w.inputs[2].astype(np.float64), w.inputs[3].astype(np.float64)
    out = dict(zip(w.output_names, E.evaluate(w.desc, w.inputs)))
    for i in range(4):
        h = [x[i, j] + res[i, j] for j in range(12)]
        mu = math.fsum(h) / 12
        var = math.fsum((t - mu) ** 2 for t in h) / 12
        rs = 1 / math.sqrt(var + 1e-5)
        assert abs(out["mean"][i] - mu) < 1e-14 and abs(out["rstd"][i] - rs) < 1e-13
        for j in range(12):
            assert abs(out["y"][i, j] - ((h[j] - mu) * rs * ga[j] + be[j])) < 1e-13
            assert out["h"][i, j] == h[j]


def test_c5_restated_and_mask_identity():
    w = C.c5(M=5, N=24)
    a, gt, col, row = [_bf(t) for t in w.inputs]
    h, mask, mean, var = E.evaluate(w.desc, w.inputs)
    assert mask.dtype == np.int64 and np.array_equal(mask, (a > 0).astype(np.int64))
    for i in range(5):
        hr = [a[i, j] * (1 / (1 + math.exp(-gt[i, j]))) * col[0, j] * row[i, 0] for j in range(24)]
        np.testing.assert_allclose(h[i], hr, rtol=1e-14)
        mu = math.fsum(hr) / 24
        assert abs(mean[i] - mu) < 1e-14
        assert abs(var[i] - math.fsum((t - mu) ** 2 for t in hr) / 24) < 1e-14


# ---------------------------------------------------------------------------
# the comparison rule
# ---------------------------------------------------------------------------
def test_tolerance_rule_matches_the_papers_ladder():
    rows = {r[0]: r for r in _gold("tolerance_ladder.txt")}
    # bf16 rtol used here is the paper's printed t = -5 value, itself 10^(-1.796) to two digits
    k = float(rows["bfloat16"][1])
    assert float(f"{10 ** (-5 * k / 5):.1e}") == float(rows["bfloat16"][2]) == E.TOLERANCES[D.BF16][0]
    assert float(rows["float16"][2]) == E.TOLERANCES[D.F16][0] and float(rows["float16"][3]) == E.TOLERANCES[D.F16][1]
    assert float(f"{10 ** (-float(rows['float32'][1])):.1e}") == float(rows["float32"][2])
    assert float(rows["others"][2]) == 0.0       # integers and booleans: exact
    ref = np.array([1.0, 100.0, 0.0, np.inf, np.nan])
    ok = E.compare(ref * (1 + 9e-6) + np.array([0, 0, 9e-7, 0, 0]), ref, D.F32)
    assert ok["ok"] and ok["violations"] == 0
    assert not E.compare(ref * (1 + 2e-5), ref, D.F32)["ok"]
    assert not E.compare(np.array([1.0, 100.0, 0.0, -np.inf, np.nan]), ref, D.F32)["ok"]
    assert not E.compare(np.array([1.0, 100.0, 0.0, np.inf, 0.0]), ref, D.F32)["ok"]
    assert not E.compare(np.array([1.0, np.nan, 0.0, np.inf, np.nan]), ref, D.F32)["ok"]
    assert E.compare(np.array([1.015]), np.array([1.0]), D.BF16)["ok"]
    assert not E.compare(np.array([1.02]), np.array([1.0]), D.BF16)["ok"]
    # a reference beyond the output type's range is an infinity once stored (IEEE overflow)
    assert E.compare(np.array([np.inf, -np.inf]), np.array([2.7e43, -1e39]), D.F32)["ok"]
    assert not E.compare(np.array([3.0e38]), np.array([2.7e43]), D.F32)["ok"]
    assert E.compare(np.array([np.inf]), np.array([70000.0]), D.F16)["ok"]
    assert not E.compare(np.array([np.inf]), np.array([3.0e38]), D.F32)["ok"]
    assert not E.compare(np.array([1, 2, 4]), np.array([1, 2, 3]), D.I64)["ok"]
    assert E.compare(np.array([1, 2, 3], np.int8), np.array([1, 2, 3]), D.I8)["ok"]


# ---------------------------------------------------------------------------
# index operators: roll + slice as the paper's index arithmetic
# ---------------------------------------------------------------------------
def test_roll_slice_view_match_the_papers_index_formula():
    """Section 4.4 / Appendix H, case 1: roll(shift) followed by slice[:SC] on an [S, S, C] tensor
    equals reading row (S + i - shift) mod S, column (S + j - shift) mod S."""
    S, SC, Cc, shift = 7, 5, 4, 3
    rng = np.random.default_rng(9)
    x = rng.standard_normal((1, S * S, Cc)).astype(np.float32)
    g = GraphBuilder()
    xi = g.input(D.F32, x.shape)
    v = g.op("view", [xi], D.F32, (S, S, Cc))
    r = g.op("roll", [g.op("roll", [v], D.F32, (S, S, Cc), attr=[0, shift])], D.F32, (S, S, Cc), attr=[1, shift])
    s = g.op("slice", [g.op("slice", [r], D.F32, (SC, S, Cc), attr=[0, 0])], D.F32, (SC, SC, Cc), attr=[1, 0])
    g.mark_output(g.op("view", [s], D.F32, (1, SC * SC, Cc)))
    got = E.evaluate(g.build(), [x])[0]
    x3 = x.reshape(S, S, Cc)
    for i in range(SC):
        for j in range(SC):
            src = x3[(S + i - shift) % S, (S + j - shift) % S]
            assert np.array_equal(got[0, i * SC + j], src.astype(np.float64))
    # negative and oversized shifts wrap; a slice that starts inside the tensor
    a = np.arange(10, dtype=np.float32).reshape(5, 2)
    for sh in (-1, 7):
        out = run1("roll", [a], [D.F32], D.F32, (5, 2), attr=(0, sh))
        assert out[:, 0].tolist() == [float(a[(i - sh) % 5, 0]) for i in range(5)]
    out = run1("slice", [a], [D.F32], D.F32, (2, 2), attr=(0, 2))
    assert out.tolist() == [[4.0, 5.0], [6.0, 7.0]]
    # the same two operators along the last dimension (the halves of a gated activation are two such
    # slices of one tensor), element by element from the definition
    b = np.arange(12, dtype=np.float32).reshape(2, 6)
    for sh in (2, -1, 13):
        out = run1("roll", [b], [D.F32], D.F32, (2, 6), attr=(1, sh))
        assert out.tolist() == [[float(b[i, (j - sh) % 6]) for j in range(6)] for i in range(2)]
    out = run1("slice", [b], [D.F32], D.F32, (2, 3), attr=(1, 3))
    assert out.tolist() == [[3.0, 4.0, 5.0], [9.0, 10.0, 11.0]]


def test_n1_restated():
    w = C.n1(S=6, SC=4, Cc=8, shift=2)
    x, res, ga, be = [_bf(t) for t in w.inputs]
    out = dict(zip(w.output_names, E.evaluate(w.desc, w.inputs)))
    x3 = x.reshape(6, 6, 8)
    for i in range(4):
        for j in range(4):
            h = [res[0, i * 4 + j, c] + x3[(6 + i - 2) % 6, (6 + j - 2) % 6, c] for c in range(8)]
            mu = math.fsum(h) / 8
            var = math.fsum((t - mu) ** 2 for t in h) / 8
            for c in range(8):
                assert out["add"][0, i * 4 + j, c] == h[c]
                ref = (h[c] - mu) / math.sqrt(var + 1e-5) * ga[c] + be[c]
                assert abs(out["layer_norm"][0, i * 4 + j, c] - ref) < 1e-12


# ---------------------------------------------------------------------------
# reductions over a leading dimension, cat, and masked mean pooling
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("shape,dim", [((5, 3), 0), ((4, 6, 5), 1), ((4, 6, 5), 0), ((2, 3, 4, 5), 2), ((2, 3, 4, 5), 1)])
def test_reductions_over_a_leading_dimension_brute_force(shape, dim):
    x = np.random.default_rng(21).standard_normal(shape).astype(np.float32)
    out_shape = shape[:dim] + shape[dim + 1:]
    got = {op: run1(op, [x], [D.F32], D.F32, out_shape, attr=(dim, 0)) for op in ("sum_dim", "mean_dim", "amax_dim", "amin_dim")}
    for idx in np.ndindex(*out_shape):
        line = [float(x[idx[:dim] + (k,) + idx[dim:]]) for k in range(shape[dim])]
        assert abs(got["sum_dim"][idx] - math.fsum(line)) < 1e-13
        assert abs(got["mean_dim"][idx] - math.fsum(line) / len(line)) < 1e-14
        assert got["amax_dim"][idx] == max(line) and got["amin_dim"][idx] == min(line)
    # the reduced dimension kept as 1 is the same values under the other shape
    kept = shape[:dim] + (1,) + shape[dim + 1:]
    assert np.array_equal(run1("sum_dim", [x], [D.F32], D.F32, kept, attr=(dim, 0)).reshape(out_shape), got["sum_dim"])


def test_reductions_over_a_leading_dimension_closed_forms_and_nan():
    # x[b, s, d] = b + 10 s + 100 d:  sum over s = S b + 10 S (S - 1) / 2 + 100 S d
    B, S, Dh = 3, 7, 4
    b, s, d = np.meshgrid(np.arange(B), np.arange(S), np.arange(Dh), indexing="ij")
    x = (b + 10 * s + 100 * d).astype(np.float32)
    tot = run1("sum_dim", [x], [D.F32], D.F32, (B, Dh), attr=(1, 0))
    for bb in range(B):
        for dd in range(Dh):
            assert tot[bb, dd] == S * bb + 10 * S * (S - 1) // 2 + 100 * S * dd
    assert np.array_equal(run1("amax_dim", [x], [D.F32], D.F32, (B, Dh), attr=(1, 0)), x[:, S - 1, :])
    assert np.array_equal(run1("amin_dim", [x], [D.F32], D.F32, (B, Dh), attr=(1, 0)), x[:, 0, :])
    x[1, 3, 2] = np.nan
    mx = run1("amax_dim", [x], [D.F32], D.F32, (B, Dh), attr=(1, 0))
    assert np.isnan(mx[1, 2]) and np.isnan(mx).sum() == 1
    assert np.isnan(run1("sum_dim", [x], [D.F32], D.F32, (B, Dh), attr=(1, 0))[1, 2])
    # integer tensors are summed exactly
    m = np.arange(24, dtype=np.int64).reshape(2, 3, 4) % 2
    cnt = run1("sum_dim", [m], [D.I64], D.F32, (2, 4), attr=(1, 0))
    assert cnt.tolist() == [[0.0, 3.0, 0.0, 3.0], [0.0, 3.0, 0.0, 3.0]]


def test_cat_of_one_operand_is_the_identity_and_of_two_is_stacking():
    a = np.arange(6, dtype=np.float32).reshape(2, 3); b = -a
    assert np.array_equal(run1("cat", [a], [D.F32], D.F32, (2, 3), attr=(1, 0)), a)
    out = run1("cat", [a, b], [D.F32, D.F32], D.F32, (2, 6), attr=(1, 0))
    assert out.tolist() == [[0, 1, 2, -0.0, -1, -2], [3, 4, 5, -3, -4, -5]]
    out = run1("cat", [a, b], [D.F32, D.F32], D.F32, (4, 3), attr=(0, 0))
    assert out[2:].tolist() == b.tolist() and out[:2].tolist() == a.tolist()


@pytest.mark.parametrize("dense_mask,mask_dtype", [(False, D.I64), (True, D.F32), (True, D.I8)])
def test_n2_masked_mean_pooling_restated(dense_mask, mask_dtype):
    """Appendix H, case 2: out[b, d] = sum_s(hidden * mask) / max(sum_s(mask), 1e-9)."""
    w = C.n2(B=3, S=9, Dh=5, dense_mask=dense_mask, mask_dtype=mask_dtype)
    mask, hidden = w.inputs
    h = _bf(hidden)
    m = np.broadcast_to(np.asarray(mask, dtype=np.float64), h.shape)
    out = E.evaluate(w.desc, w.inputs)[0]
    assert out.shape == (3, 5)
    for b in range(3):
        for d in range(5):
            num = math.fsum(h[b, s, d] * m[b, s, d] for s in range(9))
            cnt = math.fsum(m[b, s, d] for s in range(9))
            assert abs(out[b, d] - num / max(cnt, 1e-9)) < 1e-14
    assert 1 <= w.notes["lengths_min"] <= w.notes["lengths_max"] <= 9


def test_masked_mean_pooling_special_cases():
    rows = dict((r[0], r) for r in _gold("sparkle_max_diff.txt"))
    assert float(rows["masked_mean_pooling"][1]) == 0.0      # Table 2: the fused kernel is bitwise identical
    w = C.n2(B=4, S=6, Dh=8)
    mask, hidden = [a.copy() for a in w.inputs]
    h = _bf(hidden)
    mask[0, :, 0] = 1                     # nothing masked: the plain mean over S
    mask[1, :, 0] = 0                     # everything masked: 0 / 1e-9 = 0
    mask[2, :, 0] = 0; mask[2, 4, 0] = 1  # one position kept: that row of hidden, exactly
    out = E.evaluate(w.desc, [mask, hidden])[0]
    assert np.allclose(out[0], h[0].sum(axis=0) / 6, rtol=0, atol=1e-15)
    assert np.array_equal(out[1], np.zeros(8))
    assert np.array_equal(out[2], h[2, 4])


# ---------------------------------------------------------------------------
# conventions at the edges: NaN operands, casts to bool / integer, gamma of rms_norm, fp16 rounding.
# Each expected value below is written out by hand or comes from the struct module's IEEE half
# conversion, never from the function under test.
# ---------------------------------------------------------------------------
def test_binary_max_min_propagate_nan_from_either_operand():
    """Pins `max` / `min`: the elementwise maximum of array libraries returns NaN when either
    operand is NaN (an `fmax`-style "ignore the NaN" would return the number instead)."""
    nan = float("nan")
    a, b = f32(nan, 1.0, nan, -2.0, 3.0), f32(1.0, nan, nan, 5.0, -7.0)
    mx = run1("max", [a, b], [D.F32, D.F32], D.F32, (5,))
    mn = run1("min", [a, b], [D.F32, D.F32], D.F32, (5,))
    assert np.isnan(mx[:3]).all() and mx[3:].tolist() == [5.0, 3.0]
    assert np.isnan(mn[:3]).all() and mn[3:].tolist() == [-2.0, -7.0]
    # the same through an immediate operand, and through clamp (max then min)
    assert np.isnan(run1("max", [f32(nan)], [D.F32], D.F32, (1,), imms=[0.0])[0])
    cl = run1("clamp", [f32(nan, -9.0, 9.0)], [D.F32], D.F32, (3,), imms=[-1.0, 1.0])
    assert np.isnan(cl[0]) and cl[1:].tolist() == [-1.0, 1.0]


def test_relu_keeps_nan_and_maps_the_rest_of_the_extended_line():
    """Pins `relu`: NaN stays NaN (a `where(x > 0, x, 0)` would give 0), -inf -> 0, +inf stays."""
    got = run1("relu", [f32(float("nan"), -np.inf, np.inf, -0.0, -1e-30, 2.5)], [D.F32], D.F32, (6,))
    assert np.isnan(got[0]) and got[1:].tolist() == [0.0, np.inf, 0.0, 0.0, 2.5]


def test_logsumexp_of_rows_holding_nan_or_infinities():
    """Pins the special rows of `logsumexp`: a NaN anywhere gives NaN (also beside an infinity),
    a +inf gives +inf, a row of -inf gives -inf, and -inf entries add nothing."""
    nan, inf = float("nan"), np.inf
    x = np.array([[0.0, nan, 1.0], [nan, inf, 0.0], [inf, 0.0, -inf], [-inf, -inf, -inf], [-inf, 0.0, 0.0]], dtype=np.float32)
    got = run1("logsumexp", [x], [D.F32], D.F32, (5,))
    assert np.isnan(got[0]) and np.isnan(got[1]) and got[2] == inf and got[3] == -inf
    assert got[4] == math.log(2.0)
    # log_softmax of the NaN row is NaN throughout; softmax likewise
    assert np.isnan(run1("log_softmax", [x[:1]], [D.F32], D.F32, (1, 3))).all()
    assert np.isnan(run1("softmax", [x[:1]], [D.F32], D.F32, (1, 3))).all()


def test_cast_to_bool_and_to_integers():
    """Pins `cast`: to bool is "non-zero" (so -0.0 is false, NaN and fractions are true); float to
    integer truncates toward zero; integer to float keeps the value."""
    src = f32(0.0, -0.0, 0.5, float("nan"), -3.0, 1e-40)
    assert run1("cast", [src], [D.F32], D.BOOL, (6,)).tolist() == [0, 0, 1, 1, 1, 1]
    assert run1("cast", [f32(-1.7, 1.7, -0.5, 0.99, 126.5)], [D.F32], D.I8, (5,)).tolist() == [-1, 1, 0, 0, 126]
    assert run1("cast", [f32(-1.7, 70000.9)], [D.F32], D.I32, (2,)).tolist() == [-1, 70000]
    assert run1("cast", [np.array([-128, 0, 127], np.int8)], [D.I8], D.BOOL, (3,)).tolist() == [1, 0, 1]
    back = run1("cast", [np.array([-5, 0, 2**40], np.int64)], [D.I64], D.F32, (3,))
    assert back.dtype == np.float64 and back.tolist() == [-5.0, 0.0, float(2**40)]


def test_rms_norm_with_gamma_against_plain_python():
    """Pins `rms_norm`'s gamma: y_j = x_j / sqrt(sum(x^2)/N + eps) * gamma_j, restated with
    Python floats (a dropped or transposed gamma, or eps outside the root, fails)."""
    x = [[3.0, -4.0, 12.0, 0.5], [1.0, 1.0, -1.0, 2.0]]
    gamma = [2.0, -0.5, 0.25, 3.0]
    eps = 0.125
    want = []
    for row in x:
        ms = sum(v * v for v in row) / len(row)
        want.append([v / math.sqrt(ms + eps) * g for v, g in zip(row, gamma)])
    got = run1("rms_norm", [np.array(x, np.float32), np.array(gamma, np.float32)], [D.F32, D.F32], D.F32, (2, 4), extra_imm=[eps])
    np.testing.assert_allclose(got, want, rtol=1e-15)
    # 3-4-12 with eps = 0: the root mean square is 13/2 exactly
    g0 = run1("rms_norm", [f32(3.0, 4.0, 12.0, 0.0)[None, :]], [D.F32], D.F32, (1, 4), extra_imm=[0.0])
    np.testing.assert_allclose(g0[0], [6.0 / 13.0, 8.0 / 13.0, 24.0 / 13.0, 0.0], rtol=1e-15)


def test_round_to_f16_against_the_ieee_half_type_everywhere():
    """Pins `round_to_f16` against the struct module's binary16 conversion: every finite half
    value is a fixed point, every midpoint of two neighbouring halves goes to the one with the
    even mantissa, points a little to either side of a midpoint go to their nearer neighbour,
    and the overflow threshold is 65520."""
    bits = np.arange(0x7C00, dtype=np.uint16)                      # all non-negative finite halves
    vals = np.array([struct.unpack("<e", struct.pack("<H", int(b)))[0] for b in bits])
    assert np.array_equal(E.round_to_f16(vals), vals) and np.array_equal(E.round_to_f16(-vals), -vals)
    mids = (vals[:-1] + vals[1:]) / 2
    want_mid = np.where(bits[:-1] % 2 == 0, vals[:-1], vals[1:])
    assert np.array_equal(E.round_to_f16(mids), want_mid)
    gap = vals[1:] - vals[:-1]
    assert np.array_equal(E.round_to_f16(mids - gap / 8), vals[:-1]) and np.array_equal(E.round_to_f16(mids + gap / 8), vals[1:])
    # the struct module agrees on the same points (it rounds a double to half, nearest even)
    probe = np.concatenate([mids[::97], mids[::89] + gap[::89] / 8, vals[::101] * (1 + 2.0 ** -30)])
    ref = np.array([struct.unpack("<e", struct.pack("<e", float(v)))[0] for v in probe])
    assert np.array_equal(E.round_to_f16(probe), ref)
    assert E.round_to_f16(np.array([65519.9, 65520.0, -65520.0, 2.0 ** -25, 2.0 ** -25 * 1.01])).tolist() == [65504.0, np.inf, -np.inf, 0.0, 2.0 ** -24]
