"""GPU parity of every operator of the descriptor format against the CPU oracle, through the
C ABI: one-node and small multi-node graphs over ragged shapes, broadcast patterns, storage
types and the special values (NaN, infinities, ties, fully masked rows), each on the
generated kernels and on the interpreter."""
import math

import numpy as np
import pytest

import paper_2605_29357_b200 as pn
from oracle import evaluator as E
from pn_workloads import configs as C
from pn_workloads import descriptor as D
from pn_workloads.descriptor import GraphBuilder, Imm

from gpu_util import check_against_oracle, run_graph

pytestmark = pytest.mark.gpu

MODES = {"generated": 0, "interpreter": pn.FLAG_INTERPRET}


def rnd(shape, seed, scale=1.0, dtype=D.F32):
    x = (np.random.default_rng(seed).standard_normal(shape) * scale).astype(np.float32)
    return x if dtype == D.F32 else (C.to_bf16_bits(x) if dtype == D.BF16 else x.astype(np.float16))


def check(g, inputs, flags=0, names=None):
    desc = g.build()
    metas = [g.tensor_meta(t) for t in g.output_ids()]
    h = pn.Graph(desc, 0, flags)
    outs = run_graph(h, inputs)
    return check_against_oracle(desc, inputs, outs, metas, names)


UNARY = ["neg", "abs", "exp", "log", "sqrt", "rsqrt", "recip", "tanh", "sigmoid", "silu", "gelu_tanh",
         "gelu_erf", "relu", "square", "erf"]


@pytest.mark.parametrize("mode", list(MODES))
@pytest.mark.parametrize("op", UNARY)
def test_unary(op, mode):
    shape = (7, 1001)                                   # ragged: element-wise memory path
    x = rnd(shape, 1, 2.0)
    if op in ("log", "sqrt", "rsqrt"):
        x = np.abs(x) + np.float32(0.05)
    if op == "recip":
        x = np.where(np.abs(x) < 0.05, np.float32(0.5), x)
    x[0, :6] = [0.0, -0.0, 30.0, -30.0, 1e-6, -1e-6] if op not in ("log", "sqrt", "rsqrt", "recip") else x[0, :6]
    g = GraphBuilder(); xi = g.input(D.F32, shape)
    g.mark_output(g.op(op, [xi], D.F32, shape))
    check(g, [x], MODES[mode])


@pytest.mark.parametrize("mode", list(MODES))
def test_unary_on_vector_path_with_special_values(mode):
    shape = (3, 1024)
    x = rnd(shape, 2, 3.0)
    x[0, :8] = [np.inf, -np.inf, np.nan, 0.0, 88.0, -88.0, 100.0, -100.0]
    for op in ("exp", "sigmoid", "silu", "gelu_tanh", "relu", "tanh", "abs"):
        g = GraphBuilder(); xi = g.input(D.F32, shape)
        g.mark_output(g.op(op, [xi], D.F32, shape))
        check(g, [x], MODES[mode])


BINARY = ["add", "sub", "mul", "div", "max", "min", "gt", "ge", "lt", "le", "eq", "ne"]


@pytest.mark.parametrize("mode", list(MODES))
@pytest.mark.parametrize("op", BINARY)
def test_binary_with_broadcast_and_immediates(op, mode):
    a = rnd((5, 3, 40), 3); b = rnd((3, 1), 4); c = rnd((40,), 5)
    a[0, 0, :4] = [1.0, np.nan, np.inf, 2.0]; c[:4] = [1.0, 1.0, np.inf, np.nan]
    cmp_op = op in ("gt", "ge", "lt", "le", "eq", "ne")
    odt = D.BOOL if cmp_op else D.F32
    g = GraphBuilder()
    ai = g.input(D.F32, a.shape); bi = g.input(D.F32, b.shape); ci = g.input(D.F32, c.shape)
    g.mark_output(g.op(op, [ai, bi], odt, (5, 3, 40)))           # column vector against a full tensor
    g.mark_output(g.op(op, [ci, ai], odt, (5, 3, 40)))           # row vector first: operand order matters
    g.mark_output(g.op(op, [ai, Imm(0.5)], odt, (5, 3, 40)))
    g.mark_output(g.op(op, [Imm(0.5), ai], odt, (5, 3, 40)))
    check(g, [a, b, c], MODES[mode])


@pytest.mark.parametrize("mode", list(MODES))
def test_ternary_and_casts(mode):
    shape = (4, 264)
    a = rnd(shape, 6); b = rnd(shape, 7)
    m8 = (np.random.default_rng(8).integers(-1, 2, shape)).astype(np.int8)
    mb = (np.random.default_rng(9).integers(0, 2, (264,))).astype(np.uint8)
    i32 = np.random.default_rng(10).integers(-1000, 1000, shape).astype(np.int32)
    g = GraphBuilder()
    ai = g.input(D.F32, shape); bi = g.input(D.F32, shape); mi = g.input(D.I8, shape)
    bb = g.input(D.BOOL, (264,)); ii = g.input(D.I32, shape)
    g.mark_output(g.op("where", [mi, ai, bi], D.F32, shape))                   # int8 mask, tested as bytes
    g.mark_output(g.op("where", [bb, ai, Imm(-math.inf)], D.F32, shape))       # broadcast bool mask
    gt = g.op("gt", [ai, bi], D.BOOL, shape)
    g.mark_output(g.op("where", [gt, ai, bi], D.F32, shape))                   # computed condition
    g.mark_output(g.op("clamp", [ai, Imm(-0.5), Imm(0.75)], D.F32, shape))
    g.mark_output(g.op("fma", [ai, bi, Imm(2.0)], D.F32, shape))
    check(g, [a * 3, b, m8, mb, i32], MODES[mode])
    g = GraphBuilder()
    ai = g.input(D.F32, shape); bi = g.input(D.F32, shape); ii = g.input(D.I32, shape)
    gt = g.op("gt", [ai, bi], D.BOOL, shape)
    g.mark_output(g.op("cast", [ai, ], D.I32, shape))                           # truncation toward zero
    g.mark_output(g.op("cast", [ai], D.BOOL, shape))
    g.mark_output(g.op("cast", [gt], D.I8, shape))
    f = g.op("cast", [ii], D.F32, shape)
    g.mark_output(g.op("mul", [f, Imm(0.25)], D.F32, shape))
    g.mark_output(g.op("cast", [ai], D.BF16, shape))
    g.mark_output(g.op("cast", [ai], D.F16, shape))
    check(g, [a * 3, b, i32], MODES[mode])


@pytest.mark.parametrize("mode", list(MODES))
def test_declared_narrow_intermediate_is_rounded(mode):
    shape = (3, 512)
    a = rnd(shape, 11, 4.0)
    g = GraphBuilder(); ai = g.input(D.F32, shape)
    nb = g.op("cast", [ai], D.BF16, shape)
    d = g.op("sub", [nb, ai], D.F32, shape)          # the rounding error itself: exact in fp32
    g.mark_output(d)
    nh = g.op("mul", [ai, Imm(1.0)], D.F16, shape)   # any node may declare a narrow type
    g.mark_output(g.op("sub", [nh, ai], D.F32, shape))
    check(g, [a], MODES[mode])


REDUCTIONS = [("sum", D.F32), ("mean", D.F32), ("var", D.F32), ("amax", D.F32), ("amin", D.F32),
              ("argmax", D.I64), ("argmin", D.I32), ("logsumexp", D.F32)]
ROW_LENGTHS = [1, 2, 7, 8, 33, 255, 256, 1000, 1024, 1025, 4096, 4104, 20000]


@pytest.mark.parametrize("mode", list(MODES))
@pytest.mark.parametrize("n", ROW_LENGTHS)
def test_all_reductions_over_row_lengths(n, mode):
    rows = 5 if n < 5000 else 3
    x = np.round(rnd((rows, n), 12 + n, 2.0) * 4) / 4            # quarter steps: many exact ties
    x = x.astype(np.float32)
    for half in (REDUCTIONS[:4], REDUCTIONS[4:]):             # a stage takes four reductions
        g = GraphBuilder(); xi = g.input(D.F32, (rows, n))
        for k, (op, dt) in enumerate(half):
            dims = (rows,) if k % 2 == 0 else (rows, 1)          # dropped and kept last dim
            g.mark_output(g.op(op, [xi], dt, dims, attr=[1 if (op == "var" and n > 1) else 0, 0]))
        check(g, [x], MODES[mode])


@pytest.mark.parametrize("force", [0, pn.FLAG_FORCE_WARP, pn.FLAG_FORCE_BLOCK, pn.FLAG_FORCE_CLUSTER,
                                   pn.FLAG_FORCE_BLOCK | pn.FLAG_FORCE_MULTICHUNK, pn.FLAG_FORCE_SCALAR,
                                   pn.FLAG_PREFETCH, pn.FLAG_PREFETCH | pn.FLAG_FORCE_CLUSTER, pn.FLAG_FORCE_SPLIT])
def test_reductions_with_nan_and_infinities_in_every_family(force):
    x = rnd((6, 2048), 13, 2.0)
    x[0, 100] = np.nan; x[0, 1500] = np.nan              # first NaN wins argmax / argmin; sums are NaN
    x[1, :] = -np.inf                                    # lse = -inf, softmax NaN
    x[2, 7] = np.inf                                     # lse = +inf
    x[3, :] = 1.5                                        # all tied: index 0
    x[4, 2047] = 50.0; x[4, 3] = 50.0
    for half in (REDUCTIONS[:4], REDUCTIONS[4:]):
        g = GraphBuilder(); xi = g.input(D.F32, x.shape)
        for op, dt in half:
            g.mark_output(g.op(op, [xi], dt, (6,)))
        check(g, [x], force)
    for op in ("softmax", "log_softmax"):
        g = GraphBuilder(); xi = g.input(D.F32, x.shape)
        g.mark_output(g.op(op, [xi], D.F32, x.shape))
        check(g, [x], force)


@pytest.mark.parametrize("mode", list(MODES))
@pytest.mark.parametrize("dtype", [D.F32, D.BF16, D.F16])
@pytest.mark.parametrize("n", [8, 200, 512, 1000, 2048, 4096, 9000])
def test_composites(n, dtype, mode):
    rows = 6
    x = rnd((rows, n), 14 + n, 1.5, dtype); ga = rnd((n,), 15, 0.3) + 1; be = rnd((n,), 16, 0.1)
    for op in ("softmax", "log_softmax", "layer_norm", "rms_norm"):
        g = GraphBuilder(); xi = g.input(dtype, (rows, n)); gi = g.input(D.F32, (n,)); bi = g.input(D.F32, (n,))
        xf = g.op("cast", [xi], D.F32, (rows, n)) if dtype != D.F32 else xi
        if op == "layer_norm":
            y, mean, rstd = g.node(op, [xf, gi, bi], [D.F32] * 3, [(rows, n), (rows, 1), (rows,)], extra_imm=[1e-5])
            g.mark_output(mean); g.mark_output(rstd)
        elif op == "rms_norm":
            y = g.op(op, [xf, gi], D.F32, (rows, n), extra_imm=[1e-6])
        else:
            y = g.op(op, [xf], D.F32, (rows, n))
        g.mark_output(g.op("cast", [y], dtype, (rows, n)) if dtype != D.F32 else y)
        check(g, [x, ga.astype(np.float32), be.astype(np.float32)], MODES[mode])


@pytest.mark.parametrize("mode", list(MODES))
def test_user_written_two_stage_softmax_and_scalar_arithmetic(mode):
    """Reductions feeding later stages by hand: m = amax(x); e = exp(x - m); y = e / sum(e),
    with per-row scalar arithmetic in between, and the clamped divide of the paper's masked
    mean pooling kernel (Appendix H, case 2) on per-row values."""
    rows, n = 9, 1536
    x = rnd((rows, n), 17, 2.0); msk = (np.random.default_rng(18).random((rows, n)) < 0.3).astype(np.float32)
    msk[4, :] = 0                                        # empty mask row: the clamp decides
    g = GraphBuilder(); xi = g.input(D.F32, (rows, n)); mi = g.input(D.F32, (rows, n))
    m = g.op("amax", [xi], D.F32, (rows, 1))
    e = g.op("exp", [g.op("sub", [xi, m], D.F32, (rows, n))], D.F32, (rows, n))
    s = g.op("sum", [e], D.F32, (rows, 1))
    g.mark_output(g.op("div", [e, s], D.F32, (rows, n)))
    hm = g.op("mul", [xi, mi], D.F32, (rows, n))
    num = g.op("sum", [hm], D.F32, (rows, 1)); den = g.op("sum", [mi], D.F32, (rows, 1))
    g.mark_output(g.op("div", [num, g.op("clamp", [den, Imm(1e-9), Imm(math.inf)], D.F32, (rows, 1))], D.F32, (rows, 1)))
    idx = g.op("argmax", [xi], D.I64, (rows, 1))
    g.mark_output(g.op("mul", [g.op("cast", [idx], D.F32, (rows, 1)), Imm(0.5)], D.F32, (rows, 1)))
    check(g, [x, msk], MODES[mode])


def test_rank4_broadcast_patterns():
    a = rnd((2, 3, 4, 64), 19); b = rnd((3, 1, 64), 20); c = rnd((2, 1, 4, 1), 21); d = rnd((1,), 22)
    g = GraphBuilder()
    ai = g.input(D.F32, a.shape); bi = g.input(D.F32, b.shape); ci = g.input(D.F32, c.shape); di = g.input(D.F32, d.shape)
    t = g.op("add", [g.op("mul", [ai, bi], D.F32, a.shape), ci], D.F32, a.shape)
    t = g.op("sub", [t, di], D.F32, a.shape)
    g.mark_output(t)
    g.mark_output(g.op("softmax", [t], D.F32, a.shape))
    g.mark_output(g.op("sum", [t], D.F32, (2, 3, 4)))
    for flags in (0, pn.FLAG_INTERPRET, pn.FLAG_UNFUSED):
        check(g, [a, b, c, d], flags)


def test_edge_shapes():
    for shape in [(1,), (1, 1), (1, 8), (3, 1), (4097,), (2, 0, 8)]:
        x = rnd(shape, 23)
        g = GraphBuilder(); xi = g.input(D.F32, shape)
        g.mark_output(g.op("gelu_tanh", [xi], D.F32, shape))
        if 0 not in shape:
            g.mark_output(g.op("sum", [xi], D.F32, shape[:-1]))
        h = pn.Graph(g.build(), 0, 0)
        outs = run_graph(h, [x])
        if 0 not in shape:
            check(g, [x], 0)
        else:
            assert all(o.size == 0 for o in outs)


def test_run_errors_leave_the_device_alone():
    import torch
    w = C.c1(M=4, N=64)
    h = pn.Graph(w.desc, 0, 0)
    buf = torch.zeros(4 * 64 * 4 + 64, dtype=torch.uint8, device="cuda")
    good = [buf.data_ptr()] * 4
    with pytest.raises(pn.PnError) as e:
        h.run(good[:3], [buf.data_ptr()])
    assert e.value.status == -7                                   # count
    with pytest.raises(pn.PnError) as e:
        h.run(good, [buf.data_ptr()])
    assert e.value.status == -1                                   # output overlaps an input
    out = torch.zeros(4 * 64 * 4 + 64, dtype=torch.uint8, device="cuda")
    with pytest.raises(pn.PnError) as e:
        h.run([good[0] + 4] + good[1:], [out.data_ptr()])
    assert e.value.status == -6                                   # alignment
    with pytest.raises(pn.PnError) as e:
        h.run([0] + good[1:], [out.data_ptr()])
    assert e.value.status == -1                                   # null pointer
    torch.cuda.synchronize()


def test_results_repeat_bit_for_bit():
    w = C.c5(M=64, N=14336)
    h = pn.Graph(w.desc, 0, 0)
    a = run_graph(h, w.inputs); b = run_graph(h, w.inputs)
    assert all(np.array_equal(x, y) for x, y in zip(a, b))
    w = C.c4(M=4, N=262144)
    h = pn.Graph(w.desc, 0, 0)
    a = run_graph(h, w.inputs); b = run_graph(h, w.inputs)
    assert all(np.array_equal(x, y) for x, y in zip(a, b))


@pytest.mark.parametrize("dtype", [D.F32, D.BF16])
@pytest.mark.parametrize("rows,n", [(1, 8), (5, 16), (37, 24), (64, 40), (3, 64), (1001, 96), (130, 128), (7, 32)])
def test_short_rows_that_share_a_warp(rows, n, dtype):
    """Rows of at most 16 (8) vector groups are owned by half (quarter) warps; row counts that leave
    some of a warp's teams without a row in the last round; every kind of reduction, an index
    result, a composite with a full-shape output."""
    x = np.round(rnd((rows, n), 40 + rows + n, 2.0) * 4) / 4
    x = x.astype(np.float32)
    xs = x if dtype == D.F32 else C.to_bf16_bits(x)
    gamma = rnd((n,), 41); beta = rnd((n,), 42)
    g = GraphBuilder(); xi = g.input(dtype, (rows, n)); gi = g.input(D.F32, (n,)); bi = g.input(D.F32, (n,))
    xf = g.op("cast", [xi], D.F32, (rows, n)) if dtype != D.F32 else xi
    y, mean, rstd = g.node("layer_norm", [xf, gi, bi], [D.F32, D.F32, D.F32], [(rows, n), (rows,), (rows,)], extra_imm=[1e-5])
    g.mark_output(g.op("cast", [y], dtype, (rows, n)) if dtype != D.F32 else y)
    g.mark_output(mean); g.mark_output(rstd)
    g.mark_output(g.op("argmax", [xf], D.I64, (rows,)))
    g.mark_output(g.op("sum", [xf], D.F32, (rows, 1)))
    for flags in (pn.FLAG_PREFETCH, pn.FLAG_NO_HOIST, pn.FLAG_BOUNDS):     # loads issued a tile ahead, nothing hoisted, checked
        hf = pn.Graph(g.build(), 0, flags)
        check_against_oracle(g.build(), [xs, gamma, beta], run_graph(hf, [xs, gamma, beta]), [g.tensor_meta(t) for t in g.output_ids()])
        if flags == pn.FLAG_BOUNDS:
            assert hf.bounds_status == 0
    h = pn.Graph(g.build(), 0, 0)
    k = h.kernel_info[0]
    assert pn.FAMILY_NAMES[k["family"]] == "warp-per-row"
    outs = run_graph(h, [xs, gamma, beta])
    check_against_oracle(g.build(), [xs, gamma, beta], outs, [g.tensor_meta(t) for t in g.output_ids()])
    again = run_graph(h, [xs, gamma, beta])
    assert all(np.array_equal(a, b, equal_nan=True) for a, b in zip(outs, again))
    g = GraphBuilder(); xi = g.input(dtype, (rows, n))
    xf = g.op("cast", [xi], D.F32, (rows, n)) if dtype != D.F32 else xi
    sm = g.op("softmax", [xf], D.F32, (rows, n))
    g.mark_output(g.op("cast", [sm], dtype, (rows, n)) if dtype != D.F32 else sm)
    g.mark_output(g.op("logsumexp", [xf], D.F32, (rows,)))
    check(g, [xs])
