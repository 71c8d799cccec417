"""GPU parity of the reductions over a leading dimension (the masked-mean-pooling shape of the
paper's second case study, Section 4.4 / Appendix H case 2) against the CPU oracle, through the
C ABI: each reduction alone over ranks, dimensions and ragged sizes; graphs with values before
and after the reduction; the pooling subgraph at reduced and full size, fused and unfused, on
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

FORCES = {
    "default": 0,
    "interpret": pn.FLAG_INTERPRET,
    "unfused": pn.FLAG_UNFUSED,
    "interpret_unfused": pn.FLAG_INTERPRET | pn.FLAG_UNFUSED,
    "scalar": pn.FLAG_FORCE_SCALAR,
    "block64": pn.tune(block=64),
    "block1024": pn.tune(block=1024),
    "groups2": pn.tune(groups=2),
}


def _quarters(shape, seed, dtype=D.F32):
    """Multiples of 1/4 of modest size: fp32 sums of thousands of them are exact, so the
    comparison judges the indexing and the combine order, not rounding."""
    x = np.round(np.random.default_rng(seed).standard_normal(shape) * 8) / 4
    x = x.astype(np.float32)
    return x if dtype == D.F32 else (C.to_bf16_bits(x) if dtype == D.BF16 else x.astype(np.float16))


def _run(g, inputs, flags=0):
    desc = g.build()
    gr = pn.Graph(desc, 0, flags)
    outs = run_graph(gr, inputs)
    check_against_oracle(desc, inputs, outs, [g.tensor_meta(t) for t in g.output_ids()])
    return gr, outs


@pytest.mark.parametrize("force", list(FORCES))
@pytest.mark.parametrize("kw", [dict(B=3, S=37, Dh=200), dict(B=2, S=300, Dh=203), dict(B=5, S=1, Dh=64),
                                dict(B=1, S=70, Dh=1032, dense_mask=True, mask_dtype=D.F32),
                                dict(B=4, S=33, Dh=96, dense_mask=True, mask_dtype=D.I8),
                                dict(B=2, S=19, Dh=520, dtype=D.F32, mask_dtype=D.BOOL)])
def test_masked_mean_pooling_small(kw, force):
    w = C.n2(**kw)
    g = pn.Graph(w.desc, 0, FORCES[force])
    outs = run_graph(g, w.inputs)
    check_against_oracle(w.desc, w.inputs, outs, w.output_meta, w.output_names)
    if "unfused" not in force:
        assert g.n_kernels == 1 and pn.FAMILY_NAMES[g.kernel_info[0]["family"]] == "column-reduce"
    else:
        assert g.n_kernels == w.n_nodes == 7           # the paper's 7 -> 1


def test_masked_mean_pooling_special_rows():
    """Nothing masked, everything masked (0 / 1e-9 = 0) and a single position kept (that row of
    hidden, bit for bit: Table 2 reports a maximum difference of 0.0 for this kernel)."""
    w = C.n2(B=4, S=50, Dh=256)
    mask, hidden = [a.copy() for a in w.inputs]
    mask[0, :, 0] = 1
    mask[1, :, 0] = 0
    mask[2, :, 0] = 0; mask[2, 41, 0] = 1
    g = pn.Graph(w.desc, 0, 0)
    outs = run_graph(g, [mask, hidden])
    check_against_oracle(w.desc, [mask, hidden], outs, w.output_meta)
    assert np.array_equal(outs[0][1], np.zeros(256, np.float32))
    assert np.array_equal(outs[0][2], E.widen(hidden[2, 41], D.BF16).astype(np.float32))


def test_masked_mean_pooling_full_size():
    w = C.n2()
    g = pn.Graph(w.desc, 0, 0)
    assert g.n_kernels == 1 and g.compulsory_bytes == w.compulsory_bytes
    outs = run_graph(g, w.inputs)
    refs = []
    for lo in range(0, 256, 32):                        # batches are independent: bounded fp64 intermediates
        sub = C.n2(B=32)
        refs.append(E.evaluate(sub.desc, [w.inputs[0][lo:lo + 32], w.inputs[1][lo:lo + 32]])[0])
    check_against_oracle(w.desc, w.inputs, outs, w.output_meta, w.output_names, ref=[np.concatenate(refs, axis=0)])
    # run to run the result repeats bit for bit (fixed combine order)
    again = run_graph(g, w.inputs)
    assert np.array_equal(outs[0], again[0])


SHAPES = [((5, 40), 0), ((1000, 8), 0), ((4, 6, 24), 1), ((4, 6, 24), 0), ((2, 3, 4, 16), 2), ((2, 3, 4, 16), 1),
          ((3, 2500, 7), 1), ((2, 129, 1), 1), ((1, 64, 300), 1), ((7, 1, 33), 1)]


@pytest.mark.parametrize("flags", [0, pn.FLAG_INTERPRET, pn.FLAG_FORCE_SCALAR])
@pytest.mark.parametrize("shape,dim", SHAPES)
def test_each_reduction_over_a_leading_dimension(shape, dim, flags):
    x = _quarters(shape, 30 + dim + len(shape))
    drop = shape[:dim] + shape[dim + 1:]
    keep = shape[:dim] + (1,) + shape[dim + 1:]
    # the interpreter's kernels have room for two accumulators: two graphs of two each
    for ops in (("sum_dim", "mean_dim", "amax_dim"), ("sum_dim", "amin_dim")):
        g = GraphBuilder(); xi = g.input(D.F32, shape)
        for k, op in enumerate(ops):
            g.mark_output(g.op(op, [xi], D.F32, drop if k % 2 == 0 else keep, attr=[dim, 0]))
        gr, outs = _run(g, [x], flags)
        assert gr.n_kernels == 1
        assert np.array_equal(outs[0], x.astype(np.float64).sum(axis=dim).astype(np.float32))   # exact sums


@pytest.mark.parametrize("dtype", [D.BF16, D.F16, D.I32])
def test_storage_types_and_special_values(dtype):
    shape = (3, 45, 136)
    if dtype == D.I32:
        x = np.random.default_rng(5).integers(-500, 500, size=shape, dtype=np.int32)
    else:
        x = _quarters(shape, 6, dtype)
    g = GraphBuilder(); xi = g.input(dtype, shape)
    xf = g.op("cast", [xi], D.F32, shape)
    g.mark_output(g.op("sum_dim", [xf], D.F32, (3, 136), attr=[1, 0]))
    g.mark_output(g.op("cast", [g.op("amax_dim", [xf], D.F32, (3, 136), attr=[1, 0])], dtype if dtype != D.I32 else D.I32, (3, 136)))
    _run(g, [x])
    # NaN and infinities travel through sums and extremes as IEEE says
    y = _quarters((2, 30, 64), 7)
    y[0, 3, 5] = np.nan; y[0, 4, 6] = np.inf; y[1, 7, 6] = -np.inf; y[1, 8, 9] = np.inf; y[1, 9, 9] = -np.inf
    g = GraphBuilder(); yi = g.input(D.F32, y.shape)
    for op in ("sum_dim", "amax_dim", "amin_dim", "mean_dim"):
        g.mark_output(g.op(op, [yi], D.F32, (2, 64), attr=[1, 0]))
    _run(g, [y], 0)
    for pair in (("sum_dim", "amax_dim"), ("mean_dim", "amin_dim")):
        g = GraphBuilder(); yi = g.input(D.F32, y.shape)
        for op in pair:
            g.mark_output(g.op(op, [yi], D.F32, (2, 64), attr=[1, 0]))
        _run(g, [y], pn.FLAG_INTERPRET)


@pytest.mark.parametrize("flags", [0, pn.FLAG_INTERPRET, pn.FLAG_UNFUSED])
def test_values_before_and_after_the_reduction(flags):
    """A pointwise chain with broadcast operands before the reduction (one of its values is also
    an output), and an epilogue on the reduced values that reads graph inputs of the reduced
    shape."""
    B, S, Dh = 3, 29, 72
    x = _quarters((B, S, Dh), 8); w = _quarters((Dh,), 9); c = _quarters((B, 1, 1), 10)
    bias = _quarters((Dh,), 11); scale = _quarters((B, 1), 12)
    g = GraphBuilder()
    xi = g.input(D.F32, (B, S, Dh)); wi = g.input(D.F32, (Dh,)); ci = g.input(D.F32, (B, 1, 1))
    bi = g.input(D.F32, (Dh,)); si = g.input(D.F32, (B, 1))
    t = g.op("mul", [xi, wi], D.F32, (B, S, Dh))
    t = g.op("add", [t, ci], D.F32, (B, S, Dh))
    r = g.op("relu", [t], D.F32, (B, S, Dh))
    g.mark_output(r)                                                  # full-shape output of the walk
    tot = g.op("sum_dim", [r], D.F32, (B, 1, Dh), attr=[1, 0])       # reduced dimension kept as 1
    mx = g.op("amax_dim", [t], D.F32, (B, 1, Dh), attr=[1, 0])
    e = g.op("fma", [tot, Imm(0.5), mx], D.F32, (B, 1, Dh))
    g.mark_output(e)
    tot2 = g.op("sum_dim", [r], D.F32, (B, Dh), attr=[1, 0])         # the same reduction, dimension dropped
    f = g.op("mul", [g.op("add", [tot2, bi], D.F32, (B, Dh)), si], D.F32, (B, Dh))
    g.mark_output(g.op("cast", [f], D.BF16, (B, Dh)))
    gr, _ = _run(g, [x, w, c, bias, scale], flags)
    if not flags & pn.FLAG_UNFUSED:
        assert gr.n_kernels == 1


SLICED = {
    "default": 0,
    "two": pn.FLAG_FORCE_SPLIT,
    "three": pn.tune(cluster=3),
    "fifteen": pn.tune(cluster=15),
    "five_block64": pn.tune(cluster=5, block=64),
    "interpret_four": pn.FLAG_INTERPRET | pn.tune(cluster=4),
    "scalar_two": pn.FLAG_FORCE_SCALAR | pn.FLAG_FORCE_SPLIT,
    "bounds_seven": pn.FLAG_BOUNDS | pn.tune(cluster=7),
}


@pytest.mark.parametrize("force", list(SLICED))
@pytest.mark.parametrize("shape,dim", [((1, 5000, 40), 1), ((3, 2500, 7), 1), ((4099, 24), 0), ((2, 700, 3, 16), 1),
                                       ((2, 129, 1), 1), ((1, 64, 300), 1), ((1, 65536, 64), 1)])
def test_reduced_dimension_cut_into_slices(shape, dim, force):
    """Few columns under a long reduced dimension: blocks over slices of that dimension, combined by
    whichever block arrives last, in slice order.  Sums of quarters are exact in fp32, so they also
    judge that every step is folded exactly once; extremes judge the identity of empty slices."""
    flags = SLICED[force]
    x = _quarters(shape, 40 + dim + len(shape))
    drop = shape[:dim] + shape[dim + 1:]
    for ops in (("sum_dim", "amax_dim"), ("mean_dim", "amin_dim")):
        g = GraphBuilder(); xi = g.input(D.F32, shape)
        t = g.op("mul", [xi, Imm(0.5)], D.F32, shape)
        outs_t = [g.op(op, [t], D.F32, drop, attr=[dim, 0]) for op in ops]
        for o in outs_t:
            g.mark_output(o)
        g.mark_output(g.op("sub", outs_t, D.F32, drop))           # an epilogue on the combined values
        gr, outs = _run(g, [x], flags)
        info = gr.kernel_info[0]
        assert gr.n_kernels == 1 and pn.FAMILY_NAMES[info["family"]] == "column-reduce"
        R = shape[dim]
        if force != "default":
            want = {"two": 2, "three": 3, "fifteen": 15, "five_block64": 5, "interpret_four": 4, "scalar_two": 2, "bounds_seven": 7}[force]
            at_least = "two" in force                                 # PN_FLAG_FORCE_SPLIT: two or whatever the lowering wants
            assert at_least or 0 <= info["slices"] <= want
            if R >= 2048:
                assert (info["slices"] >= want if at_least else info["slices"] == want) and gr.workspace_bytes > 0
        elif shape == (1, 65536, 64):
            assert info["slices"] > 8                                 # the lowering's own choice fills the GPU
        if ops[0] == "sum_dim":
            assert np.array_equal(outs[0], (x.astype(np.float64) * 0.5).sum(axis=dim).astype(np.float32))
        again = run_graph(gr, [x])                                    # counters back at zero; same bits
        for a, b in zip(outs, again):
            assert np.array_equal(a, b)
        if flags & pn.FLAG_BOUNDS:
            assert gr.bounds_status == 0


def test_masked_mean_pooling_in_slices():
    """The pooling subgraph of the second case study with a small batch of long sequences, the
    sequence dimension cut into slices: the mask count (a reduction carried by one element of the
    tile) and the masked sum go through the same partials."""
    w = C.n2(B=2, S=4096, Dh=256)
    for flags in (0, pn.tune(cluster=6), pn.FLAG_INTERPRET | pn.FLAG_FORCE_SPLIT):
        g = pn.Graph(w.desc, 0, flags)
        outs = run_graph(g, w.inputs)
        check_against_oracle(w.desc, w.inputs, outs, w.output_meta, w.output_names)
        assert g.n_kernels == 1 and g.kernel_info[0]["slices"] >= 2
