"""The split-row family (few long rows reduced by independent blocks over slices of the rows, which
meet per row through partials in the handle's workspace) against the CPU oracle, through the C ABI: every reduction over ragged and
exact row lengths, special values, a pointwise chain before and scalar arithmetic after the
reductions, checked accessors, and launch after launch of one handle (the arrival counters must be
back at zero each time) with bit-identical results whichever block arrives last."""
import numpy as np
import pytest

import paper_2605_29357_b200 as pn
from pn_workloads import configs as C
from pn_workloads import descriptor as D
from pn_workloads.descriptor import GraphBuilder, Imm

from gpu_util import check_against_oracle, run_graph

pytestmark = pytest.mark.gpu

SPLIT = pn.FLAG_FORCE_SPLIT
REDUCTIONS = [("sum", D.F32), ("mean", D.F32), ("var", D.F32), ("amax", D.F32), ("amin", D.F32),
              ("argmax", D.I64), ("argmin", D.I32), ("logsumexp", D.F32)]


def rnd(shape, seed, scale=1.0, dtype=D.F32):
    x = (np.random.default_rng(seed).standard_normal(shape) * scale).astype(np.float32)
    return x if dtype == D.F32 else (C.to_bf16_bits(x) if dtype == D.BF16 else x.astype(np.float16))


def check(g, inputs, flags, want_family=5):
    desc = g.build()
    metas = [g.tensor_meta(t) for t in g.output_ids()]
    h = pn.Graph(desc, 0, flags)
    assert h.n_kernels == 1 and h.kernel_info[0]["family"] == want_family, h.kernel_info
    outs = run_graph(h, inputs)
    check_against_oracle(desc, inputs, outs, metas)
    return h, outs


@pytest.mark.parametrize("how", [0, pn.tune(cluster=2), pn.tune(groups=1, block=64)])   # the lowering's slices; two tiles per slice; many small slices
@pytest.mark.parametrize("dtype", [D.F32, D.BF16, D.F16])
@pytest.mark.parametrize("rows,n", [(1, 1024), (3, 4096), (5, 4104), (2, 20000), (7, 66000), (1, 300000), (300, 8192)])
def test_all_reductions_split_over_blocks(rows, n, dtype, how):
    x = np.round(rnd((rows, n), 3 * n + rows, 2.0) * 4) / 4          # quarter steps: many exact ties
    x = x.astype(np.float32)
    x = x if dtype == D.F32 else (C.to_bf16_bits(x) if dtype == D.BF16 else x.astype(np.float16))
    for half in (REDUCTIONS[:4], REDUCTIONS[4:]):
        g = GraphBuilder(); xi = g.input(dtype, (rows, n))
        xf = xi if dtype == D.F32 else g.op("cast", [xi], D.F32, (rows, n))
        for k, (op, dt) in enumerate(half):
            dims = (rows,) if k % 2 == 0 else (rows, 1)
            g.mark_output(g.op(op, [xf], dt, dims, attr=[1 if op == "var" else 0, 0]))
        h, _ = check(g, [x], SPLIT | how)
        assert h.workspace_bytes > 0


def test_special_values_meet_across_slices():
    x = rnd((6, 40000), 13, 2.0)
    x[0, 100] = np.nan; x[0, 39000] = np.nan             # first NaN wins argmax / argmin; sums are NaN
    x[1, :] = -np.inf                                    # lse = -inf
    x[2, 35000] = np.inf                                 # lse = +inf
    x[3, :] = 1.5                                        # all tied: index 0
    x[4, 39999] = 50.0; x[4, 3] = 50.0                   # ties in the first and the last slice
    x[5, 20000] = -50.0; x[5, 20001] = -50.0
    for half in (REDUCTIONS[:4], REDUCTIONS[4:]):
        g = GraphBuilder(); xi = g.input(D.F32, x.shape)
        for op, dt in half:
            g.mark_output(g.op(op, [xi], dt, (6,)))
        check(g, [x], SPLIT)


def test_pointwise_chain_before_and_scalar_arithmetic_after():
    rows, n = 4, 50000
    x, w = rnd((rows, n), 1), rnd((n,), 2)
    r = (np.random.default_rng(3).uniform(0.5, 2.0, (rows, 1))).astype(np.float32)
    g = GraphBuilder()
    xi, wi, ri = g.input(D.F32, (rows, n)), g.input(D.F32, (n,)), g.input(D.F32, (rows, 1))
    t = g.op("mul", [g.op("fma", [xi, wi, Imm(0.25)], D.F32, (rows, n)), ri], D.F32, (rows, n))
    s = g.op("sum", [t], D.F32, (rows, 1))
    m = g.op("amax", [t], D.F32, (rows, 1))
    lse = g.op("logsumexp", [t], D.F32, (rows, 1))
    g.mark_output(g.op("sub", [lse, m], D.F32, (rows, 1)))            # per-row scalar arithmetic on reduced values
    g.mark_output(g.op("div", [s, g.op("add", [m, Imm(100.0)], D.F32, (rows, 1))], D.F32, (rows, 1)))
    g.mark_output(g.op("argmax", [t], D.I64, (rows,)))
    check(g, [x, w, r], SPLIT)


def test_launch_after_launch_gives_the_same_bits_and_the_default_choice_for_long_rows_is_split():
    w = C.c4(M=6, N=262144)
    h = pn.Graph(w.desc, 0, 0)                          # no forcing: few long rows, a single stage
    assert h.kernel_info[0]["family"] == 5
    first = run_graph(h, w.inputs)
    check_against_oracle(w.desc, w.inputs, first, w.output_meta, w.output_names)
    for _ in range(5):
        again = run_graph(h, w.inputs)
        assert all(np.array_equal(a, b) for a, b in zip(first, again))
    # a graph that needs the row again after its reduction cannot be split: it stays with clusters
    x = rnd((4, 100000), 5)
    g = GraphBuilder(); xi = g.input(D.F32, x.shape)
    g.mark_output(g.op("softmax", [xi], D.F32, x.shape))
    hs = pn.Graph(g.build(), 0, 0)
    assert hs.kernel_info[0]["family"] == 3


def test_split_rows_under_checked_accessors():
    x = rnd((3, 33000), 8)
    g = GraphBuilder(); xi = g.input(D.F32, x.shape)
    g.mark_output(g.op("logsumexp", [xi], D.F32, (3,)))
    g.mark_output(g.op("argmin", [xi], D.I64, (3,)))
    h, _ = check(g, [x], SPLIT | pn.FLAG_BOUNDS)
    assert h.bounds_status == 0
