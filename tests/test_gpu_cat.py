"""Concatenations of several operands against the CPU oracle, through the C ABI.  A cat is not
computed: every operand is stored straight into its block of the result, by the kernel that
produces it (an output-address remap, the mirror of the index-remapped loads); a result that is
read again is read by a later launch."""
import numpy as np
import pytest

import paper_2605_29357_b200 as pn
from pn_workloads import configs as C
from pn_workloads import descriptor as D
from pn_workloads.descriptor import GraphBuilder, Imm

from gpu_util import check_against_oracle, run_graph

pytestmark = pytest.mark.gpu


def rnd(shape, seed, dtype=D.F32):
    x = np.random.default_rng(seed).standard_normal(shape).astype(np.float32)
    return x if dtype == D.F32 else (C.to_bf16_bits(x) if dtype == D.BF16 else x.astype(np.float16))


def check(g, inputs, flags=0):
    desc = g.build()
    h = pn.Graph(desc, 0, flags | pn.FLAG_BOUNDS)
    outs = run_graph(h, inputs)
    check_against_oracle(desc, inputs, outs, [g.tensor_meta(t) for t in g.output_ids()])
    assert h.bounds_status == 0
    return h


@pytest.mark.parametrize("flags", [0, pn.FLAG_UNFUSED, pn.FLAG_INTERPRET, pn.FLAG_FORCE_SCALAR])
@pytest.mark.parametrize("dtype", [D.F32, D.BF16])
@pytest.mark.parametrize("shapes,dim", [([(4, 6, 8), (4, 3, 8)], 1), ([(5, 16), (7, 16), (1, 16)], 0), ([(5, 16), (5, 8)], 1),
                                        ([(5, 7), (5, 9), (5, 1), (5, 4)], 1), ([(2, 3, 4, 8), (2, 3, 2, 8)], 2), ([(3, 1000), (3, 24)], 1)])
def test_cat_of_graph_inputs(shapes, dim, dtype, flags):
    g = GraphBuilder()
    ins = [g.input(dtype, s) for s in shapes]
    out = list(shapes[0]); out[dim] = sum(s[dim] for s in shapes)
    g.mark_output(g.op("cat", ins, dtype, tuple(out), attr=[dim, 0]))
    h = check(g, [rnd(s, 10 + k, dtype) for k, s in enumerate(shapes)], flags)
    assert h.n_nodes == 1 and h.n_kernels == len(shapes)         # one store per operand, nothing else


def test_computed_operands_are_stored_by_the_kernels_that_make_them():
    # same iteration shape: one kernel writes both blocks
    g = GraphBuilder(); a = g.input(D.F32, (37, 200))
    ta = g.op("tanh", [a], D.F32, (37, 200)); tb = g.op("sigmoid", [a], D.F32, (37, 200))
    g.mark_output(g.op("cat", [ta, tb], D.F32, (37, 400), attr=[1, 0]))
    g.mark_output(g.op("cat", [tb, ta, tb], D.F32, (111, 200), attr=[0, 0]))   # an operand used twice, and by two cats
    g.mark_output(ta)                                                          # ... and a graph output itself
    assert check(g, [rnd((37, 200), 1)]).n_kernels == 1
    # different shapes: one launch per shape; then the result is read again
    g = GraphBuilder(); a = g.input(D.BF16, (9, 512)); b = g.input(D.BF16, (9, 256))
    fa = g.op("gelu_tanh", [g.op("cast", [a], D.F32, (9, 512))], D.F32, (9, 512))
    fb = g.op("mul", [g.op("cast", [b], D.F32, (9, 256)), Imm(0.5)], D.F32, (9, 256))
    c = g.op("cat", [fa, fb], D.F32, (9, 768), attr=[1, 0])
    y = g.node("layer_norm", [c], [D.F32], [(9, 768)], extra_imm=[1e-5])[0]
    g.mark_output(g.op("cast", [y], D.BF16, (9, 768)))
    h = check(g, [rnd((9, 512), 2, D.BF16), rnd((9, 256), 3, D.BF16)])
    assert h.n_kernels == 3 and h.workspace_bytes >= 9 * 768 * 4
    # per-row results side by side
    g = GraphBuilder(); a = g.input(D.F32, (12, 300))
    m = g.op("mean", [a], D.F32, (12, 1)); v = g.op("amax", [a], D.F32, (12, 1))
    g.mark_output(g.op("cat", [m, v], D.F32, (12, 2), attr=[1, 0]))
    check(g, [rnd((12, 300), 4)])


def test_a_roll_written_as_slices_and_a_cat_equals_the_roll():
    """The decomposition a graph compiler makes of a roll (Section 4.4, first case study): the last
    `shift` rows first, then the rest."""
    S, n, shift = 21, 96, 3
    x = rnd((S, S, n), 5, D.BF16)
    g = GraphBuilder(); xi = g.input(D.BF16, (S, S, n))
    tail = g.op("slice", [xi], D.BF16, (shift, S, n), attr=[0, S - shift])
    head = g.op("slice", [xi], D.BF16, (S - shift, S, n), attr=[0, 0])
    g.mark_output(g.op("cat", [tail, head], D.BF16, (S, S, n), attr=[0, 0]))
    g.mark_output(g.op("roll", [xi], D.BF16, (S, S, n), attr=[0, shift]))
    desc = g.build()
    h = pn.Graph(desc, 0, 0)
    outs = run_graph(h, [x])
    assert np.array_equal(outs[0], outs[1])                       # both spellings of the same re-indexing
    check_against_oracle(desc, [x], outs, [g.tensor_meta(t) for t in g.output_ids()])
