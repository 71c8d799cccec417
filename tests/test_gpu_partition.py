"""Graphs that do not fit one kernel are cut into a few fused launches (the paper's fusible subgraphs
run to 35 operators and its classical ones to 62, Section 3.3): results against the CPU oracle,
through the C ABI, and the refusal that PN_FLAG_ONE_KERNEL asks for instead."""
import numpy as np
import pytest

import paper_2605_29357_b200 as pn
from pn_workloads import descriptor as D
from pn_workloads.descriptor import GraphBuilder, Imm

from gpu_util import check_against_oracle, run_graph

pytestmark = pytest.mark.gpu


def _check(g, inputs, flags=0):
    desc = g.build()
    h = pn.Graph(desc, 0, flags)
    outs = run_graph(h, inputs)
    check_against_oracle(desc, inputs, outs, [g.tensor_meta(t) for t in g.output_ids()])
    return h


def test_six_levels_of_reductions_and_two_softmaxes_become_a_few_launches():
    rows, n = 37, 1000
    x = (np.random.default_rng(1).standard_normal((rows, n)) * 0.5).astype(np.float32)
    g = GraphBuilder()
    xi = g.input(D.F32, (rows, n))
    a = g.op("softmax", [xi], D.F32, (rows, n))
    b = g.op("mul", [a, Imm(float(n))], D.F32, (rows, n))
    c = g.op("log_softmax", [b], D.F32, (rows, n))
    d = g.op("layer_norm", [c], D.F32, (rows, n), extra_imm=[1e-5])
    e = g.op("softmax", [d], D.F32, (rows, n))                # a second softmax, and the fifth level of reductions
    f = g.op("rms_norm", [g.op("add", [e, Imm(1.0)], D.F32, (rows, n))], D.F32, (rows, n), extra_imm=[1e-6])
    s = g.op("sum", [f], D.F32, (rows, 1))
    g.mark_output(g.op("div", [f, s], D.F32, (rows, n)))
    g.mark_output(g.op("argmax", [xi], D.I64, (rows,)))
    h = _check(g, [x])
    assert 2 <= h.n_kernels <= 4 and h.workspace_bytes >= rows * n * 4
    with pytest.raises(pn.PnError) as one:
        pn.Graph(g.build(), 0, pn.FLAG_ONE_KERNEL)
    assert one.value.status in (-3, -5)
    # launch after launch of the cut graph, and through a bound launch: the same bits
    desc = g.build()
    outs1 = run_graph(h, [x]); outs2 = run_graph(h, [x])
    assert all(np.array_equal(p, q) for p, q in zip(outs1, outs2))


def test_a_chain_of_62_operators_still_fits_one_kernel():
    rows, n = 5, 4100
    x = (np.random.default_rng(2).random((rows, n)) + 0.5).astype(np.float32)
    g = GraphBuilder()
    v = g.input(D.F32, (rows, n))
    ops = ["sqrt", "sigmoid", "tanh", "gelu_tanh", "silu", "abs", "relu", "erf"]
    for k in range(62):
        v = g.op(ops[k % len(ops)], [v], D.F32, (rows, n)) if k % 3 else g.op("fma", [v, Imm(0.75), Imm(0.5)], D.F32, (rows, n))
    g.mark_output(v)
    h = _check(g, [x])
    assert h.n_kernels == 1 and h.n_nodes == 62


def test_more_outputs_than_one_kernel_takes():
    rows, n = 9, 520
    x = (np.random.default_rng(3).random((rows, n)) + 0.5).astype(np.float32)
    g = GraphBuilder()
    v = g.input(D.F32, (rows, n))
    for k in range(14):                                        # 14 outputs + 1 input: beyond the 12 tensors of one kernel
        v = g.op("mul", [g.op("sqrt", [v], D.F32, (rows, n)), Imm(1.0 + 0.125 * k)], D.F32, (rows, n))
        g.mark_output(v)
    h = _check(g, [x])
    assert h.n_kernels >= 2


def test_combinations_that_one_kernel_refuses_run_as_two():
    rng = np.random.default_rng(4)
    x = rng.standard_normal((4, 6, 8)).astype(np.float32)
    # an index operator on a computed value: the value is materialised, the roll is a copy of its own
    g = GraphBuilder(); xi = g.input(D.F32, (4, 6, 8))
    y = g.op("tanh", [xi], D.F32, (4, 6, 8))
    g.mark_output(g.op("roll", [y], D.F32, (4, 6, 8), attr=[1, 2]))
    assert _check(g, [x]).n_kernels == 2
    # a value reduced over a leading dimension flows back into the tensor: a second pass, as a second launch
    g = GraphBuilder(); xi = g.input(D.F32, (4, 6, 8))
    s = g.op("mean_dim", [xi], D.F32, (4, 1, 8), attr=[1, 0])
    g.mark_output(g.op("sub", [xi, s], D.F32, (4, 6, 8)))
    assert _check(g, [x]).n_kernels == 2
    # reductions over two different dimensions
    g = GraphBuilder(); xi = g.input(D.F32, (4, 6, 8))
    g.mark_output(g.op("sum_dim", [xi], D.F32, (4, 8), attr=[1, 0]))
    g.mark_output(g.op("amax_dim", [xi], D.F32, (6, 8), attr=[0, 0]))
    assert _check(g, [x]).n_kernels == 2
    # a leading-dimension reduction next to a last-dimension one
    g = GraphBuilder(); xi = g.input(D.F32, (4, 6, 8))
    g.mark_output(g.op("sum_dim", [xi], D.F32, (4, 8), attr=[1, 0]))
    g.mark_output(g.op("softmax", [xi], D.F32, (4, 6, 8)))
    assert _check(g, [x]).n_kernels == 2
