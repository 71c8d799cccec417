"""GPU parity of the index operators (roll, slice, view: Section 3.2's index-remapped
loads) against the CPU oracle: each operator alone, chains of them feeding arithmetic, and
the roll + slice + add + LayerNorm subgraph at reduced and full size."""
import numpy as np
import pytest

import paper_2605_29357_b200 as pn
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
    "warp": pn.FLAG_FORCE_WARP,
    "block": pn.FLAG_FORCE_BLOCK,
    "cluster": pn.FLAG_FORCE_CLUSTER,
    "block_multichunk": pn.FLAG_FORCE_BLOCK | pn.FLAG_FORCE_MULTICHUNK,
}


def _values(shape, dtype, seed):
    rng = np.random.default_rng(seed)
    if dtype == D.I32:
        return rng.integers(-1000, 1000, size=shape, dtype=np.int32)
    x = rng.standard_normal(shape).astype(np.float32)
    if dtype == D.BF16:
        return C.to_bf16_bits(x)
    if dtype == D.F16:
        return x.astype(np.float16)
    return x


def _run(g, inputs, flags=0):
    desc = g.build()
    gr = pn.Graph(desc, 0, flags)
    outs = run_graph(gr, inputs)
    metas = [g.tensor_meta(t) for t in g.output_ids()]
    check_against_oracle(desc, inputs, outs, metas)
    return gr, outs


@pytest.mark.parametrize("force", list(FORCES))
@pytest.mark.parametrize("kw", [dict(S=13, SC=8, Cc=40, shift=3), dict(S=9, SC=9, Cc=96, shift=2),
                                dict(S=11, SC=7, Cc=1000, shift=5, dtype=D.F32)])
def test_roll_slice_add_layernorm_small(kw, force):
    w = C.n1(**kw)
    g = pn.Graph(w.desc, 0, FORCES[force])
    outs = run_graph(g, w.inputs)
    check_against_oracle(w.desc, w.inputs, outs, w.output_meta, w.output_names)
    if force == "default":
        assert g.n_kernels == 1          # no data movement kernel: the chain became addressing


def test_roll_slice_add_layernorm_full_size():
    w = C.n1()
    g = pn.Graph(w.desc, 0, 0)
    assert g.n_kernels == 1
    outs = run_graph(g, w.inputs)
    check_against_oracle(w.desc, w.inputs, outs, w.output_meta, w.output_names)


@pytest.mark.parametrize("dtype", [D.F32, D.BF16, D.I32])
@pytest.mark.parametrize("shape,dim,shift", [((7, 40), 0, 2), ((5, 6, 24), 0, -1), ((5, 6, 24), 1, 4),
                                             ((3, 4, 5, 16), 2, 7), ((3, 4, 5, 16), 0, 1), ((6, 33), 0, 0)])
@pytest.mark.parametrize("flags", [0, pn.FLAG_INTERPRET, pn.FLAG_FORCE_SCALAR])
def test_roll_alone_is_a_copy_with_moved_rows(shape, dim, shift, dtype, flags):
    g = GraphBuilder()
    x = g.input(dtype, shape)
    g.mark_output(g.op("roll", [x], dtype, shape, attr=[dim, shift]))
    a = _values(shape, dtype, 1)
    _, outs = _run(g, [a], flags)
    assert np.array_equal(outs[0], np.roll(a, shift, axis=dim))   # bit-exact: nothing is computed


@pytest.mark.parametrize("shape,dim,start,length", [((9, 40), 0, 2, 5), ((5, 6, 24), 1, 1, 4),
                                                    ((3, 4, 5, 16), 0, 1, 2), ((3, 4, 5, 16), 2, 0, 5)])
@pytest.mark.parametrize("flags", [0, pn.FLAG_INTERPRET])
def test_slice_alone(shape, dim, start, length, flags):
    g = GraphBuilder()
    x = g.input(D.F32, shape)
    out_shape = tuple(length if d == dim else n for d, n in enumerate(shape))
    g.mark_output(g.op("slice", [x], D.F32, out_shape, attr=[dim, start]))
    a = _values(shape, D.F32, 2)
    _, outs = _run(g, [a], flags)
    assert np.array_equal(outs[0], np.take(a, range(start, start + length), axis=dim))


@pytest.mark.parametrize("flags", [0, pn.FLAG_INTERPRET, pn.FLAG_UNFUSED])
def test_view_regroups_leading_dimensions(flags):
    g = GraphBuilder()
    x = g.input(D.F32, (6, 4, 32))
    b = g.input(D.F32, (8, 1, 32))
    v = g.op("view", [x], D.F32, (8, 3, 32))
    g.mark_output(g.op("add", [v, b], D.F32, (8, 3, 32)))
    a = _values((6, 4, 32), D.F32, 3); bb = _values((8, 1, 32), D.F32, 4)
    _, outs = _run(g, [a, bb], flags)
    assert np.array_equal(outs[0], a.reshape(8, 3, 32) + bb)


@pytest.mark.parametrize("flags", [0, pn.FLAG_INTERPRET, pn.FLAG_UNFUSED, pn.FLAG_FORCE_SCALAR])
def test_two_differently_rolled_reads_of_one_input(flags):
    """One tensor read through two different chains, plus directly: three streams, one buffer."""
    g = GraphBuilder()
    shape = (6, 10, 48)
    x = g.input(D.F32, shape)
    up = g.op("roll", [x], D.F32, shape, attr=[0, 1])
    left = g.op("roll", [x], D.F32, shape, attr=[1, -2])
    s = g.op("add", [up, left], D.F32, shape)
    g.mark_output(g.op("sub", [s, x], D.F32, shape))
    a = _values(shape, D.F32, 5)
    _, outs = _run(g, [a], flags)
    assert np.array_equal(outs[0], (np.roll(a, 1, 0) + np.roll(a, -2, 1)) - a)


@pytest.mark.parametrize("flags", [0, pn.FLAG_INTERPRET, pn.FLAG_UNFUSED, pn.FLAG_FORCE_BLOCK])
def test_rolled_slice_feeds_a_row_reduction(flags):
    g = GraphBuilder()
    x = g.input(D.BF16, (12, 9, 200))
    r = g.op("roll", [x], D.BF16, (12, 9, 200), attr=[0, -5])
    s = g.op("slice", [r], D.BF16, (7, 9, 200), attr=[0, 3])
    s2 = g.op("slice", [s], D.BF16, (7, 4, 200), attr=[1, 2])
    f = g.op("cast", [s2], D.F32, (7, 4, 200))
    e = g.op("mul", [f, Imm(0.5)], D.F32, (7, 4, 200))
    g.mark_output(g.op("softmax", [e], D.F32, (7, 4, 200)))
    g.mark_output(g.op("sum", [f], D.F32, (7, 4, 1)))
    _run(g, [_values((12, 9, 200), D.BF16, 6)], flags)


def test_slice_then_slice_and_roll_compose():
    g = GraphBuilder()
    x = g.input(D.F32, (20, 16))
    a = g.op("roll", [x], D.F32, (20, 16), attr=[0, 7])
    b = g.op("roll", [a], D.F32, (20, 16), attr=[0, 6])      # two rolls add up
    c = g.op("slice", [b], D.F32, (15, 16), attr=[0, 4])
    d = g.op("slice", [c], D.F32, (5, 16), attr=[0, 9])      # two slices add up
    g.mark_output(g.op("neg", [d], D.F32, (5, 16)))
    v = _values((20, 16), D.F32, 7)
    _, outs = _run(g, [v])
    assert np.array_equal(outs[0], -np.roll(v, 13, 0)[13:18])
