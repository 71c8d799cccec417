"""GPU parity of the index operators (roll, slice, view: Section 3.2's index-remapped
loads) against the CPU oracle: each operator alone, over leading dimensions and over the last
one, chains of them feeding arithmetic, and the roll + slice + add + LayerNorm subgraph at
reduced and full size."""
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


LAST = {"default": 0, "interpret": pn.FLAG_INTERPRET, "unfused": pn.FLAG_UNFUSED, "scalar": pn.FLAG_FORCE_SCALAR,
        "bounds": pn.FLAG_BOUNDS, "block": pn.FLAG_FORCE_BLOCK}


@pytest.mark.parametrize("force", list(LAST))
@pytest.mark.parametrize("dtype", [D.F32, D.BF16])
@pytest.mark.parametrize("shape,shift", [((7, 64), 8), ((7, 64), 5), ((3, 5, 96), -16), ((2, 3, 4, 40), 39), ((1, 1000), 250),
                                         ((9, 33), 4)])
def test_roll_over_the_last_dimension(shape, shift, dtype, force):
    """Column c is read at (c - shift) mod N: whole 128-bit groups when the shift and the row length
    allow it, element by element otherwise."""
    x = _values(shape, dtype, 70)
    g = GraphBuilder(); xi = g.input(dtype, shape)
    r = g.op("roll", [xi], dtype, shape, attr=[len(shape) - 1, shift])
    g.mark_output(r)                                                   # the roll alone: a copy with moved columns
    f = g.op("cast", [r], D.F32, shape)
    g.mark_output(g.op("sum", [g.op("mul", [f, f], D.F32, shape)], D.F32, shape[:-1]))   # and feeding a row reduction
    gr, outs = _run(g, [x], LAST[force])
    assert np.array_equal(outs[0], np.roll(x, shift, axis=len(shape) - 1))
    if force == "default":
        assert gr.n_kernels == 1
    if force == "bounds":
        assert gr.bounds_status == 0


@pytest.mark.parametrize("force", list(LAST))
@pytest.mark.parametrize("dtype", [D.F32, D.BF16])
@pytest.mark.parametrize("shape,start,length", [((7, 64), 8, 32), ((7, 64), 3, 31), ((3, 5, 96), 48, 48), ((2, 3, 4, 40), 0, 8),
                                                ((1, 1000), 500, 500), ((16, 2048), 1024, 1024)])
def test_slice_of_the_last_dimension(shape, start, length, dtype, force):
    x = _values(shape, dtype, 71)
    out_shape = shape[:-1] + (length,)
    g = GraphBuilder(); xi = g.input(dtype, shape)
    s = g.op("slice", [xi], dtype, out_shape, attr=[len(shape) - 1, start])
    g.mark_output(s)
    f = g.op("cast", [s], D.F32, out_shape)
    g.mark_output(g.op("softmax", [f], D.F32, out_shape))
    gr, outs = _run(g, [x], LAST[force])
    assert np.array_equal(outs[0], x[..., start:start + length])
    if force == "default":
        assert gr.n_kernels == 1
    if force == "bounds":
        assert gr.bounds_status == 0


@pytest.mark.parametrize("flags", [0, pn.FLAG_INTERPRET, pn.FLAG_UNFUSED, pn.FLAG_FORCE_SCALAR, pn.FLAG_BOUNDS])
@pytest.mark.parametrize("M,N", [(64, 1024), (5, 24), (3, 7)])
def test_gated_activation_reads_both_halves_of_one_tensor(M, N, flags):
    """x[..., :N] * silu(x[..., N:]) with a LayerNorm behind it: two slices of the last dimension of
    one input, each its own view of the same buffer, in one kernel."""
    x = _values((M, 2 * N), D.BF16, 72)
    ga = _values((N,), D.F32, 73); be = _values((N,), D.F32, 74)
    g = GraphBuilder(); xi = g.input(D.BF16, (M, 2 * N)); gi = g.input(D.F32, (N,)); bi = g.input(D.F32, (N,))
    a = g.op("cast", [g.op("slice", [xi], D.BF16, (M, N), attr=[1, 0])], D.F32, (M, N))
    b = g.op("cast", [g.op("slice", [xi], D.BF16, (M, N), attr=[1, N])], D.F32, (M, N))
    h = g.op("mul", [a, g.op("silu", [b], D.F32, (M, N))], D.F32, (M, N))
    y = g.node("layer_norm", [h, gi, bi], [D.F32], [(M, N)], extra_imm=[1e-5])[0]
    g.mark_output(g.op("cast", [y], D.BF16, (M, N)))
    gr, _ = _run(g, [x, ga, be], flags)
    if not flags & pn.FLAG_UNFUSED:
        assert gr.n_kernels == 1
        assert gr.compulsory_bytes == x.nbytes + ga.nbytes + be.nbytes + M * N * 2


@pytest.mark.parametrize("flags", [0, pn.FLAG_INTERPRET, pn.FLAG_UNFUSED])
def test_rolls_and_slices_over_leading_and_last_dimensions_compose(flags):
    """One node rolling a leading and the last dimension at once, a slice of both behind it, then a
    second slice of the last dimension; and a view of a dense input that regroups the last dimension."""
    x = _values((6, 10, 48), D.F32, 75)
    g = GraphBuilder(); xi = g.input(D.F32, x.shape)
    r = g.op("roll", [xi], D.F32, (6, 10, 48), attr=[1, 3], extra_imm=[3, 8])             # dims 1 and 2
    s = g.op("slice", [r], D.F32, (6, 7, 32), attr=[1, 2], extra_imm=[3, 4])              # rows 2.., columns 4..
    s2 = g.op("slice", [s], D.F32, (6, 7, 16), attr=[2, 8])
    g.mark_output(g.op("exp", [s2], D.F32, (6, 7, 16)))
    gr, outs = _run(g, [x], flags)
    want = np.roll(np.roll(x, 3, axis=1), 8, axis=2)[:, 2:9, 4:36][:, :, 8:24]
    assert np.allclose(outs[0], np.exp(want.astype(np.float64)), rtol=1e-5)
    v = GraphBuilder(); vi = v.input(D.F32, (6, 10, 48))
    w = v.op("view", [vi], D.F32, (60, 4, 12))
    v.mark_output(v.op("relu", [v.op("slice", [w], D.F32, (60, 4, 6), attr=[2, 6])], D.F32, (60, 4, 6)))
    _run(v, [x], flags)


def test_gated_halves_workload_small_and_full_size():
    """The supplementary sweep shape: every element at a reduced size; at the size the benchmark
    times, the rows of a sample (rows are independent) and the byte count."""
    from oracle import evaluator as E
    w = C.gated_halves(M=19, N=1432)
    g = pn.Graph(w.desc, 0, 0)
    check_against_oracle(w.desc, w.inputs, run_graph(g, w.inputs), w.output_meta, w.output_names)
    w = C.gated_halves()
    g = pn.Graph(w.desc, 0, 0)
    assert g.n_kernels == 1 and g.compulsory_bytes == w.inputs[0].nbytes * 3 // 2
    out = run_graph(g, w.inputs)[0]
    rows = np.random.default_rng(5).choice(w.inputs[0].shape[0], size=64, replace=False)
    sub = C.gated_halves(M=64)
    ref = E.evaluate(sub.desc, [np.ascontiguousarray(w.inputs[0][rows])])
    check_against_oracle(sub.desc, None, [out[rows]], sub.output_meta, sub.output_names, ref=ref)
