"""Seeded random graphs against the CPU oracle, through the C ABI, with checked accessors on: the
register allocator, the stage splitter and the spill / fill paths of the lowering meet graph
structures nobody wrote by hand (the paper's demand that a rewrite hold in general rather than fit
one instance, Section 3.1, applied to the graph itself).  Every graph runs fused on generated
kernels (one launch, or a few where a kernel budget cuts the graph); in turn also on the
interpreter, node by node (unfused), and in a forced kernel family.  A mode that refuses a graph
must do so with a documented status."""
import numpy as np
import pytest

import paper_2605_29357_b200 as pn

import rand_graphs
from gpu_util import check_against_oracle, run_graph
from oracle import evaluator as E

pytestmark = pytest.mark.gpu

N_SEEDS = 200
FORCED = [pn.FLAG_FORCE_WARP, pn.FLAG_FORCE_BLOCK, pn.FLAG_FORCE_CLUSTER, pn.FLAG_FORCE_BLOCK | pn.FLAG_FORCE_MULTICHUNK,
          pn.FLAG_FORCE_SCALAR, pn.FLAG_FORCE_SPLIT, pn.FLAG_FORCE_CLUSTER | pn.FLAG_FORCE_MULTICHUNK, pn.FLAG_NO_HOIST]
DOCUMENTED_REFUSALS = {-3, -5}


def _modes(seed):
    m = [("generated", 0)]
    if seed % 2 == 0:
        m.append(("forced", FORCED[(seed // 2) % len(FORCED)]))
    else:
        m.append(("interpreter", pn.FLAG_INTERPRET))
    if seed % 4 == 1:
        m.append(("unfused interpreter", pn.FLAG_UNFUSED | pn.FLAG_INTERPRET))
    if seed % 20 == 7:
        m.append(("unfused generated", pn.FLAG_UNFUSED))
    return m


@pytest.mark.parametrize("seed", range(N_SEEDS))
def test_random_graph(seed):
    rg = rand_graphs.make(seed)
    ref = E.evaluate(rg.desc, rg.inputs)
    ran = 0
    for label, flags in _modes(seed):
        try:
            g = pn.Graph(rg.desc, 0, flags | pn.FLAG_BOUNDS)
        except pn.PnError as e:
            assert e.status in DOCUMENTED_REFUSALS, (seed, label, e.status, e.detail)
            continue
        outs = run_graph(g, rg.inputs)
        check_against_oracle(rg.desc, rg.inputs, outs, rg.output_meta, names=[f"seed {seed} {label} out {k}" for k in range(len(outs))], ref=ref)
        assert g.bounds_status == 0, (seed, label)
        ran += 1
        g.close()
    if ran == 0:           # refused as one kernel in every mode tried: node by node it must run
        g = pn.Graph(rg.desc, 0, pn.FLAG_UNFUSED | pn.FLAG_INTERPRET | pn.FLAG_BOUNDS)
        outs = run_graph(g, rg.inputs)
        check_against_oracle(rg.desc, rg.inputs, outs, rg.output_meta, ref=ref)
        assert g.bounds_status == 0


COLUMN_MODES = [("generated", 0), ("interpreter", pn.FLAG_INTERPRET), ("slices", pn.FLAG_FORCE_SPLIT),
                ("three slices", pn.tune(cluster=3)), ("unfused", pn.FLAG_UNFUSED), ("scalar", pn.FLAG_FORCE_SCALAR)]


@pytest.mark.parametrize("seed", list(range(80)) + [711])      # (711: the kernel that spilled under its register bound)
def test_random_column_graph(seed):
    """Random graphs that reduce over a leading dimension (chains with broadcast operands before the
    reductions and on the reduced values after them): generated kernels, and in turn the interpreter,
    the reduced dimension cut into slices, node by node, element-wise accesses."""
    rg = rand_graphs.make_column(seed)
    ref = E.evaluate(rg.desc, rg.inputs)
    ran = 0
    for label, flags in [COLUMN_MODES[0], COLUMN_MODES[1 + seed % (len(COLUMN_MODES) - 1)]]:
        try:
            g = pn.Graph(rg.desc, 0, flags | pn.FLAG_BOUNDS)
        except pn.PnError as e:
            assert e.status in DOCUMENTED_REFUSALS, (seed, label, e.status, e.detail)
            continue
        outs = run_graph(g, rg.inputs)
        check_against_oracle(rg.desc, rg.inputs, outs, rg.output_meta, names=[f"column seed {seed} {label} out {k}" for k in range(len(outs))], ref=ref)
        again = run_graph(g, rg.inputs)                     # arrival counters back at zero; the same bits
        assert all(np.array_equal(a.view(np.uint8), b.view(np.uint8)) for a, b in zip(outs, again)), (seed, label)
        assert g.bounds_status == 0, (seed, label)
        ran += 1
        g.close()
    assert ran >= 1, seed
