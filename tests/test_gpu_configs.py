"""GPU parity of the five benchmark subgraphs against the CPU oracle, through the C ABI:
reduced sizes in every kernel family (element by element), and the full benchmark sizes in
the launch configuration the benchmark times."""
import numpy as np
import pytest

import paper_2605_29357_b200 as pn
from oracle import evaluator as E
from pn_workloads import configs as C

from gpu_util import check_against_oracle, run_graph

pytestmark = pytest.mark.gpu

FORCES = {
    "default": 0,
    "interpret": pn.FLAG_INTERPRET,
    "interpret_unfused": pn.FLAG_INTERPRET | pn.FLAG_UNFUSED,
    "interpret_cluster": pn.FLAG_INTERPRET | pn.FLAG_FORCE_CLUSTER,
    "interpret_block_multichunk": pn.FLAG_INTERPRET | pn.FLAG_FORCE_BLOCK | pn.FLAG_FORCE_MULTICHUNK,
    "unfused": pn.FLAG_UNFUSED,
    "scalar": pn.FLAG_FORCE_SCALAR,
    "warp": pn.FLAG_FORCE_WARP,
    "block": pn.FLAG_FORCE_BLOCK,
    "cluster": pn.FLAG_FORCE_CLUSTER,
    "block_multichunk": pn.FLAG_FORCE_BLOCK | pn.FLAG_FORCE_MULTICHUNK,
    "cluster_multichunk": pn.FLAG_FORCE_CLUSTER | pn.FLAG_FORCE_MULTICHUNK,
    "warp_scalar": pn.FLAG_FORCE_WARP | pn.FLAG_FORCE_SCALAR,
    "split": pn.FLAG_FORCE_SPLIT,
}


@pytest.mark.parametrize("force", list(FORCES))
@pytest.mark.parametrize("cfg", ["c1", "c2", "c3", "c4", "c5"])
def test_small_config(cfg, force):
    w = C.CONFIGS[cfg](**C.SMALL[cfg])
    g = pn.Graph(w.desc, 0, FORCES[force])
    outs = run_graph(g, w.inputs)
    check_against_oracle(w.desc, w.inputs, outs, w.output_meta, w.output_names)
    want_spec = 0 if force.startswith("interpret") else 1
    assert all(k["specialised"] == want_spec for k in g.kernel_info)
    if force == "default":
        assert g.n_kernels == 1
    if force == "unfused":
        assert g.n_kernels == w.n_nodes


@pytest.mark.parametrize("cfg,kw", [
    ("c1", dict(M=64, N=1024)), ("c2", dict(B=2, Q=64, K=512)), ("c3", dict(M=40, N=4096)),
    ("c4", dict(M=3, N=262144)), ("c5", dict(M=24, N=14336)),
    ("c1", dict(M=5, N=1024, dtype=2)), ("c3", dict(M=9, N=4096, dtype=0)),
    ("c5", dict(M=7, N=14336, dtype=1)), ("c2", dict(B=2, Q=16, K=512, dtype=1)),
    ("c3", dict(M=6, N=1024, also_output_sum=True)),
])
def test_benchmark_row_lengths_few_rows(cfg, kw):
    """The benchmark row lengths (so the same family and tile as the full size) on few rows,
    plus the other storage types of the same graphs."""
    w = C.CONFIGS[cfg](**kw)
    g = pn.Graph(w.desc, 0, 0)
    outs = run_graph(g, w.inputs)
    check_against_oracle(w.desc, w.inputs, outs, w.output_meta, w.output_names)


def _oracle_by_row_blocks(w, builder, kw, row_key, rows, block):
    """Oracle results for the full problem, computed on blocks of rows so that the fp64
    intermediates stay bounded.  Rows are independent, so each block is its own problem."""
    refs = None
    for lo in range(0, rows, block):
        hi = min(rows, lo + block)
        kw2 = dict(kw); kw2[row_key] = hi - lo
        sub = builder(**kw2)            # descriptor of the smaller shape (its inputs are ignored)
        ins = []
        for arr, (dt, dims) in zip(w.inputs, w.input_meta):
            sliced = len(dims) == len(w.input_meta[0][1]) and dims[0] == rows
            ins.append(arr[lo:hi] if sliced else arr)
        r = E.evaluate(sub.desc, ins)
        refs = [[x] for x in r] if refs is None else [a + [x] for a, x in zip(refs, r)]
    return [np.concatenate(a, axis=0) for a in refs]


@pytest.mark.parametrize("cfg", ["c1", "c2", "c3", "c4", "c5"])
def test_full_size_config(cfg):
    w = C.CONFIGS[cfg]()
    g = pn.Graph(w.desc, 0, 0)
    assert g.n_kernels == 1 and g.compulsory_bytes == w.compulsory_bytes
    outs = run_graph(g, w.inputs)
    rows = w.input_meta[0][1][0]
    key = "B" if cfg == "c2" else "M"
    block = {"c1": 1024, "c2": 32, "c3": 2048, "c4": 64, "c5": 512}[cfg]
    ref = _oracle_by_row_blocks(w, C.CONFIGS[cfg], {}, key, rows, block)
    check_against_oracle(w.desc, w.inputs, outs, w.output_meta, w.output_names, ref=ref)
    if cfg == "c4":
        assert w.notes["spikes_per_row_min"] >= 2
        x = w.inputs[0]
        first = np.array([np.flatnonzero(r == np.float32(30.0))[0] for r in x])
        assert np.array_equal(outs[1], first)        # lowest index among the tied maxima
    if cfg == "c5":
        a = E.widen(w.inputs[0], w.input_meta[0][0])
        assert np.array_equal(outs[1], (a > 0).astype(np.int8))
