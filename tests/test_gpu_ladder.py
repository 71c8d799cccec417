"""Every instance of the error-aware speedup sweep against the CPU oracle.

The sweep of the report module (seven workload graphs x ten shapes x {f32, f16, bf16} = 210
instances) scores "correct at t" by comparing the fused handle with the unfused one of the same
library, and both run the same device functions.  What makes that score rest on the paper's rule
(Definition 3.2, Eq. 1; the ladder of Section 3.5) is this test: the fused handle of every one of
those instances, run through the C ABI, against the oracle under the per-dtype tolerance.  Small
instances are compared element by element; in the large ones the rows are independent problems,
so blocks of the leading dimension (first, last, middle and two drawn at random) are compared
element by element, each evaluated by the oracle as a problem of its own."""
import numpy as np
import pytest

import paper_2605_29357_b200 as pn
from oracle import evaluator as E
from paper_2605_29357_b200 import report as R
from pn_workloads import configs as C
from pn_workloads import descriptor as D

from gpu_util import run_graph

pytestmark = pytest.mark.gpu

MAKERS = {**C.CONFIGS, **C.EXTENDED}
LEAD_KEY = {"c1": "M", "c2": "B", "c3": "M", "c4": "M", "c5": "M", "n2": "B"}      # n1's rows are re-indexed: always whole
WHOLE_BELOW = 3_000_000                                                              # elements of the largest tensor
DTYPES = {"f32": D.F32, "f16": D.F16, "bf16": D.BF16}
LADDER = R._shape_ladder()
CASES = [(name, i, dn) for name in LADDER for i in range(len(LADDER[name])) for dn in DTYPES]


def _compare(got, ref, metas, label):
    for k, (a, r, (dt, _dims)) in enumerate(zip(got, ref, metas)):
        res = E.compare(E.widen(a, dt), r, dt)
        assert res["ok"], (label, k, res)


@pytest.mark.parametrize("name,index,dname", CASES, ids=[f"{n}-{i}-{d}" for n, i, d in CASES])
def test_ladder_instance_matches_the_oracle(name, index, dname):
    shape = LADDER[name][index]
    w = MAKERS[name](dtype=DTYPES[dname], **shape)
    g = pn.Graph(w.desc, 0, 0)
    assert g.n_kernels == 1
    outs = run_graph(g, w.inputs)
    biggest = max(int(np.prod(dims, dtype=np.int64)) for _dt, dims in w.input_meta + w.output_meta)
    label = f"{name}{sorted(shape.items())}/{dname}"
    if biggest <= WHOLE_BELOW or name not in LEAD_KEY:
        _compare(outs, E.evaluate(w.desc, w.inputs), w.output_meta, label)
        return
    key = LEAD_KEY[name]
    rows = shape[key]
    full_rank = len(w.input_meta[0][1])
    block = max(1, min(rows, WHOLE_BELOW // max(1, biggest // rows)))
    rng = np.random.default_rng(index)
    starts = sorted({0, max(0, rows - block), max(0, rows // 2 - block // 2)} |
                    {int(s) for s in rng.integers(0, max(1, rows - block + 1), size=2)})
    for lo in starts:
        hi = min(rows, lo + block)
        sub = MAKERS[name](dtype=DTYPES[dname], **dict(shape, **{key: hi - lo}))   # the descriptor of the block (its own inputs are ignored)
        ins = [arr[lo:hi] if (len(dims) == full_rank and dims[0] == rows) else arr for arr, (_dt, dims) in zip(w.inputs, w.input_meta)]
        ref = E.evaluate(sub.desc, ins)
        got = [o[lo:hi] if (len(dims) >= 1 and dims[0] == rows) else o for o, (_dt, dims) in zip(outs, w.output_meta)]
        _compare(got, ref, sub.output_meta, f"{label} rows {lo}:{hi}")
