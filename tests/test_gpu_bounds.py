"""Checked accessors (PN_FLAG_BOUNDS): with every global access of the kernels tested against the
extent of its tensor, all workloads still match the oracle and the status word stays 0 -- on the
generated kernels, on the interpreter and on the unfused path.  (This is the library's stand-in for
a memory checker: no access outside a tensor goes unnoticed.)"""
import numpy as np
import pytest

import paper_2605_29357_b200 as pn
from pn_workloads import configs as C
from pn_workloads import descriptor as D
from pn_workloads.descriptor import GraphBuilder

from gpu_util import check_against_oracle, run_graph

pytestmark = pytest.mark.gpu

ALL = {**C.CONFIGS, **C.EXTENDED}
MODES = {"generated": 0, "interpreter": pn.FLAG_INTERPRET, "unfused": pn.FLAG_UNFUSED, "scalar": pn.FLAG_FORCE_SCALAR,
         "cluster": pn.FLAG_FORCE_CLUSTER, "block_multichunk": pn.FLAG_FORCE_BLOCK | pn.FLAG_FORCE_MULTICHUNK}


@pytest.mark.parametrize("mode", list(MODES))
@pytest.mark.parametrize("cfg", list(ALL))
def test_no_access_leaves_its_tensor(cfg, mode):
    if cfg == "n2" and mode in ("cluster", "block_multichunk"):
        pytest.skip("row-kernel forcing flags do not apply to column kernels")
    w = ALL[cfg](**C.SMALL[cfg])
    g = pn.Graph(w.desc, 0, MODES[mode] | pn.FLAG_BOUNDS)
    outs = run_graph(g, w.inputs)
    check_against_oracle(w.desc, w.inputs, outs, w.output_meta, w.output_names)
    assert g.bounds_status == 0


@pytest.mark.parametrize("rows,n", [(3, 7), (5, 1001), (33, 96), (2, 20000), (130, 40)])
def test_ragged_shapes_under_checking(rows, n):
    x = np.random.default_rng(rows * n).standard_normal((rows, n)).astype(np.float32)
    g = GraphBuilder(); xi = g.input(D.F32, (rows, n))
    sm = g.op("softmax", [xi], D.F32, (rows, n))
    g.mark_output(g.op("cast", [sm], D.BF16, (rows, n)))
    g.mark_output(g.op("argmax", [xi], D.I64, (rows,)))
    g.mark_output(g.op("sum", [xi], D.F32, (rows, 1)))
    for flags in (0, pn.FLAG_INTERPRET):
        h = pn.Graph(g.build(), 0, flags | pn.FLAG_BOUNDS)
        outs = run_graph(h, [x])
        check_against_oracle(g.build(), [x], outs, [g.tensor_meta(t) for t in g.output_ids()])
        assert h.bounds_status == 0


def test_status_query_needs_the_flag():
    w = C.c1(**C.SMALL["c1"])
    g = pn.Graph(w.desc, 0, 0)
    with pytest.raises(pn.PnError) as e:
        g.bounds_status
    assert e.value.status == -1
