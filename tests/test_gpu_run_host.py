"""pn_graph_run_host (tensors in host memory): the result equals the device-pointer path bit for
bit, for inputs large enough to be copied and computed in overlapping pieces along the outermost
dimension, for every kernel family, and for small inputs that go in one piece."""
import numpy as np
import pytest

import paper_2605_29357_b200 as pn
from pn_workloads import configs as C
from pn_workloads import descriptor as D

from gpu_util import check_against_oracle, run_graph

pytestmark = pytest.mark.gpu

CASES = {
    "c1_flat_pointwise": lambda: C.c1(M=3000, N=2048),
    "c1_ragged": lambda: C.c1(M=2999, N=2050),
    "c2_warp_rows": lambda: C.c2(B=100, Q=512, K=512),
    "c3_block_rows": lambda: C.c3(M=5000, N=4096),
    "c4_cluster_rows": lambda: C.c4(M=64, N=262144),
    "c5_block_chunks": lambda: C.c5(M=1100, N=14336),
    "n2_columns": lambda: C.n2(B=50),
    "n1_mapped_input": lambda: C.n1(),
    "c3_small": lambda: C.c3(**C.SMALL["c3"]),
}


def _run_host(g, w, pinned):
    import torch
    ins = [torch.from_numpy(np.ascontiguousarray(a).reshape(-1).view(np.uint8).copy()) for a in w.inputs]
    sizes = [D.DTYPE_BYTES[dt] * int(np.prod(dims, dtype=np.int64)) for dt, dims in w.output_meta]
    outs = [torch.full((max(s, 16),), 0xFF, dtype=torch.uint8) for s in sizes]
    if pinned:
        ins = [t.pin_memory() for t in ins]; outs = [t.pin_memory() for t in outs]
    g.run_host([t.data_ptr() for t in ins], [t.data_ptr() for t in outs], torch.cuda.current_stream().cuda_stream)
    return [t.numpy()[:s].view(C.NP_STORAGE[dt]).reshape(dims) for t, (dt, dims), s in zip(outs, w.output_meta, sizes)]


@pytest.mark.parametrize("case", list(CASES))
def test_host_path_equals_device_path(case):
    w = CASES[case]()
    g = pn.Graph(w.desc, 0, 0)
    ref = run_graph(g, w.inputs)
    for pinned in (True, False):
        got = _run_host(g, w, pinned)
        for a, b, name in zip(got, ref, w.output_names):
            assert np.array_equal(a, b, equal_nan=True), (case, name, pinned)
    again = run_graph(g, w.inputs)                 # the handle still runs whole afterwards
    assert all(np.array_equal(a, b, equal_nan=True) for a, b in zip(again, ref))
    if case == "c3_small":
        check_against_oracle(w.desc, w.inputs, got, w.output_meta, w.output_names)


def test_unfused_handle_through_host_memory():
    w = C.c5(M=64, N=1432)
    g = pn.Graph(w.desc, 0, pn.FLAG_UNFUSED)
    got = _run_host(g, w, True)
    check_against_oracle(w.desc, w.inputs, got, w.output_meta, w.output_names)


def test_bound_launch_equals_plain_run():
    """Graph.bind marshals the pointer arrays once; launching through it gives the same bits."""
    import torch
    from gpu_util import device_bytes, poisoned
    w = C.c5(**C.SMALL["c5"])
    g = pn.Graph(w.desc, 0, 0)
    ref = run_graph(g, w.inputs)
    d_in = [device_bytes(a) for a in w.inputs]
    sizes = [D.DTYPE_BYTES[dt] * int(np.prod(dims, dtype=np.int64)) for dt, dims in w.output_meta]
    d_out = [poisoned(s) for s in sizes]
    launch = g.bind([t.data_ptr() for t in d_in], [t.data_ptr() for t in d_out])
    for _ in range(2):
        launch(torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    for t, (dt, dims), s, r in zip(d_out, w.output_meta, sizes, ref):
        assert np.array_equal(t.cpu().numpy()[:s].view(C.NP_STORAGE[dt]).reshape(dims), r, equal_nan=True)
    with pytest.raises(pn.PnError):
        g.bind([t.data_ptr() for t in d_in][:-1], [t.data_ptr() for t in d_out])(0)
