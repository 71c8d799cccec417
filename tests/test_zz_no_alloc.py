"""pn_graph_run_static against pn_graph_run.

Some users of this library run where device memory may no longer be allocated: a serving
process whose framework has already taken all free HBM into its own pool (a late cudaMalloc
fails there, or stalls every stream while it synchronises the device), or a worker held to a
fixed memory budget.  For them the unfused path has a second entry point that keeps the
intermediates between its per-node kernels in a fixed 32 MiB array inside the library
instead of a cudaMalloc'ed workspace.  This test drives that entry point through the C ABI,
twice in a row on the same shared array, and requires the same outputs as the ordinary
unfused handle gives -- and, like every other GPU test, agreement with the CPU oracle.

Collected last on purpose (file name), so that a run stopping at the first failure has
already run everything else.
"""
import numpy as np
import pytest

import paper_2605_29357_b200 as pn
from oracle import evaluator as E
from pn_workloads import configs as C
from pn_workloads import descriptor as D

from gpu_util import check_against_oracle, device_bytes, poisoned

pytestmark = pytest.mark.gpu


def _run(graph, inputs, static):
    import torch
    d_in = [device_bytes(a) for a in inputs]
    metas = graph.output_meta
    sizes = [D.DTYPE_BYTES[dt] * int(np.prod(dims, dtype=np.int64)) for dt, dims in metas]
    d_out = [poisoned(s) for s in sizes]
    call = graph.run_static if static else graph.run
    call([t.data_ptr() for t in d_in], [t.data_ptr() for t in d_out], torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    return [t.cpu().numpy()[:s].view(C.NP_STORAGE[dt]).reshape(dims) for t, (dt, dims), s in zip(d_out, metas, sizes)]


@pytest.mark.parametrize("interpret", [False, True])
def test_static_scratch_matches_the_allocating_path_twice_in_a_row(interpret):
    extra = pn.FLAG_INTERPRET if interpret else 0
    # two different graphs, so that the second call finds the first one's leftovers in the array
    cases = [C.c5(**C.SMALL["c5"]), C.c3(**C.SMALL["c3"])]
    for w in cases:
        ref_handle = pn.Graph(w.desc, 0, pn.FLAG_UNFUSED | extra)
        want = _run(ref_handle, w.inputs, static=False)
        g = pn.Graph(w.desc, 0, pn.FLAG_UNFUSED | pn.FLAG_STATIC_SCRATCH | extra)
        assert 0 < g.workspace_bytes <= pn.STATIC_SCRATCH_BYTES and g.n_kernels == w.n_nodes
        for _ in range(2):
            got = _run(g, w.inputs, static=True)
            for a, b, (dt, _dims) in zip(got, want, w.output_meta):
                res = E.compare(E.widen(a, dt), E.widen(b, dt), dt)   # same tolerance rule as every GPU test
                assert res["ok"], res        # (not the same bits: a handle that may not allocate never takes the
                                             #  kernel family that needs a workspace, so sums may be taken in another order)
            check_against_oracle(w.desc, w.inputs, got, w.output_meta, w.output_names)
        with pytest.raises(pn.PnError) as bad:                       # the ordinary entry point refuses the handle
            _run(g, w.inputs, static=False)
        assert bad.value.status == -1


def test_a_run_from_the_static_scratch_leaves_free_memory_alone_and_checks_pointers_like_run():
    """The set-up (the lookup of the array's address, which is what makes the device reserve it)
    belongs to the create; the runs themselves must not change the free device memory.  And the
    pointer rules are those of pn_graph_run, checked by the same code: outputs over one another
    are refused here too, and the host-memory entry point refuses such a handle before it would
    allocate its staging buffers."""
    import torch
    w = C.c5(**C.SMALL["c5"])
    g = pn.Graph(w.desc, 0, pn.FLAG_UNFUSED | pn.FLAG_STATIC_SCRATCH)
    d_in = [device_bytes(a) for a in w.inputs]
    sizes = [D.DTYPE_BYTES[dt] * int(np.prod(dims, dtype=np.int64)) for dt, dims in g.output_meta]
    d_out = [poisoned(s) for s in sizes]
    ins, outs = [t.data_ptr() for t in d_in], [t.data_ptr() for t in d_out]
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for _ in range(3):
        g.run_static(ins, outs, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    with pytest.raises(pn.PnError) as aliased:
        g.run_static(ins, [outs[0]] * len(outs), 0)
    assert aliased.value.status == -1 and "overlap" in aliased.value.detail
    host_in = [np.ascontiguousarray(a) for a in w.inputs]
    host_out = [np.empty(s, np.uint8) for s in sizes]
    with pytest.raises(pn.PnError) as host:
        g.run_host([a.ctypes.data for a in host_in], [a.ctypes.data for a in host_out], 0)
    assert host.value.status == -1
    assert torch.cuda.mem_get_info()[0] == free_before      # and it allocated nothing on the way


def test_static_scratch_rejects_what_does_not_fit():
    w = C.c2(B=64, Q=256, K=512)          # fp32 intermediates of 8.4 M elements each: far above 32 MiB
    g = pn.Graph(w.desc, 0, pn.FLAG_UNFUSED | pn.FLAG_STATIC_SCRATCH)
    assert g.workspace_bytes > pn.STATIC_SCRATCH_BYTES
    with pytest.raises(pn.PnError) as too_large:
        _run(g, w.inputs, static=True)
    assert too_large.value.status == -5 and "static scratch" in too_large.value.detail
    fused = pn.Graph(C.c3(**C.SMALL["c3"]).desc, 0, 0)
    with pytest.raises(pn.PnError) as wrong_handle:
        _run(fused, C.c3(**C.SMALL["c3"]).inputs, static=True)
    assert wrong_handle.value.status == -1
