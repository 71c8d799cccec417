"""Helpers shared by the GPU tests: move seeded inputs to the device, run a graph through
the C ABI with poisoned output buffers, and judge the result against the CPU oracle."""
import numpy as np

from oracle import evaluator as E
from pn_workloads import configs as C
from pn_workloads import descriptor as D


def device_bytes(arr):
    import torch
    flat = np.ascontiguousarray(arr).reshape(-1).view(np.uint8)
    if flat.size == 0:
        return torch.empty(16, dtype=torch.uint8, device="cuda")
    return torch.from_numpy(flat.copy()).cuda()


def poisoned(nbytes):
    """Output buffer filled with 0xFF bytes (NaN for floats, -1 for integers): a kernel that
    skips an element cannot pass by finding stale data there."""
    import torch
    return torch.full((max(int(nbytes), 16),), 0xFF, dtype=torch.uint8, device="cuda")


def run_graph(graph, inputs, stream=None):
    """inputs: host arrays in descriptor order.  Returns host arrays in storage dtype."""
    import torch
    d_in = [device_bytes(a) for a in inputs]
    metas = graph.output_meta
    sizes = [D.DTYPE_BYTES[dt] * int(np.prod(dims, dtype=np.int64)) for dt, dims in metas]
    d_out = [poisoned(s) for s in sizes]
    graph.run([t.data_ptr() for t in d_in], [t.data_ptr() for t in d_out],
              0 if stream is None else stream.cuda_stream)
    torch.cuda.synchronize()
    outs = []
    for t, (dt, dims), s in zip(d_out, metas, sizes):
        host = t.cpu().numpy()[:s]
        outs.append(host.view(C.NP_STORAGE[dt]).reshape(dims))
    return outs


def check_against_oracle(desc, inputs, outs, metas, names=None, ref=None):
    """Every element of every output against the oracle under the per-dtype rule."""
    if ref is None:
        ref = E.evaluate(desc, inputs)
    report = []
    for i, (got, r, (dt, dims)) in enumerate(zip(outs, ref, metas)):
        val = E.widen(got, dt)
        res = E.compare(val, r, dt)
        res["name"] = names[i] if names else str(i)
        report.append(res)
    bad = [r for r in report if not r["ok"]]
    assert not bad, f"oracle mismatch: {bad}"
    return report
