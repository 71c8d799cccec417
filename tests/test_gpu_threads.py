"""Several host threads at once: creating handles of the same graph (the kernel cache must hand all
of them one kernel) and running one fused handle on different buffers and streams (a run only reads
the handle).  ctypes releases the interpreter lock during the calls, so the calls do overlap."""
import threading

import numpy as np
import pytest

import paper_2605_29357_b200 as pn
from pn_workloads import configs as C
from pn_workloads import descriptor as D

from gpu_util import check_against_oracle, device_bytes, poisoned

pytestmark = pytest.mark.gpu


def _sizes(w):
    return [D.DTYPE_BYTES[dt] * int(np.prod(dims, dtype=np.int64)) for dt, dims in w.output_meta]


def test_threads_create_the_same_graph_and_share_its_kernel():
    w = C.c3(M=21, N=1096)                      # a shape no other test compiles
    made, errors = [None] * 6, []

    def create(i):
        try:
            made[i] = pn.Graph(w.desc, 0, 0)
        except Exception as e:                  # reported below, in the main thread
            errors.append(e)

    other = pn.Graph(C.c1(M=4, N=64).desc, 0, 0)
    before = other.kernel_cache[1]              # kernels that a live handle uses (unused ones may be unloaded at any time)
    threads = [threading.Thread(target=create, args=(i,)) for i in range(len(made))]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    modules, in_use = made[0].kernel_cache
    assert in_use == before + 1                 # six handles, one kernel loaded for them
    from gpu_util import run_graph
    for g in made:
        check_against_oracle(w.desc, w.inputs, run_graph(g, w.inputs), w.output_meta, w.output_names)
        g.close()
    other.close()


@pytest.mark.parametrize("cfg", ["c2", "c3", "n1"])
def test_threads_run_one_handle_on_their_own_buffers(cfg):
    import torch
    makers = {**C.CONFIGS, **C.EXTENDED}
    n_threads, runs = 4, 50
    works = [makers[cfg](seed=10 + i, **C.SMALL[cfg]) for i in range(n_threads)]
    g = pn.Graph(works[0].desc, 0, 0)
    assert g.workspace_bytes == 0               # nothing but the caller's buffers is written
    sizes = _sizes(works[0])
    d_in = [[device_bytes(a) for a in w.inputs] for w in works]
    d_out = [[poisoned(s) for s in sizes] for _ in works]
    streams = [torch.cuda.Stream() for _ in works]
    torch.cuda.synchronize()
    errors = []

    def run(i):
        try:
            ins, outs = [t.data_ptr() for t in d_in[i]], [t.data_ptr() for t in d_out[i]]
            for _ in range(runs):
                g.run(ins, outs, streams[i].cuda_stream)
        except Exception as e:
            errors.append(e)

    threads = [threading.Thread(target=run, args=(i,)) for i in range(n_threads)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    torch.cuda.synchronize()
    assert not errors, errors
    for w, outs in zip(works, d_out):
        got = [t.cpu().numpy()[:s].view(C.NP_STORAGE[dt]).reshape(dims) for t, s, (dt, dims) in zip(outs, sizes, w.output_meta)]
        check_against_oracle(w.desc, w.inputs, got, w.output_meta, w.output_names)
    g.close()
