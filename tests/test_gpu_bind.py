"""pn_graph_bind / pn_bound_run: the same results as pn_graph_run, from a handle that is only read
(two bound objects of one handle on different buffers stay independent), and the calling
thread's current device is what it was."""
import numpy as np
import pytest

import paper_2605_29357_b200 as pn
from pn_workloads import configs as C
from pn_workloads import descriptor as D

from gpu_util import check_against_oracle, device_bytes, poisoned

pytestmark = pytest.mark.gpu


def _buffers(w):
    d_in = [device_bytes(a) for a in w.inputs]
    sizes = [D.DTYPE_BYTES[dt] * int(np.prod(dims, dtype=np.int64)) for dt, dims in w.output_meta]
    return d_in, [poisoned(s) for s in sizes], sizes


def _host(d_out, sizes, metas):
    return [t.cpu().numpy()[:s].view(C.NP_STORAGE[dt]).reshape(dims) for t, s, (dt, dims) in zip(d_out, sizes, metas)]


@pytest.mark.parametrize("cfg", ["c1", "c2", "c3", "c4", "c5", "n1", "n2"])
@pytest.mark.parametrize("flags", [0, pn.FLAG_UNFUSED, pn.FLAG_INTERPRET])
def test_bound_launches_equal_direct_runs_and_do_not_disturb_each_other(cfg, flags):
    import torch
    makers = {**C.CONFIGS, **C.EXTENDED}
    wa, wb = makers[cfg](seed=1, **C.SMALL[cfg]), makers[cfg](seed=2, **C.SMALL[cfg])
    g = pn.Graph(wa.desc, 0, flags)
    stream = torch.cuda.current_stream().cuda_stream
    ina, outa, sizes = _buffers(wa)
    inb, outb, _ = _buffers(wb)
    fa = g.bind([t.data_ptr() for t in ina], [t.data_ptr() for t in outa])
    fb = g.bind([t.data_ptr() for t in inb], [t.data_ptr() for t in outb])
    before = torch.cuda.current_device()
    fa(stream); fb(stream); fa(stream)          # interleaved: neither sees the other's pointers
    torch.cuda.synchronize()
    assert torch.cuda.current_device() == before
    got_a, got_b = _host(outa, sizes, wa.output_meta), _host(outb, sizes, wb.output_meta)
    check_against_oracle(wa.desc, wa.inputs, got_a, wa.output_meta, wa.output_names)
    check_against_oracle(wb.desc, wb.inputs, got_b, wb.output_meta, wb.output_names)
    # bit for bit what the checked entry point gives
    _, outc, _ = _buffers(wa)
    g.run([t.data_ptr() for t in ina], [t.data_ptr() for t in outc], stream)
    torch.cuda.synchronize()
    for x, y in zip(got_a, _host(outc, sizes, wa.output_meta)):
        assert np.array_equal(x.view(np.uint8), y.view(np.uint8))
    fa.close(); fb.close(); g.close()


def test_bind_runs_the_argument_checks_once_and_for_all():
    import torch
    w = C.c3(**C.SMALL["c3"])
    g = pn.Graph(w.desc, 0, 0)
    d_in, d_out, _ = _buffers(w)
    ins, outs = [t.data_ptr() for t in d_in], [t.data_ptr() for t in d_out]
    with pytest.raises(pn.PnError) as e:
        g.bind(ins[:-1], outs)
    assert e.value.status == -7
    with pytest.raises(pn.PnError) as e:
        g.bind([ins[0] + 2] + ins[1:], outs)
    assert e.value.status == -6
    with pytest.raises(pn.PnError) as e:
        g.bind(ins, [outs[0]] * len(outs))      # outputs over one another
    assert e.value.status == -1
    with pytest.raises(pn.PnError) as e:
        g.bind(ins, [ins[0]] + outs[1:])        # an output over an input, exactly
    assert e.value.status == -1
    st = pn.Graph(w.desc, 0, pn.FLAG_UNFUSED | pn.FLAG_STATIC_SCRATCH)
    with pytest.raises(pn.PnError) as e:
        st.bind(ins, outs)
    assert e.value.status == -1
    torch.cuda.synchronize()


def test_many_bound_launches_in_one_call():
    """pn_bound_run_many: the launches of several bound objects (different graphs, fused and cut into
    several kernels) in the order given, by one call; the same bits as one pn_bound_run each."""
    import torch
    makers = {**C.CONFIGS, **C.EXTENDED}
    stream = torch.cuda.current_stream().cuda_stream
    graphs, bound, outs_many, outs_one, keep = [], [], [], [], []
    for cfg, flags in (("c1", 0), ("c3", 0), ("c5", pn.FLAG_UNFUSED), ("n1", 0), ("c4", 0), ("n2", 0)):
        w = makers[cfg](seed=3, **C.SMALL[cfg])
        g = pn.Graph(w.desc, 0, flags)
        d_in, d_out, sizes = _buffers(w)
        _, d_ref, _ = _buffers(w)
        ins = [t.data_ptr() for t in d_in]
        bound.append(g.bind(ins, [t.data_ptr() for t in d_out]))
        one = g.bind(ins, [t.data_ptr() for t in d_ref])
        one(stream)
        graphs.append((g, w, sizes)); outs_many.append(d_out); outs_one.append(d_ref); keep.append((d_in, one))
    many = pn.BoundList(bound)
    before = torch.cuda.current_device()
    many(stream)
    many(stream)                                   # (arrival counters of split kernels are back at zero)
    torch.cuda.synchronize()
    assert torch.cuda.current_device() == before
    for (g, w, sizes), d_out, d_ref in zip(graphs, outs_many, outs_one):
        got = _host(d_out, sizes, w.output_meta)
        check_against_oracle(w.desc, w.inputs, got, w.output_meta, w.output_names)
        for x, y in zip(got, _host(d_ref, sizes, w.output_meta)):
            assert np.array_equal(x.view(np.uint8), y.view(np.uint8))
    pn.BoundList([])(stream)                       # nothing to launch: a no-op


def test_overlapped_launches_keep_stream_order():
    """Generated kernels are launched so that their set-up overlaps the tail of the kernel before
    them in the stream, and wait at their head for it to complete: a producer of another library
    right before a launch, and a chain of two handles where the second reads what the first wrote,
    give the bits of plain stream order (PN_FLAG_PLAIN_LAUNCH)."""
    import torch
    from pn_workloads.descriptor import GraphBuilder, Imm
    M, N = 256, 4096
    def scale_graph(k):
        g = GraphBuilder(); x = g.input(D.F32, (M, N))
        g.mark_output(g.op("mul", [g.op("add", [x, Imm(1.0)], D.F32, (M, N)), Imm(k)], D.F32, (M, N)))
        return g.build()
    stream = torch.cuda.current_stream().cuda_stream
    results = {}
    for label, flags in (("overlapped", 0), ("plain", pn.FLAG_PLAIN_LAUNCH)):
        a, b = pn.Graph(scale_graph(0.5), 0, flags), pn.Graph(scale_graph(3.0), 0, flags)
        x = torch.zeros(M, N, device="cuda"); mid = torch.empty_like(x); out = torch.empty_like(x)
        fa, fb = a.bind([x.data_ptr()], [mid.data_ptr()]), b.bind([mid.data_ptr()], [out.data_ptr()])
        got = []
        for step in range(30):
            x.fill_(float(step))                  # a kernel of another library writes the input ...
            fa(stream); fb(stream)                # ... and the two launches follow at once, the second reading the first
            got.append(out[::37, ::129].clone())
        torch.cuda.synchronize()
        results[label] = torch.stack(got).cpu().numpy()
        for step in range(30):
            assert np.all(results[label][step] == np.float32((step + 1.0) * 0.5 + 1.0) * np.float32(3.0)), (label, step)
        a.close(); b.close()
    assert np.array_equal(results["overlapped"], results["plain"])
