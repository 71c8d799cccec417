"""GPU tests of the sequence calls (many small evaluations replayed with one launch): a
recorded sequence reproduces what the same handles give when run one by one, against the
oracle, for chained items (the output of one is the input of the next), for independent items
on parallel branches, and for unfused handles; refusals are reported, not executed."""
import numpy as np
import pytest

import paper_2605_29357_b200 as pn
from oracle import evaluator as E
from pn_workloads import configs as C
from pn_workloads import descriptor as D
from pn_workloads.descriptor import GraphBuilder, Imm

from gpu_util import device_bytes, poisoned

pytestmark = pytest.mark.gpu

ALL = {**C.CONFIGS, **C.EXTENDED}


def _buffers(w):
    d_in = [device_bytes(a) for a in w.inputs]
    sizes = [D.DTYPE_BYTES[dt] * int(np.prod(dims, dtype=np.int64)) for dt, dims in w.output_meta]
    d_out = [poisoned(s) for s in sizes]
    return d_in, d_out, sizes


def _check(w, d_out, sizes):
    ref = E.evaluate(w.desc, w.inputs)
    for t, (dt, dims), s, r, name in zip(d_out, w.output_meta, sizes, ref, w.output_names):
        got = E.widen(t.cpu().numpy()[:s].view(C.NP_STORAGE[dt]).reshape(dims), dt)
        res = E.compare(got, r, dt)
        assert res["ok"], (w.name, name, res)


@pytest.mark.parametrize("independent", [False, True])
@pytest.mark.parametrize("flags", [0, pn.FLAG_INTERPRET, pn.FLAG_UNFUSED])
def test_sequence_of_the_small_subgraphs_matches_the_oracle(flags, independent):
    import torch
    ws = [ALL[name](**C.SMALL[name]) for name in ALL] + [C.c1(M=3, N=64, seed=5), C.c3(M=2, N=256, seed=6)]
    graphs = [pn.Graph(w.desc, 0, flags) for w in ws]
    bufs = [_buffers(w) for w in ws]
    items = [(g, [t.data_ptr() for t in b[0]], [t.data_ptr() for t in b[1]]) for g, b in zip(graphs, bufs)]
    seq = pn.Sequence(items, independent=independent)
    assert seq.n_items == len(ws) and seq.n_kernels == sum(g.n_kernels for g in graphs)
    stream = torch.cuda.Stream()
    for _ in range(2):                                  # a replay overwrites every output again
        for b in bufs:
            for t in b[1]:
                t.fill_(0xFF)
        torch.cuda.synchronize()
        seq.run(stream.cuda_stream)
        stream.synchronize()
        for w, b in zip(ws, bufs):
            _check(w, b[1], b[2])
    seq.close()


def test_chained_items_run_in_order():
    """Item k reads what item k-1 wrote: y0 = x + 1, y1 = 2 * y0, y2 = y1 - 3, ..., through the
    same two handles used several times with different pointers."""
    import torch
    n = 4096
    ga = GraphBuilder(); xa = ga.input(D.F32, (n,)); ga.mark_output(ga.op("add", [xa, Imm(1.0)], D.F32, (n,)))
    gm = GraphBuilder(); xm = gm.input(D.F32, (n,)); gm.mark_output(gm.op("mul", [xm, Imm(2.0)], D.F32, (n,)))
    ha, hm = pn.Graph(ga.build(), 0, 0), pn.Graph(gm.build(), 0, 0)
    x = np.arange(n, dtype=np.float32)
    bufs = [torch.from_numpy(x).cuda()] + [torch.full((n,), float("nan"), device="cuda") for _ in range(6)]
    items = [(ha if k % 2 == 0 else hm, [bufs[k].data_ptr()], [bufs[k + 1].data_ptr()]) for k in range(6)]
    seq = pn.Sequence(items)
    seq.run(torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    want = x.copy()
    for k in range(6):
        want = want + 1 if k % 2 == 0 else want * 2
        assert np.array_equal(bufs[k + 1].cpu().numpy(), want)


def test_refusals():
    w = C.c3(**C.SMALL["c3"])
    g = pn.Graph(w.desc, 0, 0)
    d_in, d_out, sizes = _buffers(w)
    ins, outs = [t.data_ptr() for t in d_in], [t.data_ptr() for t in d_out]
    with pytest.raises(pn.PnError) as e:
        pn.Sequence([(g, ins[:-1], outs)])
    assert e.value.status == -7 and "item 0" in str(e.value)          # wrong operand count, named item
    with pytest.raises(pn.PnError) as e:
        pn.Sequence([(g, ins, outs), (g, [ins[0] + 2] + ins[1:], outs)])
    assert e.value.status == -6 and "item 1" in str(e.value)          # misaligned pointer
    with pytest.raises(pn.PnError) as e:
        pn.Sequence([])
    assert e.value.status == -1
    gu = pn.Graph(w.desc, 0, pn.FLAG_UNFUSED)
    with pytest.raises(pn.PnError) as e:
        pn.Sequence([(gu, ins, outs), (gu, ins, outs)], independent=True)
    assert e.value.status == -1                                        # two runs would share one workspace
    pn.Sequence([(gu, ins, outs), (gu, ins, outs)]).close()            # in order they may
    # a failed create leaves the device usable
    seq = pn.Sequence([(g, ins, outs)])
    import torch
    seq.run(torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    _check(w, d_out, sizes)
