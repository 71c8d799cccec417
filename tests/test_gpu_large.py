"""Tensors of more than 2^31 elements (offsets that no longer fit 32 bits): a row kernel and a
pointwise kernel on [140000, 16384] bf16 (2.3 G elements, 4.6 GB per tensor), checked against the
oracle on sampled rows from the start, the middle, around the 2^31-element boundary and the end.
Rows are independent, so a sampled row is its own small problem for the oracle."""
import numpy as np
import pytest

import paper_2605_29357_b200 as pn
from oracle import evaluator as E
from pn_workloads import configs as C
from pn_workloads import descriptor as D
from pn_workloads.descriptor import GraphBuilder, Imm

pytestmark = pytest.mark.gpu

ROWS, N = 140000, 16384


def _graph(rows, with_reduction):
    g = GraphBuilder()
    x = g.input(D.BF16, (rows, N))
    xf = g.op("cast", [x], D.F32, (rows, N))
    y = g.op("fma", [g.op("gelu_tanh", [xf], D.F32, (rows, N)), Imm(0.5), xf], D.F32, (rows, N))
    g.mark_output(g.op("cast", [y], D.BF16, (rows, N)))
    if with_reduction:
        g.mark_output(g.op("sum", [y], D.F32, (rows,)))
        g.mark_output(g.op("argmax", [xf], D.I64, (rows,)))
    return g


@pytest.mark.parametrize("with_reduction", [False, True])
def test_offsets_beyond_32_bits(with_reduction):
    import torch
    if torch.cuda.mem_get_info()[0] < 16 * (1 << 30):
        pytest.skip("needs 16 GB of free device memory")
    assert ROWS * N > 2 ** 31
    gen = torch.Generator(device="cuda"); gen.manual_seed(7)
    x = torch.empty((ROWS, N), dtype=torch.bfloat16, device="cuda")
    for lo in range(0, ROWS, 20000):                     # drawn in slabs: bounded fp32 temporaries
        hi = min(ROWS, lo + 20000)
        x[lo:hi] = torch.randn((hi - lo, N), generator=gen, device="cuda").to(torch.bfloat16)
    g = _graph(ROWS, with_reduction)
    h = pn.Graph(g.build(), 0, 0)
    assert h.n_kernels == 1
    y = torch.full((ROWS, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    outs = [y]
    if with_reduction:
        outs += [torch.full((ROWS,), float("nan"), dtype=torch.float32, device="cuda"),
                 torch.full((ROWS,), -1, dtype=torch.int64, device="cuda")]
    h.run([x.data_ptr()], [t.data_ptr() for t in outs], torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    edge = 2 ** 31 // N                                   # the row in which element 2^31 lies
    rows = sorted({0, 1, 77, ROWS // 2, edge - 1, edge, edge + 1, ROWS - 2, ROWS - 1} | set(range(edge - 3, edge + 3)))
    idx = torch.tensor(rows, device="cuda")
    xs = x[idx].view(torch.int16).cpu().numpy().view(np.uint16)
    sub = _graph(len(rows), with_reduction)
    ref = E.evaluate(sub.build(), [xs])
    got = [y[idx].view(torch.int16).cpu().numpy().view(np.uint16)]
    if with_reduction:
        got += [outs[1][idx].cpu().numpy(), outs[2][idx].cpu().numpy()]
    for a, r, t in zip(got, ref, sub.output_ids()):
        dt, _ = sub.tensor_meta(t)
        res = E.compare(E.widen(a, dt), r, dt)
        assert res["ok"], res
    assert not torch.isnan(y).any().item()                # every element of the large output was written
    if with_reduction:
        assert not torch.isnan(outs[1]).any().item() and (outs[2] >= 0).all().item()
