"""pn_stream_probe: the bytes it writes are the bytes it read (so that the rate it reports is the
rate of a kernel that really moved them), for every mix and every way of loading, and the status
word of the bounded waits reads 0."""
import numpy as np
import pytest

from paper_2605_29357_b200 import binding as B

pytestmark = pytest.mark.gpu

LOADERS = {"ldg": dict(loader=B.PROBE_LDG, unroll=4, layout=0), "ldg_noalloc_ranges": dict(loader=B.PROBE_LDG_NOALLOC, unroll=2, layout=1),
           "bulk": dict(loader=B.PROBE_BULK, stages=3, tile_units=256, layout=1, unroll=1)}


@pytest.mark.parametrize("mix", [B.MIX_READ, B.MIX_WRITE, B.MIX_1_1, B.MIX_2_1, B.MIX_4_3])
@pytest.mark.parametrize("how", list(LOADERS))
@pytest.mark.parametrize("units", [1, 1000, 148 * 256 * 3 + 77])   # less than a tile, a ragged tail, several tiles per block
def test_probe_moves_the_bytes(mix, how, units):
    import torch
    if mix == B.MIX_WRITE and how == "bulk":
        pytest.skip("nothing to load")
    kw = LOADERS[how]
    cfg = B.ProbeConfig(kw["loader"], 1 if how == "bulk" else 0, kw["layout"], 128, kw["unroll"], 148, kw.get("stages", 0), kw.get("tile_units", 0))
    rng = np.random.default_rng(units)
    ha = rng.integers(0, 2**32, size=units * 4, dtype=np.uint32)
    hb = rng.integers(0, 2**32, size=units * 4, dtype=np.uint32)
    a = torch.from_numpy(ha.view(np.int32)).cuda()
    b = torch.from_numpy(hb.view(np.int32)).cuda()
    c = torch.full((units * 4 + 4,), -1, dtype=torch.int32, device="cuda")
    d = torch.full((units * 2 + 4,), -1, dtype=torch.int32, device="cuda")
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    B.stream_probe(mix, cfg, a.data_ptr(), b.data_ptr(), c.data_ptr(), d.data_ptr(), units, status.data_ptr(),
                   torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert int(status[0].item()) == 0
    got_c, got_d = c.cpu().numpy().view(np.uint32), d.cpu().numpy().view(np.uint32)
    x = {B.MIX_READ: ha, B.MIX_1_1: ha, B.MIX_2_1: ha ^ hb, B.MIX_4_3: ha ^ hb}.get(mix)
    if mix == B.MIX_WRITE:
        want = np.tile(np.array([0, 1, 2, 3], dtype=np.uint32), units)
        want[0::4] = 0
        # element 0 of a unit is the unroll slot it was written from: any value below the unroll count
        assert np.array_equal(got_c[:units * 4].reshape(-1, 4)[:, 1:], want.reshape(-1, 4)[:, 1:])
        assert (got_c[:units * 4].reshape(-1, 4)[:, 0] < 8).all()
    elif mix != B.MIX_READ:
        assert np.array_equal(got_c[:units * 4], x)
    if mix == B.MIX_4_3:
        q = x.reshape(-1, 4)
        assert np.array_equal(got_d[:units * 2].reshape(-1, 2), np.stack([q[:, 0] ^ q[:, 2], q[:, 1] ^ q[:, 3]], axis=1))
    else:
        assert (got_d == 0xFFFFFFFF).all()
    if mix == B.MIX_READ:
        assert (got_c == 0xFFFFFFFF).all()
    assert (got_c[units * 4:] == 0xFFFFFFFF).all() and (got_d[units * 2:] == 0xFFFFFFFF).all()   # nothing past the end


def test_probe_rejects_bad_configurations():
    import torch
    buf = torch.zeros(1024, dtype=torch.int32, device="cuda")
    p = buf.data_ptr()
    for cfg, mix in [(B.ProbeConfig(7, 0, 0, 128, 1, 1, 0, 0), B.MIX_1_1), (B.ProbeConfig(0, 0, 0, 100, 1, 1, 0, 0), B.MIX_1_1),
                     (B.ProbeConfig(0, 0, 0, 128, 3, 1, 0, 0), B.MIX_1_1), (B.ProbeConfig(2, 0, 1, 128, 1, 1, 16, 4096), B.MIX_2_1),
                     (B.ProbeConfig(2, 0, 1, 128, 1, 1, 3, 256), B.MIX_WRITE), (B.ProbeConfig(0, 0, 0, 128, 1, 1, 0, 0), 9)]:
        with pytest.raises(B.PnError):
            B.stream_probe(mix, cfg, p, p, p, p, 4, p, 0)
    with pytest.raises(B.PnError) as e:
        B.stream_probe(B.MIX_1_1, B.ProbeConfig(0, 0, 0, 128, 1, 1, 0, 0), p + 4, p, p, p, 4, p, 0)
    assert e.value.status == -6


def test_probe_command_line(capsys):
    """`python -m paper_2605_29357_b200.probe`: every mix and access pattern runs, the bounded waits
    of the bulk loader never run out, and a streaming read is far above anything a broken grid gives."""
    import json
    from paper_2605_29357_b200 import probe
    assert probe.main(["--mb", "64", "--reps", "3"]) == 0
    out = json.loads(capsys.readouterr().out)
    assert out["status_word"] == 0
    assert set(out["mixes"]) == {"read", "write", "1:1", "2:1", "4:3"}
    assert len(out["read_patterns"]) >= 20 and all(v > 100 for v in out["read_patterns"].values())
    assert out["mixes"]["read"]["gbs"] > 1000
