"""What this GPU's memory system gives a kernel that only moves bytes: `pn_stream_probe` timed over
read : write mixes, loaders and access patterns.

    python -m paper_2605_29357_b200.probe            # the five mixes, then the pattern table
    python -m paper_2605_29357_b200.probe --mb 256   # array size per buffer

One JSON document on stdout.  The mixes are those of the fused kernels (a long-row reduction only
reads; softmax reads and writes the same amount; residual + LayerNorm reads twice what it writes;
...); the pattern table reads one array in the ways a fused kernel could walk it: one short-lived
block per piece in memory order, resident blocks striding over the array, resident blocks each
streaming through a range of their own, resident blocks taking runs in turn, bulk copies into a
shared-memory ring, and the strips of a reduction over a leading dimension.  Timing: 3 warm-up
launches, then the mean of `--reps` launches between two CUDA events (single launches are timed
in steps of a microsecond or two); arrays far larger than the L2.
"""
from __future__ import annotations

import argparse
import json
import sys

MIXES = (("read", 0, 16), ("write", 1, 16), ("1:1", 2, 32), ("2:1", 3, 48), ("4:3", 4, 56))   # name, code, bytes per unit


def main(argv=None) -> int:
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("--mb", type=int, default=256, help="MiB per array (default 256)")
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--device", type=int, default=0)
    args = ap.parse_args(argv)
    import torch
    from . import binding as B
    if not torch.cuda.is_available():
        print("no CUDA device", file=sys.stderr)
        return 1
    torch.cuda.set_device(args.device)
    units = args.mb * (1 << 20) // 16
    a = torch.randint(0, 255, (units * 16,), dtype=torch.uint8, device="cuda")
    b = torch.randint(0, 255, (units * 16,), dtype=torch.uint8, device="cuda")
    c = torch.empty(units * 16, dtype=torch.uint8, device="cuda")
    d = torch.empty(units * 8, dtype=torch.uint8, device="cuda")
    status = torch.zeros(16, dtype=torch.uint8, device="cuda")
    sms = torch.cuda.get_device_properties(args.device).multi_processor_count

    def rate(mix, cfg, n_units=units, unit_bytes=16):
        s = torch.cuda.current_stream().cuda_stream
        go = lambda: B.stream_probe(mix, cfg, a.data_ptr(), b.data_ptr(), c.data_ptr(), d.data_ptr(), n_units,
                                    status.data_ptr(), s)
        for _ in range(3):
            go()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.reps):
            go()
        e1.record()
        torch.cuda.synchronize()
        return round(n_units * unit_bytes / (e0.elapsed_time(e1) / args.reps) / 1e6, 1)

    P = B.ProbeConfig
    out = {"device": torch.cuda.get_device_name(args.device), "sms": sms, "mib_per_array": args.mb, "unit": "GB/s",
           "mixes": {}, "read_patterns": {}}
    for name, code, ub in MIXES:
        best = None
        for block, unroll in ((512, 2), (256, 2), (512, 1), (256, 4)):
            for cs in ((0,) if name == "read" else (0, 1)):
                if name == "write" and unroll > 2:
                    continue
                cfg = P(B.PROBE_LDG, cs, 0, block, unroll, (units + block * unroll - 1) // (block * unroll), 0, 0, 0, 0)
                r = rate(code, cfg, units, ub)
                if best is None or r > best["gbs"]:
                    best = {"gbs": r, "block": block, "unroll": unroll, "streaming_stores": cs}
        out["mixes"][name] = best
    pat = out["read_patterns"]
    for u in (2, 4):
        pat[f"one block per {256 * u * 16 // 1024} KB piece, in memory order"] = rate(0, P(0, 0, 0, 256, u, units // (256 * u), 0, 0, 0, 0))
    for per_sm in (3, 6, 8, 16):
        pat[f"{per_sm} resident blocks per SM striding over the array"] = rate(0, P(0, 0, 0, 256, 4, per_sm * sms, 0, 0, 0, 0))
    for per_sm in (3, 6, 8):
        pat[f"{per_sm} resident blocks per SM, a contiguous range each"] = rate(0, P(0, 0, 1, 256, 4, per_sm * sms, 0, 0, 0, 0))
    for run in (1024, 2048):
        pat[f"3 resident blocks per SM taking {run * 16 // 1024} KB runs in turn"] = rate(0, P(0, 0, 2, 256, 4, 3 * sms, 0, run, 0, 0))
    for stages, tile in ((4, 1024), (6, 1024), (4, 2048)):
        pat[f"bulk copies, ring of {stages} x {tile * 16 // 1024} KB, 3 blocks per SM"] = rate(0, P(B.PROBE_BULK, 0, 1, 256, 1, 3 * sms, stages, tile, 0, 0))
    pat["bulk copies, ring of 3 x 32 KB, 1 block of 512 per SM"] = rate(0, P(B.PROBE_BULK, 0, 1, 512, 1, sms, 3, 2048, 0, 0))
    # strips of a reduction over a leading dimension: the array as [groups, 512 rows, 128 units]
    row_units, rows = 128, 512
    groups = units // (row_units * rows)
    if groups:
        n = groups * row_units * rows
        for rs in (512, 128, 64, 16):
            for blk in (128, 256):
                pat[f"strips 512 B wide x {rs} rows, {blk} threads, 4 steps in flight"] = rate(
                    0, P(0, 0, 3, blk, 4, 0, 0, row_units, 32, rs), n)
    out["status_word"] = int(status.view(torch.int32)[0].item())
    print(json.dumps(out, indent=1))
    return 0 if out["status_word"] == 0 else 2


if __name__ == "__main__":
    sys.exit(main())
