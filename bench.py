#!/usr/bin/env python
"""Benchmark of the fused-subgraph path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-sweep]

A step is one pass of the whole fused path (one pn_graph_run) over one batch of the masked
scaled softmax workload (bf16 scores [512,512,512], int8 causal mask, fp32 math): the
workload the headline metric is quoted on.  The metric is effective HBM GB/s on compulsory
bytes (every graph input read once + every output written once).  With N > 1 every rank
runs its own batch (rows are independent: no collective on the data path), so scaling is
weak and the value is the sum over ranks divided by the slowest rank's time.

One JSON line is printed by rank 0.  Beside the base keys it carries `roofline` (the fused
kernel against the measured HBM copy rate), `e2e` (the same metric through
pn_graph_run_host on pinned host buffers, copies inside the timed region),
`cpu_baseline` (the CPU oracle timed over the host's cores on the same workload) and, at
N = 1 unless --no-sweep, `mix_peaks` (the stream probe's ceilings), `sweep` (the other six
subgraphs, fused and unfused, each with its own roofline object), `tiny_graphs` (launch latency
of many small subgraphs) and `create_ms` (what creating a handle costs, with and without the
kernel caches).  With --gpus N > 1 and no launcher around it, the script starts its own N ranks.

--impl reference times the CPU oracle itself, as it stands, on the host cores.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from pn_workloads import configs as C  # noqa: E402
from pn_workloads import descriptor as D  # noqa: E402

METRIC = "fused-subgraph effective HBM GB/s on compulsory bytes"
WORKLOAD = "c2 masked scaled softmax: bf16 scores [512,512,512], int8 causal mask [512,512], fp32 math, bf16 out"
FALLBACK_HBM_GBS = 6650.0


def kernel_identity(g):
    """Name of the generated kernel of a fused handle (it carries a hash of the program) and a
    hash of the device library it is compiled against."""
    import hashlib
    import re
    m = re.search(r"__global__ void PN_LAUNCH_BOUNDS (\w+)\(", g.codegen(0))
    name = m.group(1) if m else "interpreter"
    lib = os.path.join(ROOT, "paper_2605_29357_b200", "csrc", "device_lib.cuh")
    with open(lib, "rb") as f:
        return name, hashlib.sha256(f.read()).hexdigest()[:16]


def recorded_traffic(name, lib_hash):
    """DRAM bytes (read + write) per launch of that kernel from the ncu capture summarised in
    profiles/; None when the kernel or the device library has changed since."""
    try:
        with open(os.path.join(ROOT, "profiles", "dram_traffic.txt")) as f:
            rec = json.load(f).get(name)
        if rec and rec.get("device_lib_sha256_16") == lib_hash:
            return rec["dram_bytes_read"] + rec["dram_bytes_write"]
    except Exception:
        pass
    return None


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (earlier pool measurement)"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap,clocks.mem")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, mx, mem, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
            try:
                mem.append(float(f[6]))
            except (IndexError, ValueError):
                pass
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "mem_mhz": float(np.median(mem)) if mem else None, "samples": len(sm), "reasons": sorted(reasons)}


def driver_version():
    try:
        out = subprocess.run(["nvidia-smi", "--query-gpu=driver_version", "--format=csv,noheader"], capture_output=True, text=True, timeout=20)
        return out.stdout.strip().splitlines()[0]
    except Exception:
        return None


def nbytes_of(meta):
    return [D.DTYPE_BYTES[dt] * int(np.prod(dims, dtype=np.int64)) for dt, dims in meta]


def device_sets(torch, w, n_sets):
    """n_sets distinct copies of the inputs and outputs on the device."""
    sets = []
    host = [np.ascontiguousarray(a).reshape(-1).view(np.uint8) for a in w.inputs]
    for _ in range(n_sets):
        d_in = [torch.from_numpy(h).cuda() for h in host]
        d_out = [torch.full((s,), 0xFF, dtype=torch.uint8, device="cuda") for s in nbytes_of(w.output_meta)]
        sets.append((d_in, d_out))
    return sets


def time_graph(torch, g, sets, steps, warmup, flush=None):
    """W untimed + K timed launches rotating over the buffer sets.  Returns (total ms over the
    K steps by CUDA events on the launch stream, per-step ms list)."""
    stream = torch.cuda.current_stream()
    launch = [g.bind([t.data_ptr() for t in a], [t.data_ptr() for t in b]) for a, b in sets]   # pointers marshalled once
    for i in range(warmup):
        launch[i % len(launch)](stream.cuda_stream)
    torch.cuda.synchronize()
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    evs[0].record(stream)
    for i in range(steps):
        if flush is not None:
            flush.add_(1)
        launch[i % len(launch)](stream.cuda_stream)
        evs[i + 1].record(stream)
    torch.cuda.synchronize()
    per = [evs[i].elapsed_time(evs[i + 1]) for i in range(steps)]
    return evs[0].elapsed_time(evs[steps]), per


def time_back_to_back(torch, g, sets, steps):
    """Exactly `steps` launches, one after the other on the launch stream, between two CUDA events:
    the timed region.  Nothing else is enqueued in between (an event record after every launch keeps
    one launch's tail from overlapping the next one's start, which a job that simply runs its steps
    does not pay).  Returns the total in ms."""
    stream = torch.cuda.current_stream()
    launch = [g.bind([t.data_ptr() for t in a], [t.data_ptr() for t in b]) for a, b in sets]
    n, s = len(launch), stream.cuda_stream
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(steps):
        launch[i % n](s)
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1)


def time_host_launched(torch, g, sets, steps, warmup):
    """Launches through bound launch objects (pn_bound_run: one launch call each) rotating over the
    buffer sets, one pair of events around all of them: what a caller who launches from the host
    pays per launch, without an event record between the launches.  At least 2000 launches: host
    and device run at nearly the same rate here (an empty kernel takes 2.9 us per launch on the
    same box), so a short run measures the start of the queue rather than its steady state.
    Returns ms per launch."""
    steps = max(steps, 2000)
    stream = torch.cuda.current_stream()
    launch = [g.bind([t.data_ptr() for t in a], [t.data_ptr() for t in b]) for a, b in sets]
    for i in range(max(warmup, 3)):
        launch[i % len(launch)](stream.cuda_stream)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n, s = len(launch), stream.cuda_stream
    e0.record(stream)
    for i in range(steps):
        launch[i % n](s)
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps


def time_graph_replay(torch, g, sets, steps, warmup):
    """The same launches recorded once into a CUDA graph (one launch per buffer set) and
    replayed: the device-side time per launch, free of the host's launch rate.  Used for the
    workloads whose kernels are shorter than a host launch.  Returns ms per launch."""
    ptrs = [([t.data_ptr() for t in a], [t.data_ptr() for t in b]) for a, b in sets]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for i in range(max(warmup, 3)):
            g.run(*ptrs[i % len(ptrs)], side.cuda_stream)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        for a, b in ptrs:
            g.run(a, b, torch.cuda.current_stream().cuda_stream)
    reps = max(1, steps // len(ptrs))
    graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / (reps * len(ptrs))


# read : write mix of each workload's compulsory traffic, as pn_stream_probe names them
MIX_OF = {"c1": "2:1", "c2": "1:1", "c3": "2:1", "c4": "read", "c5": "4:3", "n1": "1:1", "n2": "read"}
MIX_CODE = {"read": 0, "write": 1, "1:1": 2, "2:1": 3, "4:3": 4}
MIX_UNIT_BYTES = {"read": 16, "write": 16, "1:1": 32, "2:1": 48, "4:3": 56}   # bytes moved per 16-byte unit of an array


class StreamProbe:
    """The bandwidth ceiling of a read : write mix: pn_stream_probe (a hand-written kernel that only
    moves bytes, 128-bit accesses) timed by the same protocol as the fused kernels.  `large`: arrays
    of 512 MiB each, far beyond the L2.  `at_size`: the same total bytes per launch as a small
    workload, rotating over distinct ranges of the arrays that together exceed twice the L2,
    replayed back to back from a CUDA graph -- what launch, ramp and tail leave of the ceiling
    at that size."""
    ARRAY_BYTES = 512 << 20

    def __init__(self, torch, l2_bytes):
        from paper_2605_29357_b200 import binding as B
        self.torch, self.B, self.l2 = torch, B, l2_bytes
        n = self.ARRAY_BYTES
        self.a = torch.randint(0, 255, (n,), dtype=torch.uint8, device="cuda")
        self.b = torch.randint(0, 255, (n,), dtype=torch.uint8, device="cuda")
        self.c = torch.empty(n, dtype=torch.uint8, device="cuda")
        self.d = torch.empty(n // 2, dtype=torch.uint8, device="cuda")
        self.status = torch.zeros(16, dtype=torch.uint8, device="cuda")
        self.cache = {}

    def _configs(self, mix, units):
        out = []
        for block, unroll in ((512, 2), (256, 2), (512, 1), (256, 4)):
            for cs in ((0,) if mix == "read" else (0, 1)):
                if mix == "write" and unroll > 2:
                    continue
                grid = max(1, (units + block * unroll - 1) // (block * unroll))
                out.append(self.B.ProbeConfig(self.B.PROBE_LDG, cs, 0, block, unroll, int(grid), 0, 0))
        return out

    def _launch(self, mix, cfg, units, k, stream):
        off = k * units * 16
        self.B.stream_probe(MIX_CODE[mix], cfg, self.a.data_ptr() + off, self.b.data_ptr() + off, self.c.data_ptr() + off,
                            self.d.data_ptr() + off // 2, units, self.status.data_ptr(), stream)

    def large(self, mix, reps=10):
        if ("large", mix) in self.cache:
            return self.cache[("large", mix)]
        torch = self.torch
        units = self.ARRAY_BYTES // 16
        s = torch.cuda.current_stream()
        best = None
        for cfg in self._configs(mix, units):
            for _ in range(3):
                self._launch(mix, cfg, units, 0, s.cuda_stream)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(s)
            for i in range(reps):
                self._launch(mix, cfg, units, 0, s.cuda_stream)
            e1.record(s)
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / reps   # (single launches are timed in steps of a microsecond or two: take the mean)
            gbs = units * MIX_UNIT_BYTES[mix] / (ms * 1e-3) / 1e9
            if best is None or gbs > best["gbs"]:
                best = {"gbs": gbs, "block": cfg.block, "unroll": cfg.unroll, "streaming_stores": cfg.streaming_stores,
                        "bytes_per_launch": units * MIX_UNIT_BYTES[mix]}
        self.cache[("large", mix)] = best
        return best

    def at_size(self, mix, total_bytes, reps=20):
        torch = self.torch
        units = max(1, int(total_bytes) // MIX_UNIT_BYTES[mix])
        n_sets = int(min(self.ARRAY_BYTES // (units * 16), 2 * self.l2 // max(1, units * MIX_UNIT_BYTES[mix]) + 2))
        best = None
        side = torch.cuda.Stream()
        for cfg in self._configs(mix, units):
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                for k in range(min(3, n_sets)):
                    self._launch(mix, cfg, units, k, side.cuda_stream)
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                for k in range(n_sets):
                    self._launch(mix, cfg, units, k, torch.cuda.current_stream().cuda_stream)
            graph.replay()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                graph.replay()
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / (reps * n_sets)
            gbs = units * MIX_UNIT_BYTES[mix] / (ms * 1e-3) / 1e9
            if best is None or gbs > best["gbs"]:
                best = {"gbs": gbs, "us_per_launch": ms * 1e3, "block": cfg.block, "unroll": cfg.unroll,
                        "streaming_stores": cfg.streaming_stores, "bytes_per_launch": units * MIX_UNIT_BYTES[mix], "buffer_sets": n_sets}
            del graph
        return best

    def status_word(self):
        return int(self.status.view(self.torch.int32)[0].item())


def roofline_entry(cbytes, seconds, peak, peak_src, mix, probe, small):
    """The roofline object of one fused kernel: achieved GB/s on its algorithmic bytes against the
    measured copy rate, and against the stream-probe ceiling of its own read : write mix."""
    achieved = cbytes / seconds / 1e9
    out = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak, "peak_source": peak_src,
           "algorithmic_bytes_per_launch": int(cbytes), "mix": mix}
    if probe is not None:
        mp = probe.large(mix)
        out["mix_peak"] = mp["gbs"]
        out["frac_of_mix_peak"] = achieved / mp["gbs"]
        if small:
            sp = probe.at_size(mix, cbytes)
            out["mix_peak_at_this_size"] = sp["gbs"]
            out["frac_of_mix_peak_at_this_size"] = achieved / sp["gbs"]
    return out


def tiny_graph_latency(torch, pn, device, passes, repeats=8):
    """Latency of many small subgraphs run back to back (the regime where the paper finds fixed
    per-call overhead decisive): the reduced-size graphs of every workload, `repeats` instances
    each on their own buffers, (a) launched one by one from the host through bound launches (pn_bound_run
    from a Python loop, and pn_bound_run_many: the same launches issued by one call),
    (b) recorded once as a sequence and replayed in order, (c) the same as independent items.
    Returns microseconds per subgraph for each; the inputs are L2-resident, so this is launch
    and latency, not bandwidth."""
    makers = {**C.CONFIGS, **C.EXTENDED}
    graphs, items, keep = {}, [], []
    for rep in range(repeats):
        for name, make in makers.items():
            w = make(seed=rep, **C.SMALL[name])
            if name not in graphs:
                graphs[name] = pn.Graph(w.desc, device, 0)
            (d_in, d_out), = device_sets(torch, w, 1)
            keep.append((d_in, d_out))
            items.append((graphs[name], [t.data_ptr() for t in d_in], [t.data_ptr() for t in d_out]))
    stream = torch.cuda.current_stream()

    def timed(run_pass):
        for _ in range(3):
            run_pass()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(passes):
            run_pass()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / (passes * len(items))

    bound = [g.bind(i, o) for g, i, o in items]
    many = pn.BoundList(bound)

    def host_pass():
        for f in bound:
            f(stream.cuda_stream)

    def host_pass_one_call():
        many(stream.cuda_stream)

    out = {"subgraphs": len(items), "distinct_graphs": len(graphs), "kernels_per_pass": sum(g.n_kernels for g, _, _ in items),
           "host_launched_us_per_subgraph": timed(host_pass), "host_launched_one_call_us_per_subgraph": timed(host_pass_one_call)}
    for key, indep in (("sequence_us_per_subgraph", False), ("sequence_independent_us_per_subgraph", True)):
        seq = pn.Sequence(items, independent=indep)
        out[key] = timed(lambda: seq.run(stream.cuda_stream))
        seq.close()
    for g in graphs.values():
        g.close()
    return out


def create_times(device):
    """What pn_graph_create costs, on the unfused handle of the gated multi-output graph (13 nodes, a
    kernel each, every one compiled by NVRTC): in a fresh process with an empty on-disk kernel cache
    (PN_CACHE_DIR), a second time in that process (the process-wide kernel cache), and in another
    fresh process that finds the cubins on disk.  Milliseconds; the device context is brought up
    first by an interpreter handle (no compilation) and reported apart.  The processes load only
    the library, not torch."""
    import tempfile
    code = ("import json, time\nimport paper_2605_29357_b200 as pn\nfrom pn_workloads import configs as C\n"
            "w = C.c5(**C.SMALL['c5'])\nout = []\n"
            "t0 = time.perf_counter(); pn.Graph(C.c1(M=4, N=64).desc, %d, pn.FLAG_INTERPRET).close(); init = (time.perf_counter() - t0) * 1e3\n"
            "for _ in range(2):\n"
            "    t0 = time.perf_counter(); g = pn.Graph(w.desc, %d, pn.FLAG_UNFUSED); out.append((time.perf_counter() - t0) * 1e3)\n"
            "    n = g.n_kernels\n"
            "print(json.dumps({'ms': out, 'kernels': n, 'cache': list(g.kernel_cache), 'init': init}))\n" % (device, device))
    with tempfile.TemporaryDirectory() as d:
        env = dict(os.environ, PN_CACHE_DIR=d, PYTHONPATH=ROOT + os.pathsep + os.environ.get("PYTHONPATH", ""))
        runs = []
        for _ in range(2):
            r = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=300, cwd=ROOT)
            if r.returncode != 0:
                return {"error": (r.stderr or r.stdout).strip()[-300:]}
            runs.append(json.loads(r.stdout.strip().splitlines()[-1]))
        files = len(os.listdir(d))
    return {"graph": "c5 unfused", "kernels": runs[0]["kernels"], "device_context_ms": runs[0]["init"], "compiled_ms": runs[0]["ms"][0], "again_in_process_ms": runs[0]["ms"][1],
            "from_disk_cache_ms": runs[1]["ms"][0], "cubins_on_disk": files}


def rank_workload(name, rank, **size):
    """The batch rank `rank` works on: the same graph and shapes on every rank, inputs drawn
    from the rank's own seed.  Rows are independent, so sharding a larger job by rows needs no
    exchange between ranks at all."""
    return {**C.CONFIGS, **C.EXTENDED}[name](seed=rank, **size)


def max_over_ranks(x, world, device):
    """The slowest rank's time: what a whole-job throughput has to be divided by."""
    import torch
    t = torch.tensor([float(x)], device=device, dtype=torch.float64)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(world, bytes_per_rank, seconds_per_step):
    """Whole-job GB/s: the bytes all ranks moved in a step over the slowest rank's step time."""
    return world * bytes_per_rank / seconds_per_step / 1e9


def stats(per):
    a = np.sort(np.asarray(per))
    q1, med, q3 = np.percentile(a, [25, 50, 75])
    return {"median_ms": float(med), "min_ms": float(a[0]), "iqr_ms": float(q3 - q1)}


def oracle_sample(rows_b):
    """A bounded sample of the benchmark workload for the CPU oracle: rows_b of the 512 batches."""
    return C.c2(B=rows_b)


_C2_DESC = {}


def _c2_descriptor(b, q, k):
    """Descriptor of the benchmark graph for b batches (cached; descriptors depend on shapes only)."""
    key = (b, q, k)
    if key not in _C2_DESC:
        real = C._draw
        C._draw = lambda rng, kind, shape, a, bb, chunk=0: np.zeros(shape, dtype=np.float32)
        try:
            _C2_DESC[key] = C.c2(B=b, Q=q, K=k).desc
        finally:
            C._draw = real
    return _C2_DESC[key]


def _oracle_job(job):
    """One block of batches through the oracle (runs in a worker process)."""
    from oracle import evaluator as E
    desc, scores, mask = job
    E.evaluate(desc, [scores, mask])
    return scores.shape[0]


def _oracle_warm(_):
    from oracle import evaluator as E  # noqa: F401
    return os.getpid()


class OraclePool:
    """The CPU oracle, as it stands, over the host's cores: the batches of the benchmark workload are
    independent, so blocks of them are handed to worker processes (started with `spawn`, so that
    nothing of a CUDA context is inherited).  Each worker runs the oracle's own single-threaded
    NumPy evaluation on its block; `cores` is the number of workers."""

    def __init__(self, workers=None):
        import multiprocessing as mp
        self.cores = int(workers or os.cpu_count() or 1)
        self.pool = mp.get_context("spawn").Pool(self.cores)
        self.pids = set(self.pool.map(_oracle_warm, range(4 * self.cores)))

    def seconds(self, sample, block):
        """Wall-clock time of one evaluation of the whole sample, `block` batches per job."""
        scores, mask = sample.inputs
        jobs = [(_c2_descriptor(min(block, scores.shape[0] - lo), scores.shape[1], scores.shape[2]), scores[lo:lo + block], mask)
                for lo in range(0, scores.shape[0], block)]
        t0 = time.perf_counter()
        done = sum(self.pool.map(_oracle_job, jobs, chunksize=1))
        dt = time.perf_counter() - t0
        assert done == scores.shape[0]
        return dt

    def close(self):
        self.pool.close()
        self.pool.join()


def cpu_model():
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("model name"):
                    return line.split(":", 1)[1].strip()
    except Exception:
        pass
    return None


REF_BATCHES = 128   # batches of the 512 that one step of the reference arm evaluates


def run_reference(args, rank):
    """--impl reference: the CPU oracle, as it stands, on a bounded sample per step, its
    independent batches spread over the host's cores."""
    if rank != 0:
        return
    sample = oracle_sample(REF_BATCHES)
    pool = OraclePool()
    warm = min(args.warmup, 3)
    for _ in range(warm):
        pool.seconds(sample, 8)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        pool.seconds(sample, 8)
    dt = (time.perf_counter() - t0) / args.steps
    pool.close()
    gbs = sample.compulsory_bytes / dt / 1e9
    what = f"{REF_BATCHES} of the 512 batches per step ({REF_BATCHES * 512 * 512 / 1e6:.1f} M elements), 8 batches per job"
    line = {"impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": warm, "ms_per_step": dt * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "sample": what},
            "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": pool.cores, "kind": "oracle", "sample": what,
                             "cpu_model": cpu_model(), "host_cores": os.cpu_count()},
            "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def torchrun_command(n, argv, port):
    """The launch of n ranks of this script on this node, one per GPU, as a list of arguments."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def free_port():
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--workload", default="c2", choices=list(C.CONFIGS) + list(C.EXTENDED))
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # not under a launcher yet: start one process per GPU and let rank 0 of them report.  NCCL's
        # own start-up lines (stderr) show the communicator and its ranks.
        env = dict(os.environ)
        env.setdefault("NCCL_DEBUG", "INFO")
        env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
        raise SystemExit(subprocess.call(torchrun_command(args.gpus, sys.argv[1:], free_port()), env=env))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        if args.steps > 20:
            args.steps = 20
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist
    import paper_2605_29357_b200 as pn

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    warmup = max(args.warmup, 3)

    # ---- the benchmark workload: one batch per rank, seed = rank ---------------------------
    w = rank_workload(args.workload, rank)
    g = pn.Graph(w.desc, local_rank, 0)
    info = g.kernel_info[0]
    cbytes = g.compulsory_bytes
    l2 = torch.cuda.get_device_properties(local_rank).L2_cache_size
    n_sets = 1 if cbytes > 2 * l2 else int(2 * l2 // cbytes) + 2
    sets = device_sets(torch, w, n_sets)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    time_graph(torch, g, sets, 3, warmup)     # warm-up (and first-launch costs)
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    # the timed region: exactly K steps back to back, a barrier and a synchronize on both sides
    total_ms = time_back_to_back(torch, g, sets, args.steps)
    barrier()
    # the paper's protocol beside it: every launch between its own pair of events, the median of
    # the timed runs, measured again (up to three times in all) while the interquartile range
    # exceeds 20 % of the median
    reruns = 0
    while True:
        _, per = time_graph(torch, g, sets, args.steps, 0)
        st_try = stats(per)
        if st_try["iqr_ms"] <= 0.2 * st_try["median_ms"] or reruns >= 2:
            break
        reruns += 1
    barrier()
    # K steps of this workload last only milliseconds, less than one nvidia-smi sample: keep
    # the same step running (untimed) until the sampler has seen the GPU under this load
    if rank == 0:
        t_end = time.perf_counter() + 1.0
        while time.perf_counter() < t_end:
            time_graph(torch, g, sets, 50, 0)
    clocks = sampler.stop() if rank == 0 else None
    total_ms = max_over_ranks(total_ms, world, "cuda")
    ms_per_step = total_ms / args.steps
    value = job_value(world, cbytes, ms_per_step * 1e-3)

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region -----
    pin_in = [torch.from_numpy(np.ascontiguousarray(a).reshape(-1).view(np.uint8)).pin_memory() for a in w.inputs]
    pin_out = [torch.empty(s, dtype=torch.uint8).pin_memory() for s in nbytes_of(w.output_meta)]
    e2e_steps = max(3, min(args.steps, 10))
    stream = torch.cuda.current_stream().cuda_stream
    for _ in range(2):
        g.run_host([t_.data_ptr() for t_ in pin_in], [t_.data_ptr() for t_ in pin_out], stream)
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        g.run_host([t_.data_ptr() for t_ in pin_in], [t_.data_ptr() for t_ in pin_out], stream)
    torch.cuda.synchronize()
    e2e_s = (time.perf_counter() - t0) / e2e_steps
    e2e_s = max_over_ranks(e2e_s, world, "cuda")
    h2d = int(sum(a.nbytes for a in w.inputs))
    d2h = int(sum(nbytes_of(w.output_meta)))

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_src = measured_peak()
    kname, lib_hash = kernel_identity(g)
    st = stats(per)
    probe = StreamProbe(torch, l2)
    roof = roofline_entry(cbytes, ms_per_step * 1e-3, peak, peak_src, MIX_OF.get(args.workload, "1:1"), probe, n_sets > 1)
    roof["timing"] = "K launches back to back between two CUDA events (the timed region), mean per launch"
    roof.update({"traffic": recorded_traffic(kname, lib_hash), "kernel": kname, "device_lib_sha256_16": lib_hash,
                 "specialised": bool(info["specialised"])})
    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD if args.workload == "c2" else w.name, "compulsory_bytes": cbytes,
                   "l2": "inputs larger than L2" if n_sets == 1 else f"{n_sets} rotating buffer sets larger than 2x L2",
                   "family": pn.FAMILY_NAMES[info["family"]], "grid": info["grid"], "block": info["block"],
                   "cluster": info["cluster"], "tile": [info["vl"], info["ng"]], "kernels": g.n_kernels,
                   "nodes": g.n_nodes, "per_step": st, "reruns_for_iqr": reruns, "pct_of_8000": 100 * value / world / 8000.0,
                   "gpu": torch.cuda.get_device_name(local_rank), "driver": driver_version(), "cuda": torch.version.cuda},
        "clocks": clocks,
        "gpu_launches": args.steps * g.n_kernels,
        "e2e": {"value": job_value(world, cbytes, e2e_s), "unit": "GB/s", "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": e2e_s * 1e3, "steps": e2e_steps},
        "roofline": roof,
        # the ceiling of every read : write mix on this GPU in this run, beside the copy rate
        "mix_peaks": {m: probe.large(m) for m in MIX_CODE},
    }

    # ---- the unfused path of the same library on the same workload ---------------------------
    try:
        gu = pn.Graph(w.desc, local_rank, pn.FLAG_UNFUSED)
        _, per_u = time_graph(torch, gu, sets, max(5, args.steps // 5), 3)
        su = stats(per_u)
        line["unfused"] = {"kernels": gu.n_kernels, "median_ms": su["median_ms"],
                           "speedup_fused_over_unfused": su["median_ms"] / st["median_ms"]}
        gu.close()
    except Exception as e:  # report, do not hide
        line["unfused"] = {"error": str(e)}
    del sets
    torch.cuda.empty_cache()

    # ---- the other benchmark subgraphs (N = 1 only) ------------------------------------------
    if world == 1 and not args.no_sweep:
        sweep = {}
        for name, make in {**C.CONFIGS, **C.EXTENDED}.items():
            if name == args.workload:
                continue
            wi = make()
            gi = pn.Graph(wi.desc, local_rank, 0)
            cb = int(wi.notes.get("touched_bytes", gi.compulsory_bytes))
            ns = 1 if cb > 2 * l2 else int(2 * l2 // cb) + 2
            si = device_sets(torch, wi, ns)
            _, pi = time_graph(torch, gi, si, args.steps, warmup)
            sti = stats(pi)
            ki = gi.kernel_info[0]
            entry = {"compulsory_bytes": cb, "median_ms": sti["median_ms"], "min_ms": sti["min_ms"],
                     "iqr_ms": sti["iqr_ms"], "gbs": cb / (sti["median_ms"] * 1e-3) / 1e9,
                     "frac_of_measured_peak": cb / (sti["median_ms"] * 1e-3) / 1e9 / peak,
                     "family": pn.FAMILY_NAMES[ki["family"]], "buffer_sets": ns}
            if ns == 1:   # as the headline: K launches back to back between two events
                entry["back_to_back_ms"] = time_back_to_back(torch, gi, si, args.steps) / args.steps
                entry["gbs"] = cb / (entry["back_to_back_ms"] * 1e-3) / 1e9
                entry["frac_of_measured_peak"] = entry["gbs"] / peak
            ms_roof, timing = entry.get("back_to_back_ms", sti["median_ms"]), "K launches back to back between two CUDA events, mean per launch"
            if ns > 1:   # kernels shorter than a host launch: also the device-side time per launch
                ms_r = time_graph_replay(torch, gi, si, max(args.steps, 10 * ns), warmup)
                entry["host_launched_ms"] = time_host_launched(torch, gi, si, max(200, args.steps), warmup)
                entry["graph_replay_ms"] = ms_r
                entry["graph_replay_gbs"] = cb / (ms_r * 1e-3) / 1e9
                entry["graph_replay_frac_of_measured_peak"] = entry["graph_replay_gbs"] / peak
                ms_roof, timing = ms_r, "CUDA-graph replay over the rotating buffer sets, mean per launch"
            entry["roofline"] = roofline_entry(cb, ms_roof * 1e-3, peak, peak_src, MIX_OF[name], probe, ns > 1)
            kn_i, _ = kernel_identity(gi)
            entry["roofline"].update({"timing": timing, "kernel": kn_i, "traffic": recorded_traffic(kn_i, lib_hash)})
            try:
                gui = pn.Graph(wi.desc, local_rank, pn.FLAG_UNFUSED)
                _, pu = time_graph(torch, gui, si, max(5, args.steps // 5), 3)
                entry["unfused_kernels"] = gui.n_kernels
                entry["unfused_median_ms"] = stats(pu)["median_ms"]
                entry["speedup_fused_over_unfused"] = entry["unfused_median_ms"] / sti["median_ms"]
                gui.close()
            except Exception as e:
                entry["unfused_error"] = str(e)
            sweep[name] = entry
            gi.close()
            del si
            torch.cuda.empty_cache()
        # supplementary: the two small graphs scaled up until their inputs exceed the L2, to show their
        # kernels' bandwidth once launch, ramp and tail no longer dominate (not benchmark configs)
        # ... and a gated activation read from the two halves of one tensor (two slices of the last
        # dimension of one input, folded into the addressing)
        for name, make, mix in (("c1_scaled_8192x8192", lambda: C.c1(M=8192, N=8192), "2:1"), ("c4_scaled_256x262144", lambda: C.c4(M=256), "read"),
                                ("gated_halves_8192x28672", lambda: C.gated_halves(), "2:1")):
            wi = make()
            gi = pn.Graph(wi.desc, local_rank, 0)
            si = device_sets(torch, wi, 1)
            _, pi = time_graph(torch, gi, si, args.steps, warmup)
            sti = stats(pi)
            b2b = time_back_to_back(torch, gi, si, args.steps) / args.steps
            ki = gi.kernel_info[0]
            sweep[name] = {"supplementary": True, "compulsory_bytes": gi.compulsory_bytes, "median_ms": sti["median_ms"], "min_ms": sti["min_ms"],
                           "iqr_ms": sti["iqr_ms"], "back_to_back_ms": b2b, "gbs": gi.compulsory_bytes / (b2b * 1e-3) / 1e9,
                           "frac_of_measured_peak": gi.compulsory_bytes / (b2b * 1e-3) / 1e9 / peak,
                           "family": pn.FAMILY_NAMES[ki["family"]], "buffer_sets": 1,
                           "roofline": roofline_entry(gi.compulsory_bytes, b2b * 1e-3, peak, peak_src, mix, probe, False)}
            gi.close()
            del si, wi
            torch.cuda.empty_cache()
        line["sweep"] = sweep
        line["probe_status_word"] = probe.status_word()
        line["tiny_graphs"] = tiny_graph_latency(torch, pn, local_rank, max(10, args.steps // 2))
        line["create_ms"] = create_times(local_rank)

    # ---- the CPU oracle on a bounded sample of the same workload ------------------------------
    # the whole benchmark batch (512 batches of the softmax workload), 8 batches per job over a pool
    # of worker processes, one per host core; best of 2
    sample = w if args.workload == "c2" else C.c2(seed=rank)
    opool = OraclePool()
    t_or = min(opool.seconds(sample, 8) for _ in range(2))
    opool.close()
    line["cpu_baseline"] = {"value": sample.compulsory_bytes / t_or / 1e9, "unit": "GB/s", "cores": opool.cores,
                            "kind": "oracle", "sample": "all 512 batches of the c2 workload (134 M elements), 8 batches per job over one worker process per core, best of 2",
                            "seconds": t_or, "cpu_model": cpu_model(), "host_cores": os.cpu_count()}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
