"""Error-aware speedup report (Section 3.5 of the paper, Eqs. 2-4, and its two appendices on
the AS weights and on atol(t) / rtol(t)), computed over this library's own measurements.

For each instance i (one graph at one shape and dtype) the fused handle is timed against the
unfused one-kernel-per-node handle of the same library -- the "eager" execution the paper
takes speedups against -- giving s_i = t_unfused / t_fused, and the fused outputs are compared
with the unfused ones under the tolerance ladder: correct_{t,i} for t <= 0 is the allclose rule
|got - ref| <= atol(t) + rtol(t) |ref| with the per-dtype atol(t), rtol(t); an instance that is
not correct carries an error category c_i (1 accuracy, 2 compilation, 3 runtime) and is forgiven
once t >= c_i.

The arithmetic (pure Python, no GPU):
    s_hat(t, i) = s_i                 correct and s_i >= 1
                = s_i ** (p + 1)      correct and s_i < 1
                = b ** [t < c_i]      otherwise                                  (Eq. 2)
    ES_t = geometric mean of s_hat(t, i) over the instances                     (Eq. 3)
    AS   = prod_t ES_t ** (W_t / sum_s W_s),  t = -10 .. |E| + 1                (Eq. 4)
    W_t  = 0.001 for t <= -6 or t >= |E| + 1;  1 for -5 <= t <= -3;  0.8 ** (t + 3) otherwise
with b = 0.1, p = 0 (the values the paper's experiments use) and |E| = 3 error categories.

`python -m paper_2605_29357_b200.report` runs the sweep on cuda:0 (every workload graph over
ten shapes and three storage types) and prints one JSON document.
"""
from __future__ import annotations

import json
import math
import sys
from dataclasses import dataclass
from typing import Dict, Iterable, List, Optional, Sequence

N_ERROR_CATEGORIES = 3          # accuracy, compilation, runtime
T_MIN = -10
B_DEFAULT, P_DEFAULT = 0.1, 0.0

# exponent k of rtol(t) = 10 ** (k t / 5) per storage type (atol(t) = 10 ** t for all three)
_RTOL_K = {"bf16": 1.796, "f16": 3.0, "f32": 5.886}


def t_values(n_err: int = N_ERROR_CATEGORIES) -> List[int]:
    return list(range(T_MIN, n_err + 2))


def tolerance(dtype: str, t: int):
    """(atol, rtol) at tolerance level t <= 0 for a float storage type; (0, 0) for the others."""
    if dtype not in _RTOL_K:
        return 0.0, 0.0
    t = min(t, 0)
    return 10.0 ** t, 10.0 ** (t * _RTOL_K[dtype] / 5.0)


def weight(t: int, n_err: int = N_ERROR_CATEGORIES) -> float:
    if t <= -6 or t >= n_err + 1:
        return 0.001
    if -5 <= t <= -3:
        return 1.0
    return 0.8 ** (t + 3)


@dataclass
class Instance:
    """One measured instance.  `speedup` = t_unfused / t_fused (None when nothing ran);
    `strictest_t`: the smallest t in [-10, 0] at which the outputs pass the allclose rule (None
    when they fail even at t = 0, or nothing ran); `error`: 0 none, else the category 1..3."""
    name: str
    speedup: Optional[float]
    strictest_t: Optional[int]
    error: int = 0

    def correct(self, t: int) -> bool:
        if self.error in (2, 3) or self.speedup is None or self.strictest_t is None:
            return False
        return min(t, 0) >= self.strictest_t

    def category(self) -> int:
        """Error category used when the instance is not correct at some t."""
        return self.error if self.error else 1


def rectified_speedup(inst: Instance, t: int, b: float = B_DEFAULT, p: float = P_DEFAULT) -> float:
    if inst.correct(t):
        s = inst.speedup
        return s if s >= 1.0 else s ** (p + 1.0)
    return b if t < inst.category() else 1.0


def es(instances: Sequence[Instance], t: int, b: float = B_DEFAULT, p: float = P_DEFAULT) -> float:
    if not instances:
        raise ValueError("no instances")
    return math.exp(sum(math.log(rectified_speedup(i, t, b, p)) for i in instances) / len(instances))


def aggregated_speedup(instances: Sequence[Instance], b: float = B_DEFAULT, p: float = P_DEFAULT,
                       n_err: int = N_ERROR_CATEGORIES) -> float:
    ts = t_values(n_err)
    wsum = sum(weight(t, n_err) for t in ts)
    return math.exp(sum(weight(t, n_err) / wsum * math.log(es(instances, t, b, p)) for t in ts))


def fast_p(instances: Sequence[Instance], p: float = 1.0, t: int = -5) -> float:
    """Fraction of instances correct at level t with speedup above p."""
    return sum(1 for i in instances if i.correct(t) and i.speedup > p) / len(instances)


def summarise(instances: Sequence[Instance]) -> Dict[str, object]:
    ok = [i for i in instances if i.correct(-5)]
    gmean = math.exp(sum(math.log(i.speedup) for i in ok) / len(ok)) if ok else None
    return {"instances": len(instances), "correct_at_t-5": len(ok), "fast_1": fast_p(instances, 1.0),
            "gmean_speedup_of_correct": gmean, "ES_t": {str(t): es(instances, t) for t in t_values()},
            "AS": aggregated_speedup(instances), "b": B_DEFAULT, "p": P_DEFAULT}


# ---------------------------------------------------------------------------------------------
# comparison of two sets of outputs under the ladder (NumPy; used by the sweep)
# ---------------------------------------------------------------------------------------------
def strictest_passing_t(got, ref, dtype: str) -> Optional[int]:
    """Smallest t in [-10, 0] at which every element satisfies |got - ref| <= atol(t) +
    rtol(t) |ref| (NaN must meet NaN, infinities must be equal); None if t = 0 fails too.
    Integer and boolean outputs must be identical at every t."""
    import numpy as np
    g = np.asarray(got, dtype=np.float64); r = np.asarray(ref, dtype=np.float64)
    if g.shape != r.shape:
        return None
    fin = np.isfinite(r) & np.isfinite(g)
    special_ok = np.all((fin) | (np.isnan(r) & np.isnan(g)) | (g == r))
    if not special_ok:
        return None
    if dtype not in _RTOL_K:
        return T_MIN if np.array_equal(g[fin], r[fin]) else None
    d = np.abs(g[fin] - r[fin]); a = np.abs(r[fin])
    best = None
    for t in range(0, T_MIN - 1, -1):          # passing is monotone in t: walk towards the strict end
        atol, rtol = tolerance(dtype, t)
        if np.all(d <= atol + rtol * a):
            best = t
        else:
            break
    return best


# ---------------------------------------------------------------------------------------------
# the sweep (needs a GPU)
# ---------------------------------------------------------------------------------------------
def _shape_ladder():
    """Ten shapes per workload graph, a geometric ladder around the benchmark shape's aspect."""
    ladder = {
        "c1": [dict(M=m, N=n) for m, n in ((64, 256), (128, 512), (256, 1024), (512, 1024), (1024, 1024), (1024, 2048), (2048, 2048), (333, 1000), (4096, 4096), (8192, 1024))],
        "c2": [dict(B=b, Q=q, K=k) for b, q, k in ((4, 64, 64), (8, 128, 128), (16, 128, 256), (16, 256, 256), (32, 256, 512), (32, 512, 512), (64, 512, 512), (8, 100, 200), (16, 1024, 1024), (128, 512, 512))],
        "c3": [dict(M=m, N=n) for m, n in ((128, 256), (256, 768), (512, 1024), (1024, 1024), (2048, 2048), (4096, 4096), (8192, 4096), (1000, 1000), (2048, 8192), (16384, 1024))],
        "c4": [dict(M=m, N=n) for m, n in ((4, 4096), (8, 16384), (16, 32768), (16, 65536), (32, 65536), (64, 65536), (32, 262144), (7, 10007), (128, 32768), (64, 262144))],
        "c5": [dict(M=m, N=n) for m, n in ((64, 512), (128, 1024), (256, 2048), (512, 3584), (1024, 3584), (1024, 7168), (2048, 7168), (300, 1432), (2048, 14336), (4096, 14336))],
        "n1": [dict(S=s, SC=c, Cc=ch) for s, c, ch in ((13, 8, 96), (21, 16, 96), (37, 32, 96), (69, 64, 96), (133, 128, 96), (133, 128, 192), (69, 64, 384), (45, 40, 100), (261, 256, 96), (133, 128, 48))],
        "n2": [dict(B=b, S=s, Dh=d) for b, s, d in ((4, 64, 256), (8, 128, 384), (16, 128, 768), (32, 256, 768), (32, 512, 1024), (64, 512, 1024), (128, 512, 1024), (5, 77, 200), (16, 2048, 1024), (256, 128, 1024))],
    }
    return ladder


def run_sweep(device: int = 0, steps: int = 100, warmup: int = 20, names: Iterable[str] = ()) -> Dict[str, object]:
    import numpy as np
    import torch

    from pn_workloads import configs as C
    from pn_workloads import descriptor as D
    from . import binding as pn

    if not torch.cuda.is_available():
        raise RuntimeError("the sweep needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(device)
    makers = {**C.CONFIGS, **C.EXTENDED}
    stream = torch.cuda.current_stream()
    dts = {"f32": D.F32, "f16": D.F16, "bf16": D.BF16}
    instances: List[Instance] = []
    rows = []

    def timed(g, ins, outs):
        launch = g.bind(ins, outs)               # pointer arrays marshalled once
        for _ in range(warmup):
            launch(stream.cuda_stream)
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        ev[0].record(stream)
        for k in range(steps):
            launch(stream.cuda_stream)
            ev[k + 1].record(stream)
        torch.cuda.synchronize()
        return float(np.median([ev[k].elapsed_time(ev[k + 1]) for k in range(steps)]))

    for name, shapes in _shape_ladder().items():
        if names and name not in names:
            continue
        for shape in shapes:
            for dname, dt in dts.items():
                label = f"{name}{sorted(shape.items())}/{dname}"
                w = makers[name](dtype=dt, **shape)
                d_in = [torch.from_numpy(np.ascontiguousarray(a).reshape(-1).view(np.uint8).copy()).cuda() for a in w.inputs]
                sizes = [D.DTYPE_BYTES[m] * int(np.prod(dims, dtype=np.int64)) for m, dims in w.output_meta]
                out_f = [torch.full((max(s, 16),), 0xFF, dtype=torch.uint8, device="cuda") for s in sizes]
                out_u = [torch.full((max(s, 16),), 0xFF, dtype=torch.uint8, device="cuda") for s in sizes]
                ins = [t.data_ptr() for t in d_in]
                inst = Instance(label, None, None, 0)
                try:
                    gf = pn.Graph(w.desc, device, 0)
                    gu = pn.Graph(w.desc, device, pn.FLAG_UNFUSED)
                except pn.PnError:
                    inst.error = 2
                else:
                    try:
                        t_f = timed(gf, ins, [t.data_ptr() for t in out_f])
                        t_u = timed(gu, ins, [t.data_ptr() for t in out_u])
                    except pn.PnError:
                        inst.error = 3
                    else:
                        inst.speedup = t_u / t_f
                        worst = T_MIN
                        for tf, tu, (m, dims), s in zip(out_f, out_u, w.output_meta, sizes):
                            a = tf.cpu().numpy()[:s].view(C.NP_STORAGE[m]).reshape(dims)
                            b = tu.cpu().numpy()[:s].view(C.NP_STORAGE[m]).reshape(dims)
                            kind = {D.F32: "f32", D.F16: "f16", D.BF16: "bf16"}.get(m, "int")
                            if m == D.BF16:
                                a = (a.astype(np.uint32) << 16).view(np.float32); b = (b.astype(np.uint32) << 16).view(np.float32)
                            st = strictest_passing_t(a, b, kind)
                            worst = None if (st is None or worst is None) else max(worst, st)
                        inst.strictest_t = worst
                        if worst is None:
                            inst.error = 1
                        rows.append({"instance": label, "fused_ms": t_f, "unfused_ms": t_u, "speedup": inst.speedup,
                                     "kernels_unfused": gu.n_kernels, "strictest_t": worst})
                    gf.close(); gu.close()
                instances.append(inst)
                del d_in, out_f, out_u
        torch.cuda.empty_cache()
    doc = summarise(instances)
    doc["per_workload"] = {}
    for name in _shape_ladder():
        sub = [i for i in instances if i.name.startswith(name + "[")]
        if sub:
            doc["per_workload"][name] = {k: v for k, v in summarise(sub).items() if k in ("instances", "fast_1", "gmean_speedup_of_correct", "AS")}
    doc["errors"] = [{"instance": i.name, "category": i.error} for i in instances if i.error]
    doc["rows"] = rows
    doc["protocol"] = f"{warmup} warm-up + {steps} timed launches per handle, median, CUDA events; reference = the unfused path of the same library"
    return doc


if __name__ == "__main__":
    names = [a for a in sys.argv[1:] if not a.startswith("-")]
    print(json.dumps(run_sweep(names=names)))
