"""Seeded random fusible subgraphs for the parity tests (the paper asks of a rewrite that it hold
over shapes and dtypes rather than fit one instance, Section 3.1; here the graph *structure* is
what varies): 2 - 40 operator nodes drawn from the whole opcode table over the broadcast patterns
of the load step (full tensor, row vector [N], column [.., 1], batch-broadcast [1, R, N], scalar
immediate), 0 - 3 levels of last-dimension reductions so that 1 - 4 stages arise, a random set of
outputs and three storage types.

A random expression is only a fair test of an fp32 kernel against an fp64 oracle under a relative
tolerance if it is well conditioned, so every value carries a class and the generator combines
classes only where nothing can cancel or flip:
  P  positive, inside a tracked interval [lo, hi] (hi <= 1000): sums, products, quotients by values
     bounded away from zero, roots, the smooth activations
  E  exact: stored inputs and what negation, abs, relu, max / min, clamp, where and narrowing casts
     make of them -- the same number in fp32 and fp64, so it may be compared, truncated and
     arg-reduced without the two sides ever disagreeing on a boolean or an index
  B  booleans made from E values (or mask inputs): exact
  S  signed, well conditioned (products of E and P values, normalised rows): never added to
     anything, so no cancellation; reductions of them are limited to those that cannot cancel
Per-row results of reductions carry the same classes.  This module holds no arithmetic of the
operators: it draws inputs, keeps intervals, and writes descriptors."""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import List, Optional, Tuple

import numpy as np

from pn_workloads import configs as C
from pn_workloads import descriptor as D
from pn_workloads.descriptor import GraphBuilder, Imm

HI_MAX = 1000.0
DEN_MIN = 1e-2          # smallest lower bound of a value that may be divided by
FLOAT_STORAGE = [D.F32, D.BF16, D.F16]


@dataclass
class Val:
    tid: int
    shape: Tuple[int, ...]
    kind: str               # 'P', 'E', 'B', 'S'
    lo: float = 0.0
    hi: float = 0.0
    stage: int = 0
    scalar: bool = False    # a per-row value (result of a last-dimension reduction, or made of such)
    dtype: int = D.F32
    fresh: bool = True      # an input or one step from it (spread of values still that of the input)
    integral: bool = False  # exact small integers (counts, integer inputs)


class RandomGraph:
    def __init__(self, seed: int, max_nodes: Optional[int] = None):
        self.rng = np.random.default_rng([7919, seed])
        r = self.rng
        self.g = GraphBuilder()
        self.inputs: List[np.ndarray] = []
        self.n_nodes = 0
        rank = int(r.choice([1, 2, 2, 3, 3]))
        n = int(r.choice([1, 2, 7, 8, 24, 96, 100, 255, 256, 1000, 1024, 1032, 2048, 4100, 5000]))
        lead = {1: (), 2: (int(r.integers(1, 40)),), 3: (int(r.integers(1, 6)), int(r.integers(1, 12)))}[rank]
        self.full = tuple(lead) + (n,)
        self.row_shape = tuple(lead) + (1,)
        self.target = int(max_nodes if max_nodes else r.integers(2, 41))
        self.tiles: List[Val] = []
        self.scalars: List[Val] = []
        self.red_per_stage = [0, 0, 0, 0]
        self.softmax_done = False
        self.max_inputs = 6
        self.outputs: List[Val] = []
        self.notes: List[str] = []
        self._build()

    # ---- inputs -------------------------------------------------------------------------------
    def _pattern_shape(self) -> Tuple[int, ...]:
        r = self.rng
        opts = [self.full, self.full, self.full, (self.full[-1],), self.row_shape]
        if len(self.full) == 3:
            opts.append((1,) + self.full[1:])
        return opts[int(r.integers(len(opts)))]

    def _new_input(self, kind: str, shape=None, dtype=None) -> Optional[Val]:
        if len(self.inputs) >= self.max_inputs:
            return None
        r = self.rng
        shape = tuple(shape if shape is not None else self._pattern_shape())
        if kind == "B":
            dt = int(r.choice([D.I8, D.BOOL]))
            arr = (r.random(shape) < 0.6).astype(C.NP_STORAGE[dt])
            if dt == D.I8:
                arr = arr * r.integers(1, 5, size=shape).astype(np.int8) * r.choice([-1, 1], size=shape).astype(np.int8)   # any non-zero byte is true
            v = Val(self.g.input(dt, shape), shape, "B", dtype=dt)
        elif kind == "I":
            dt = int(r.choice([D.I32, D.I64, D.I8]))
            arr = r.integers(-5, 6, size=shape).astype(C.NP_STORAGE[dt])
            v = Val(self.g.input(dt, shape), shape, "E", lo=-5, hi=5, dtype=dt, integral=True)
        else:
            dt = int(dtype if dtype is not None else r.choice(FLOAT_STORAGE))
            # a full-shape operand is sometimes read through rolls and slices of a larger graph input,
            # over leading dimensions and over the last one (index-remapped loads)
            chain = []
            root = list(shape)
            if shape == self.full and r.random() < 0.3:
                for d in range(len(shape)):
                    if r.random() < 0.5:
                        chain.append(("roll", d, int(r.choice([1, 3, 8, -8, 16, 250]))))
                for d in range(len(shape)):
                    if r.random() < 0.5:
                        extra = int(r.choice([1, 3, 8, 8, 16, 32]))
                        chain.append(("slice", d, int(r.integers(0, extra + 1)) if r.random() < 0.5 else extra))
                        root[d] += extra
            root = tuple(root)
            if kind == "P":
                x = (r.random(root) * 1.5 + 0.5).astype(np.float32)
                x = np.clip(x, 0.5, 2.0)
                v = Val(self.g.input(dt, root), root, "P", lo=0.5, hi=2.0, dtype=dt)
            else:
                x = (r.standard_normal(root) * float(r.choice([0.5, 1.0, 3.0]))).astype(np.float32)
                x = np.round(x * 8) / 8 if r.random() < 0.3 else x          # quarter-ish steps: exact ties for the arg-reductions
                v = Val(self.g.input(dt, root), root, "E", lo=-20, hi=20, dtype=dt)
            arr = C._store(x.astype(np.float32), dt)
            cur = list(root)
            for op, d, amount in chain:                                     # rolls first, then the slices, one dimension a node
                if op == "slice":
                    cur[d] = shape[d]
                v = self._emit(op, [v], dt, tuple(cur), v.kind, v.lo, v.hi, attr=(d, amount), fresh=True)
            if chain:
                self.notes.append("indexed input: " + ", ".join(f"{o}({d},{a})" for o, d, a in chain))
        self.inputs.append(np.ascontiguousarray(arr))
        if v.dtype != D.F32 and v.kind in ("P", "E") and not v.integral:
            v = self._emit("cast", [v], D.F32, shape, v.kind, v.lo, v.hi, fresh=True)     # widen: exact
        elif v.integral:
            v = self._emit("cast", [v], D.F32, shape, "E", -5, 5, fresh=True, integral=True)
        self.tiles.append(v)
        return v

    # ---- nodes --------------------------------------------------------------------------------
    def _emit(self, op, ins, dtype, shape, kind, lo=0.0, hi=0.0, attr=(0, 0), extra_imm=(), scalar=None, fresh=False,
              integral=False) -> Val:
        ids = [x.tid if isinstance(x, Val) else x for x in ins]
        tid = self.g.op(op, ids, dtype, shape, attr=attr, extra_imm=extra_imm)
        vals = [x for x in ins if isinstance(x, Val)]
        stage = max([x.stage for x in vals] + [0])
        sc = all(x.scalar for x in vals) if scalar is None else scalar
        self.n_nodes += 1
        return Val(tid, tuple(shape), kind, float(lo), float(hi), stage, sc, dtype, fresh, integral)

    def _bshape(self, *vals) -> Tuple[int, ...]:
        return tuple(np.broadcast_shapes(*[v.shape for v in vals]))

    def _pick(self, pool, pred=lambda v: True) -> Optional[Val]:
        c = [v for v in pool if pred(v)]
        return c[int(self.rng.integers(len(c)))] if c else None

    def _keep(self, v: Val) -> Val:
        (self.scalars if v.scalar else self.tiles).append(v)
        return v

    def _is_full(self, v: Val) -> bool:
        return (not v.scalar) and v.shape == self.full

    # one step of growth; returns False when nothing could be added
    def _grow(self) -> bool:
        r = self.rng
        action = r.choice(["unaryP", "binP", "binP", "fma", "eop", "cmp", "where", "toP", "toS", "sop", "reduce", "reduce",
                           "composite", "scal", "mix", "narrow", "input", "boolmul"])
        P = lambda v: v.kind == "P"
        if action == "input":
            return self._new_input(str(r.choice(["P", "E", "E", "B", "I"]))) is not None
        if action == "unaryP":
            v = self._pick(self.tiles + self.scalars, P)
            if not v:
                return False
            cands = [("sqrt", math.sqrt(v.lo), math.sqrt(v.hi)), ("sigmoid", 0.5, 1.0), ("contiguous", v.lo, v.hi), ("tanh", math.tanh(v.lo), 1.0),
                     ("relu", v.lo, v.hi), ("abs", v.lo, v.hi), ("erf", math.erf(v.lo), 1.0),
                     ("silu", v.lo / (1 + math.exp(-v.lo)), v.hi), ("gelu_tanh", 0.5 * v.lo, v.hi), ("gelu_erf", 0.5 * v.lo, v.hi)]
            if v.hi * v.hi <= HI_MAX:
                cands.append(("square", v.lo * v.lo, v.hi * v.hi))
            if v.lo >= DEN_MIN:
                cands += [("recip", 1 / v.hi, 1 / v.lo), ("rsqrt", 1 / math.sqrt(v.hi), 1 / math.sqrt(v.lo))]
            if v.hi <= 6.0:
                cands.append(("exp", math.exp(v.lo), math.exp(v.hi)))
            if v.lo >= 1.5:
                cands.append(("log", math.log(v.lo), math.log(v.hi)))
            op, lo, hi = cands[int(r.integers(len(cands)))]
            if hi > HI_MAX:
                return False
            self._keep(self._emit(op, [v], D.F32, v.shape, "P", lo, hi))
            return True
        if action in ("binP", "fma"):
            a = self._pick(self.tiles + self.scalars, P)
            b = self._pick(self.tiles + self.scalars, P)
            if not a or not b:
                return False
            if a.scalar != b.scalar and (a if a.scalar else b).shape != self.row_shape:
                return False                      # a per-row value meets tile values only in its kept-dimension form
            shape = self._bshape(a, b)
            if action == "fma":
                c = self._pick(self.tiles + self.scalars, lambda v: P(v) and v.scalar == a.scalar)
                if not c or a.scalar != b.scalar:
                    return False
                lo, hi = a.lo * b.lo + c.lo, a.hi * b.hi + c.hi
                if hi > HI_MAX:
                    return False
                self._keep(self._emit("fma", [a, b, c], D.F32, self._bshape(a, b, c), "P", lo, hi))
                return True
            use_imm = r.random() < 0.25
            imm = float(r.choice([0.125, 0.5, 1.0, 1.5, 3.0]))
            op = str(r.choice(["add", "mul", "div", "max", "min"]))
            if use_imm:
                b2, blo, bhi, shape = Imm(imm), imm, imm, a.shape
            else:
                b2, blo, bhi = b, b.lo, b.hi
            if op == "add":
                lo, hi = a.lo + blo, a.hi + bhi
            elif op == "mul":
                lo, hi = a.lo * blo, a.hi * bhi
            elif op == "div":
                if blo < DEN_MIN:
                    return False
                lo, hi = a.lo / bhi, a.hi / blo
            elif op == "max":
                lo, hi = max(a.lo, blo), max(a.hi, bhi)
            else:
                lo, hi = min(a.lo, blo), min(a.hi, bhi)
            if hi > HI_MAX:
                return False
            self._keep(self._emit(op, [a, b2], D.F32, shape, "P", lo, hi))
            return True
        if action == "eop":        # exact in, exact out
            a = self._pick(self.tiles, lambda v: v.kind == "E")
            if not a:
                return False
            op = str(r.choice(["neg", "abs", "relu", "max", "min", "clamp"]))
            if op in ("neg", "abs", "relu"):
                self._keep(self._emit(op, [a], D.F32, a.shape, "E", -20, 20, integral=a.integral))
            elif op == "clamp":
                self._keep(self._emit("clamp", [a, Imm(-0.75), Imm(1.25)], D.F32, a.shape, "E", -0.75, 1.25))
            else:
                b = self._pick(self.tiles, lambda v: v.kind == "E")
                other = Imm(float(r.choice([-1.0, 0.0, 0.25]))) if (r.random() < 0.4 or not b) else b
                shape = a.shape if isinstance(other, Imm) else self._bshape(a, other)
                self._keep(self._emit(op, [a, other], D.F32, shape, "E", -20, 20))
            return True
        if action == "cmp":
            a = self._pick(self.tiles, lambda v: v.kind == "E")
            if not a:
                return False
            b = self._pick(self.tiles, lambda v: v.kind == "E")
            other = Imm(float(r.choice([-0.5, 0.0, 0.125, 1.0]))) if (r.random() < 0.5 or not b) else b
            shape = a.shape if isinstance(other, Imm) else self._bshape(a, other)
            op = str(r.choice(["gt", "ge", "lt", "le", "eq", "ne"]))
            self._keep(self._emit(op, [a, other], int(r.choice([D.BOOL, D.I8])), shape, "B"))
            return True
        if action == "boolmul":
            a = self._pick(self.tiles, lambda v: v.kind == "B" and v.stage >= 0 and v.dtype in (D.BOOL, D.I8) and v.tid not in self.g.input_ids())
            b = self._pick(self.tiles, lambda v: v.kind == "B" and v.tid not in self.g.input_ids())
            if not a or not b:
                return False
            self._keep(self._emit("mul", [a, b], D.BOOL, self._bshape(a, b), "B"))
            return True
        if action == "where":
            c = self._pick(self.tiles, lambda v: v.kind == "B")
            kind = str(r.choice(["P", "E"]))
            a = self._pick(self.tiles, lambda v: v.kind == kind)
            b = self._pick(self.tiles, lambda v: v.kind == kind)
            if not c or not a:
                return False
            other = b if (b and r.random() < 0.7) else Imm(1.0 if kind == "P" else float(r.choice([0.0, -2.0])))
            shape = self._bshape(*[x for x in (c, a, other) if isinstance(x, Val)])
            lo = min(a.lo, other.lo if isinstance(other, Val) else (1.0 if kind == "P" else -2.0))
            hi = max(a.hi, other.hi if isinstance(other, Val) else 1.0)
            self._keep(self._emit("where", [c, a, other], D.F32, shape, kind, lo, hi))
            return True
        if action == "toP":        # exact or signed -> positive
            a = self._pick(self.tiles, lambda v: v.kind in ("E", "S"))
            if not a:
                return False
            if r.random() < 0.5:
                m = self._emit("abs", [a], D.F32, a.shape, a.kind, 0, 20)
                self._keep(self._emit("add", [m, Imm(0.5)], D.F32, a.shape, "P", 0.5, 20.5))
            else:
                self._keep(self._emit("sigmoid", [a], D.F32, a.shape, "P", 0.0, 1.0))
            return True
        if action == "toS":        # exact times positive: signed, nothing cancels
            a = self._pick(self.tiles, lambda v: v.kind == "E" and not v.integral)
            b = self._pick(self.tiles, lambda v: P(v) and v.hi <= 30)
            if not a or not b:
                return False
            self._keep(self._emit("mul", [a, b], D.F32, self._bshape(a, b), "S", -20 * b.hi, 20 * b.hi, fresh=a.fresh and b.fresh))
            return True
        if action == "sop":
            a = self._pick(self.tiles, lambda v: v.kind == "S")
            if not a:
                return False
            op = str(r.choice(["neg", "tanh", "erf", "silu", "gelu_tanh", "gelu_erf"]))
            self._keep(self._emit(op, [a], D.F32, a.shape, "S", -max(abs(a.lo), a.hi), max(abs(a.lo), a.hi)))
            return True
        if action == "narrow":     # a declared narrow intermediate: rounded for its consumers; exact values only
            a = self._pick(self.tiles, lambda v: v.kind == "E" and not v.integral and v.dtype == D.F32)
            if not a:
                return False
            n = self._emit("cast", [a], int(r.choice([D.BF16, D.F16])), a.shape, "E", a.lo, a.hi)
            self._keep(self._emit("cast", [n], D.F32, a.shape, "E", a.lo, a.hi))
            return True
        if action == "reduce":
            x = self._pick(self.tiles, lambda v: self._is_full(v) and v.stage <= 2 and self.red_per_stage[v.stage] < 4)
            if not x:
                return False
            n = self.full[-1]
            keep = r.random() < 0.7
            shape = self.row_shape if keep else self.full[:-1]
            if x.kind == "P":
                op = str(r.choice(["sum", "mean", "var", "amax", "amin", "logsumexp"]))
                if op == "var" and (not x.fresh or n < 2):
                    op = "mean"
            elif x.kind == "E":
                op = str(r.choice(["amax", "amin", "argmax", "argmin", "logsumexp"]))
            elif x.kind == "S":
                op = str(r.choice(["amax", "amin", "logsumexp"]))
            else:
                op = "sum"         # a count: exact
            self.red_per_stage[x.stage] += 1
            if op in ("argmax", "argmin"):
                v = self._emit(op, [x], int(r.choice([D.I64, D.I32])), shape, "E", 0, n - 1, scalar=True, integral=True)
                v.stage = x.stage + 1
                self.outputs.append(v)             # indices only leave the graph
                return True
            if op == "sum":
                lo, hi = (x.lo * n, x.hi * n) if x.kind == "P" else (0, n)
            elif op == "var":
                lo, hi = 0.0, (x.hi - x.lo) ** 2
            elif op == "logsumexp":
                lo, hi = x.lo + math.log(n), x.hi + math.log(n)
            else:
                lo, hi = x.lo, x.hi
            kind = "P" if (x.kind == "P" and op != "var") else ("E" if (x.kind == "B" or (x.kind == "E" and op in ("amax", "amin"))) else "S")
            if op == "var":
                kind = "S"                         # small and positive: leaves the graph, or is added to
            if hi > HI_MAX and kind == "P":
                kind = "S"
            dt = D.F32
            v = self._emit(op, [x], dt, shape, kind, lo, hi, attr=(int(r.integers(0, 2)) if op == "var" and n > 1 else 0, 0),
                           scalar=True, integral=x.kind == "B")
            v.stage = x.stage + 1
            if keep:
                self.scalars.append(v)
            if not keep or r.random() < 0.4:
                self.outputs.append(v)
            return True
        if action == "composite":
            x = self._pick(self.tiles, lambda v: self._is_full(v) and v.stage <= 2 and v.kind in ("P", "E", "S")
                           and not v.integral and self.red_per_stage[v.stage] < 4)
            if not x:
                return False
            n = self.full[-1]
            op = str(r.choice(["softmax", "log_softmax", "layer_norm", "rms_norm"]))
            if op == "softmax" and self.softmax_done:
                op = "log_softmax"
            if op == "layer_norm" and (not x.fresh or n < 8 or x.kind == "P" and x.hi - x.lo < 0.5):
                op = "rms_norm"
            self.red_per_stage[x.stage] += 1
            if op == "softmax":
                self.softmax_done = True
                v = self._emit("softmax", [x], D.F32, self.full, "P", 0.0, 1.0, scalar=False)
            elif op == "log_softmax":
                v = self._emit("log_softmax", [x], D.F32, self.full, "S", -60 - math.log(n), 0.0, scalar=False)
            elif op == "rms_norm":
                ins = [x]
                if r.random() < 0.5:
                    gm = self._new_input("P", (n,))
                    if gm:
                        ins.append(gm)
                kind = "P" if x.kind == "P" else "S"
                v = self._emit("rms_norm", ins, D.F32, self.full, kind, 0.0, 100.0, extra_imm=[1e-6], scalar=False)
            else:
                ins = [x]
                gm = self._new_input("P", (n,)) if r.random() < 0.7 else None
                if gm:
                    ins.append(gm)
                    be = self._new_input("E", (n,)) if r.random() < 0.7 else None
                    if be:
                        ins.append(be)
                n_out = int(r.choice([1, 3]))
                outs = self.g.node("layer_norm", [i.tid for i in ins], [D.F32] * n_out,
                                   [self.full] + [self.row_shape] * (n_out - 1), extra_imm=[1e-5])
                self.n_nodes += 1
                v = Val(outs[0], self.full, "S", -100, 100, x.stage + 1, False)
                if n_out == 3:
                    for t in outs[1:]:
                        s = Val(t, self.row_shape, "S", -100, 100, x.stage + 1, True)
                        self.outputs.append(s)
            v.stage = x.stage + 1
            v.fresh = False
            self.tiles.append(v)
            return True
        if action == "scal":       # arithmetic among per-row values
            a = self._pick(self.scalars, lambda v: P(v) and v.shape == self.row_shape)
            b = self._pick(self.scalars, lambda v: P(v) and v.shape == self.row_shape)
            if not a or not b:
                return False
            op = str(r.choice(["add", "mul", "div", "sqrt", "recip"]))
            if op == "sqrt":
                self._keep(self._emit("sqrt", [a], D.F32, a.shape, "P", math.sqrt(a.lo), math.sqrt(a.hi)))
            elif op == "recip":
                if a.lo < DEN_MIN:
                    return False
                self._keep(self._emit("recip", [a], D.F32, a.shape, "P", 1 / a.hi, 1 / a.lo))
            else:
                if op == "div" and b.lo < DEN_MIN:
                    return False
                lo, hi = {"add": (a.lo + b.lo, a.hi + b.hi), "mul": (a.lo * b.lo, a.hi * b.hi), "div": (a.lo / max(b.hi, 1e-30), a.hi / max(b.lo, DEN_MIN))}[op]
                if hi > HI_MAX:
                    return False
                self._keep(self._emit(op, [a, b], D.F32, a.shape, "P", lo, hi))
            return True
        if action == "mix":        # a per-row value meets the row again
            s = self._pick(self.scalars, lambda v: v.shape == self.row_shape and v.kind in ("P", "S", "E") and not v.integral)
            x = self._pick(self.tiles, lambda v: self._is_full(v) and v.kind in ("P", "S", "E") and not v.integral)
            if not s or not x:
                return False
            if s.kind == "P" and x.kind == "P" and r.random() < 0.6:
                op = str(r.choice(["mul", "div"]))
                if op == "div" and s.lo < DEN_MIN:
                    op = "mul"
                lo, hi = (x.lo * s.lo, x.hi * s.hi) if op == "mul" else (x.lo / s.hi, x.hi / s.lo)
                if hi > HI_MAX:
                    return False
                self.tiles.append(self._emit(op, [x, s], D.F32, self.full, "P", lo, hi, scalar=False))
            else:                  # x minus its row's maximum (or any per-row value): signed, feeds exp or leaves
                d = self._emit("sub", [x, s], D.F32, self.full, "S", x.lo - s.hi, x.hi - s.lo, scalar=False)
                d.fresh = False
                self.tiles.append(d)
            return True
        return False

    def _build(self) -> None:
        r = self.rng
        self._new_input("P", self.full)
        self._new_input("E", self.full)
        if r.random() < 0.5:
            self._new_input("B")
        tries = 0
        while self.n_nodes < self.target and tries < 40 * self.target:
            tries += 1
            self._grow()
        # outputs: what was marked on the way, plus a few full-shape values and per-row values
        cands = [v for v in self.tiles if self._is_full(v) and v.tid not in self.g.input_ids()]
        r.shuffle(cands)
        extra = cands[: int(r.integers(1, 4))]
        if not extra and not self.outputs:         # nothing full-shaped was computed: make one value that is
            x = self.tiles[0]
            extra = [self._emit("mul", [x, Imm(1.5)], D.F32, self.full, "P", x.lo * 1.5, x.hi * 1.5)]
        if r.random() < 0.25:                      # a concatenation of two or three computed values leaves the graph too
            parts = [v for v in self.tiles if self._is_full(v) and v.kind in ("P", "S") and v.dtype == D.F32 and v.tid not in self.g.input_ids()]
            if len(parts) >= 2:
                k = int(r.integers(2, min(3, len(parts)) + 1))
                pick = [parts[int(i)] for i in r.choice(len(parts), size=k, replace=False)]
                dim = int(r.integers(0, len(self.full)))
                shape = list(self.full); shape[dim] = k * self.full[dim]
                c = self._emit("cat", pick, D.F32, tuple(shape), "S", attr=(dim, 0))
                self.g.mark_output(c.tid)
        outs = (self.outputs + extra)[: 11 - len(self.inputs)]
        seen = set()
        for v in outs:
            if v.tid in seen:
                continue
            seen.add(v.tid)
            o = v
            if v.kind in ("P", "S", "E") and not v.integral and v.dtype == D.F32 and r.random() < 0.5:
                o = self._emit("cast", [v], int(r.choice([D.BF16, D.F16])), v.shape, v.kind, v.lo, v.hi)
            elif v.kind == "B" and r.random() < 0.5:
                o = self._emit("cast", [v], int(r.choice([D.I8, D.BOOL])), v.shape, "B")
            elif v.integral and v.dtype == D.F32 and r.random() < 0.5:
                o = self._emit("cast", [v], int(r.choice([D.I32, D.I64])), v.shape, "E", integral=True)
            self.g.mark_output(o.tid)
        self.desc = self.g.build()
        self.output_meta = [self.g.tensor_meta(t) for t in self.g.output_ids()]


def make(seed: int, max_nodes: Optional[int] = None) -> RandomGraph:
    return RandomGraph(seed, max_nodes)


# ---------------------------------------------------------------------------------------------
# Graphs that reduce over a LEADING dimension (the masked-mean-pooling shape): a pointwise chain
# with broadcast operands before the reductions, one to three reductions over one dimension, a
# pointwise chain on the reduced values after them.  Values stay positive where they are summed
# (no cancellation), so fp32 kernels can be held to the relative tolerance.
# ---------------------------------------------------------------------------------------------
class ColumnGraph:
    def __init__(self, seed: int):
        r = self.rng = np.random.default_rng([104729, seed])
        g = self.g = GraphBuilder()
        self.inputs: List[np.ndarray] = []
        rank = int(r.choice([2, 3, 3, 4]))
        C_ = int(r.choice([1, 7, 8, 24, 64, 96, 200, 256, 1000, 1032]))
        R = int(r.choice([1, 2, 5, 33, 64, 129, 700, 2500]))
        if R * C_ > 400_000:
            R = 129
        lead = {2: (), 3: (int(r.integers(1, 7)),), 4: (int(r.integers(1, 4)), int(r.integers(1, 4)))}[rank]
        dim = len(lead)                                            # the reduced dimension: the last leading one ...
        full = tuple(lead) + (R, C_)
        if rank == 4 and r.random() < 0.5:                         # ... or, at rank 4, the one before it
            dim = 1
            full = (lead[0], R, lead[1], C_)
        self.full, self.dim = full, dim
        keep = tuple(1 if i == dim else d for i, d in enumerate(full))
        drop = tuple(d for i, d in enumerate(full) if i != dim)
        dt = int(r.choice(FLOAT_STORAGE))
        x = self._input(dt, full, "P")
        xf = g.op("cast", [x], D.F32, full) if dt != D.F32 else x
        pre, n_nodes = [xf], (1 if dt != D.F32 else 0)
        # the chain before the reductions: broadcast operands of every pattern the column family takes
        for _ in range(int(r.integers(0, 5))):
            a = pre[int(r.integers(len(pre)))]
            kind = str(r.choice(["scale", "vec", "mask", "sqrt", "imm_add", "full"]))
            if kind == "scale":
                v = g.op("mul", [a, Imm(float(r.choice([0.5, 1.25, 2.0])))], D.F32, full)
            elif kind == "imm_add":
                v = g.op("add", [a, Imm(float(r.choice([0.25, 1.0])))], D.F32, full)
            elif kind == "sqrt":
                v = g.op("sqrt", [a], D.F32, full)
            elif kind == "vec":                                    # a vector over the columns
                w = self._input(D.F32, (C_,), "P")
                v = g.op("mul", [a, w], D.F32, full)
            elif kind == "mask":                                   # one value per step of the reduced dimension
                mshape = tuple(d if i <= dim else 1 for i, d in enumerate(full))
                mdt = int(r.choice([D.I64, D.I8, D.F32]))
                m = self._input(mdt, mshape, "M")
                mf = g.op("cast", [m], D.F32, mshape) if mdt != D.F32 else m
                n_nodes += 1 if mdt != D.F32 else 0
                v = g.op("mul", [a, mf], D.F32, full)
            else:
                b2 = self._input(int(r.choice(FLOAT_STORAGE)), full, "P")
                bf = b2 if g.tensor_meta(b2)[0] == D.F32 else g.op("cast", [b2], D.F32, full)
                n_nodes += 0 if g.tensor_meta(b2)[0] == D.F32 else 1
                v = g.op(str(r.choice(["add", "mul", "max"])), [a, bf], D.F32, full)
            pre.append(v); n_nodes += 1
        self._pre, self._keep, self._drop, self._n = pre, keep, drop, n_nodes
        self._finish()

    def _input(self, dt, shape, kind):
        r = self.rng
        if kind == "M":                                            # 0 / 1 with a run of kept positions
            arr = (r.random(shape) < 0.7).astype(C.NP_STORAGE[dt])
        else:
            arr = C._store((r.random(shape) * 1.5 + 0.5).astype(np.float32), dt)
        self.inputs.append(np.ascontiguousarray(arr))
        return self.g.input(dt, shape)

    def _finish(self):
        r, g = self.rng, self.g
        pre, keep, drop, dim = self._pre, self._keep, self._drop, self.dim
        reds = []
        for _ in range(int(r.integers(1, 4))):
            src = pre[int(r.integers(len(pre)))]
            op = str(r.choice(["sum_dim", "sum_dim", "mean_dim", "amax_dim", "amin_dim"]))
            reds.append(g.op(op, [src], D.F32, keep if r.random() < 0.5 else drop, attr=[dim, 0]))
            self._n += 1
        post = list(reds)
        shape_of = lambda t: tuple(g.tensor_meta(t)[1])
        for _ in range(int(r.integers(0, 4))):                     # the epilogue on the reduced values
            a = post[int(r.integers(len(post)))]
            sh = shape_of(a)
            kind = str(r.choice(["scale", "clamp", "pair", "input"]))
            if kind == "scale":
                v = g.op("mul", [a, Imm(float(r.choice([0.5, 3.0])))], D.F32, sh)
            elif kind == "clamp":
                v = g.op("clamp", [a, Imm(0.75), Imm(50.0)], D.F32, sh)
            elif kind == "pair":
                same = [t for t in post if shape_of(t) == sh and t != a]
                if not same:
                    continue
                b2 = same[int(r.integers(len(same)))]
                v = g.op(str(r.choice(["add", "div", "max"])), [a, g.op("add", [b2, Imm(1.0)], D.F32, sh)], D.F32, sh)
                self._n += 1
            else:                                                  # a graph input of the reduced shape
                w = self._input(D.F32, sh, "P")
                v = g.op("mul", [a, w], D.F32, sh)
            post.append(v); self._n += 1
        outs = [post[-1]] + [t for t in post[:-1] if r.random() < 0.4]
        if len(pre) > 1 and r.random() < 0.3:
            outs.append(pre[-1])                                   # a full-shape value of the walk leaves the graph too
        for t in dict.fromkeys(outs):
            if r.random() < 0.3:
                t = g.op("cast", [t], int(r.choice([D.BF16, D.F16])), shape_of(t)); self._n += 1
            g.mark_output(t)
        self.n_nodes = self._n
        self.desc = g.build()
        self.output_meta = [g.tensor_meta(t) for t in g.output_ids()]


def make_column(seed: int) -> ColumnGraph:
    return ColumnGraph(seed)
