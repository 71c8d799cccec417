"""Writer for the serialized op-DAG descriptor (format version 1).

A descriptor is the byte string that states a computational graph
G = (V, E, tau, sigma) in the sense of Definition 3.1 of the paper: a table of
tensors (sigma: a static shape and a dtype per value) and a table of operator
nodes in topological order (tau: an opcode per node; E: the tensor ids each
node reads and writes).

This module only *writes* the format.  It holds no arithmetic of any operator,
so that both the CUDA library and the CPU oracle can be fed by it while each
keeps a parser of its own.

Layout (little-endian, no padding beyond what is listed):

  header   16 B : u32 magic 'PNG1' | u16 version=1 | u16 0 | u32 n_tensors | u32 n_nodes
  tensor   40 B : u8 dtype | u8 role | u8 rank | u8 0 | u32 0 | i64 dims[4]
  node     64 B : u16 opcode | u8 n_in | u8 n_out | u32 in[4] | u32 out[3]
                  | f64 imm[2] | i64 attr[2]

Tensor ids are positions in the tensor table.  Graph inputs are the tensors
with role bit 0 set, in table order; graph outputs are those with role bit 1
set, in table order.  An operand slot holding 0xFFFFFFFF / 0xFFFFFFFE names the
node's immediate imm[0] / imm[1] instead of a tensor.  All tensors are dense
row-major; broadcasting follows NumPy's size-1 rules.
"""
from __future__ import annotations

import struct
from dataclasses import dataclass, field
from typing import List, Sequence, Union

MAGIC = 0x31474E50  # bytes 'P','N','G','1'
VERSION = 1
MAX_RANK = 4

# dtype codes
F32, F16, BF16, I8, BOOL, I32, I64 = range(7)
DTYPE_NAMES = {F32: "f32", F16: "f16", BF16: "bf16", I8: "i8", BOOL: "bool", I32: "i32", I64: "i64"}
DTYPE_BYTES = {F32: 4, F16: 2, BF16: 2, I8: 1, BOOL: 1, I32: 4, I64: 8}

ROLE_INPUT = 1
ROLE_OUTPUT = 2

IMM0 = 0xFFFFFFFF
IMM1 = 0xFFFFFFFE

# opcodes (fixed by the format)
OPCODES = {
    # unary
    "neg": 1, "abs": 2, "exp": 3, "log": 4, "sqrt": 5, "rsqrt": 6, "recip": 7,
    "tanh": 8, "sigmoid": 9, "silu": 10, "gelu_tanh": 11, "gelu_erf": 12,
    "relu": 13, "cast": 14, "square": 15, "erf": 16,
    # binary
    "add": 32, "sub": 33, "mul": 34, "div": 35, "max": 36, "min": 37,
    "gt": 38, "ge": 39, "lt": 40, "le": 41, "eq": 42, "ne": 43,
    # ternary
    "where": 64, "clamp": 65, "fma": 66,
    # last-dim reductions
    "sum": 96, "mean": 97, "var": 98, "amax": 99, "amin": 100,
    "argmax": 101, "argmin": 102, "logsumexp": 103,
    # reductions over one leading dimension: attr = (dim, 0); the result has the input's shape
    # with that dimension dropped or kept as 1
    "sum_dim": 104, "mean_dim": 105, "amax_dim": 106, "amin_dim": 107,
    # composites over the last dim
    "softmax": 128, "log_softmax": 129, "layer_norm": 130, "rms_norm": 131,
    # index operators on leading dimensions (they move data, they compute nothing):
    # roll: attr = (dim, shift); slice: attr = (dim, start), length from the output shape; a second
    # dimension of either goes into the immediates as (1 + dim, shift / start), 0 meaning none;
    # view: regroups leading dimensions, the last one and the element order unchanged
    "roll": 160, "slice": 161, "view": 162,
    # cat: attr = (dim, 0); the concatenation of its operands along dim.  With one operand it is
    # the identity (graph traces keep such nodes)
    "cat": 163,
    # contiguous: the same values in the dense row-major layout every tensor here already has: the
    # identity (graph traces keep such nodes after index operators)
    "contiguous": 164,
}


@dataclass(frozen=True)
class Imm:
    """A scalar constant operand (stored as f64 in the node record)."""
    value: float


@dataclass
class _Tensor:
    dtype: int
    role: int
    dims: tuple


@dataclass
class _Node:
    opcode: int
    ins: list
    outs: list
    imm: list = field(default_factory=lambda: [0.0, 0.0])
    attr: list = field(default_factory=lambda: [0, 0])


class GraphBuilder:
    """Accumulates tensors and nodes, then serialises them with :meth:`build`.

    Shapes are given explicitly for every value (sigma is part of the graph);
    the builder performs no shape inference and no validation beyond ranks and
    operand counts: judging a descriptor is the job of whoever parses it.
    """

    def __init__(self) -> None:
        self._tensors: List[_Tensor] = []
        self._nodes: List[_Node] = []

    # -- tensors -----------------------------------------------------------
    def _add_tensor(self, dtype: int, dims: Sequence[int], role: int) -> int:
        dims = tuple(int(d) for d in dims)
        if len(dims) > MAX_RANK:
            raise ValueError("rank above 4")
        self._tensors.append(_Tensor(dtype, role, dims))
        return len(self._tensors) - 1

    def input(self, dtype: int, dims: Sequence[int]) -> int:
        return self._add_tensor(dtype, dims, ROLE_INPUT)

    def mark_output(self, tid: int) -> int:
        self._tensors[tid].role |= ROLE_OUTPUT
        return tid

    # -- nodes -------------------------------------------------------------
    def node(self, op: str, ins: Sequence[Union[int, Imm]], out_dtypes: Sequence[int],
             out_dims: Sequence[Sequence[int]], attr: Sequence[int] = (0, 0),
             extra_imm: Sequence[float] = ()) -> List[int]:
        """Append a node; returns the ids of its output tensors.

        Operands that are :class:`Imm` go into the node's immediate slots in
        order of appearance; ``extra_imm`` fills the remaining slots (eps of the
        normalisations lives there).
        """
        if len(ins) > 4 or len(out_dtypes) > 3 or len(out_dtypes) != len(out_dims):
            raise ValueError("operand count")
        imm: List[float] = []
        slots: List[int] = []
        for x in ins:
            if isinstance(x, Imm):
                if len(imm) >= 2:
                    raise ValueError("more than two immediates")
                slots.append(IMM0 - len(imm))
                imm.append(float(x.value))
            else:
                slots.append(int(x))
        for v in extra_imm:
            if len(imm) >= 2:
                raise ValueError("more than two immediates")
            imm.append(float(v))
        while len(imm) < 2:
            imm.append(0.0)
        outs = [self._add_tensor(dt, dm, 0) for dt, dm in zip(out_dtypes, out_dims)]
        a = list(attr) + [0] * (2 - len(attr))
        self._nodes.append(_Node(OPCODES[op], slots, outs, imm, a[:2]))
        return outs

    def op(self, name: str, ins: Sequence[Union[int, Imm]], dtype: int, dims: Sequence[int],
           **kw) -> int:
        """Single-output convenience form of :meth:`node`."""
        return self.node(name, ins, [dtype], [dims], **kw)[0]

    # -- serialisation -----------------------------------------------------
    def build(self) -> bytes:
        out = [struct.pack("<IHHII", MAGIC, VERSION, 0, len(self._tensors), len(self._nodes))]
        for t in self._tensors:
            dims = list(t.dims) + [0] * (MAX_RANK - len(t.dims))
            out.append(struct.pack("<BBBBI4q", t.dtype, t.role, len(t.dims), 0, 0, *dims))
        for n in self._nodes:
            ins = list(n.ins) + [0] * (4 - len(n.ins))
            outs = list(n.outs) + [0] * (3 - len(n.outs))
            out.append(struct.pack("<HBB4I3I2d2q", n.opcode, len(n.ins), len(n.outs),
                                   *ins, *outs, *n.imm, *n.attr))
        return b"".join(out)

    # -- introspection used by callers that allocate buffers ----------------
    def input_ids(self) -> List[int]:
        return [i for i, t in enumerate(self._tensors) if t.role & ROLE_INPUT]

    def output_ids(self) -> List[int]:
        return [i for i, t in enumerate(self._tensors) if t.role & ROLE_OUTPUT]

    def tensor_meta(self, tid: int):
        t = self._tensors[tid]
        return t.dtype, t.dims
