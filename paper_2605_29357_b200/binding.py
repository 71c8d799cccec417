"""ctypes binding of the C-ABI library (include/pn.h): argument marshalling only.

Every step of the computation runs in the CUDA kernels of libpn.so.  There is no CPU
fallback: if the library is missing it is built with nvcc, and if that fails the import
raises.  torch is used by callers for device memory and streams; this module itself only
needs raw device pointers.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Sequence, Tuple

from . import _build

# status codes and flags (numerically as in pn.h)
PN_OK = 0
FLAG_UNFUSED = 1 << 0
FLAG_PLAN_ONLY = 1 << 1
FLAG_ONE_KERNEL = 1 << 3
FLAG_PLAIN_LAUNCH = 1 << 2
FLAG_FORCE_WARP = 1 << 4
FLAG_FORCE_BLOCK = 1 << 5
FLAG_FORCE_CLUSTER = 1 << 6
FLAG_FORCE_SCALAR = 1 << 7
FLAG_FORCE_MULTICHUNK = 1 << 8
FLAG_INTERPRET = 1 << 9
FLAG_NO_HOIST = 1 << 10
FLAG_PREFETCH = 1 << 11
FLAG_STATIC_SCRATCH = 1 << 12
FLAG_BOUNDS = 1 << 13
FLAG_ALLOW_INTERPRET = 1 << 14
FLAG_FORCE_SPLIT = 1 << 15
STATIC_SCRATCH_BYTES = 32 << 20


def tune(cluster: int = 0, block: int = 0, groups: int = 0, waves: int = 0) -> int:
    """Flag bits overriding the lowering's cluster size, block size, groups per tile and grid size
    (waves n: at most 2^(n-1) times the resident CTAs; 7: one CTA per work item)."""
    lg = block.bit_length() - 1 if block else 0
    return ((cluster & 15) << 16) | ((lg & 15) << 20) | ((groups & 31) << 24) | ((waves & 7) << 29)

Q_N_INPUTS, Q_N_OUTPUTS, Q_INPUT_META, Q_OUTPUT_META, Q_COMPULSORY_BYTES = 1, 2, 3, 4, 5
Q_N_KERNELS, Q_N_NODES, Q_WORKSPACE_BYTES, Q_KERNEL_INFO = 6, 7, 8, 9

FAMILY_NAMES = {0: "pointwise", 1: "warp-per-row", 2: "block-per-row", 3: "cluster-per-row", 4: "column-reduce", 5: "split-row"}
EXPORTS = ["pn_graph_create", "pn_graph_run", "pn_graph_run_host", "pn_graph_run_static", "pn_graph_destroy",
           "pn_graph_bind", "pn_bound_run", "pn_bound_run_many", "pn_bound_destroy",
           "pn_graph_query", "pn_graph_codegen", "pn_status_string", "pn_last_error",
           "pn_sequence_create", "pn_sequence_run", "pn_sequence_query", "pn_sequence_destroy",
           "pn_stream_probe"]
SEQ_INDEPENDENT = 1 << 0
MIX_READ, MIX_WRITE, MIX_1_1, MIX_2_1, MIX_4_3 = range(5)
PROBE_LDG, PROBE_LDG_NOALLOC, PROBE_BULK = range(3)


class ProbeConfig(ctypes.Structure):
    """pn_probe_config: how pn_stream_probe moves its bytes."""
    _fields_ = [("loader", ctypes.c_int), ("streaming_stores", ctypes.c_int), ("layout", ctypes.c_int),
                ("block", ctypes.c_int), ("unroll", ctypes.c_int), ("grid", ctypes.c_int),
                ("stages", ctypes.c_int), ("tile_units", ctypes.c_int), ("strip_units", ctypes.c_int),
                ("rows_per_block", ctypes.c_int)]


class PnError(RuntimeError):
    def __init__(self, status: int, what: str, detail: str):
        super().__init__(f"{what}: {detail} (status {status})")
        self.status = status
        self.detail = detail


_lib = None


def library_path() -> str:
    return _build.LIB


def load_library() -> ctypes.CDLL:
    """Load libpn.so, building it first if it is not there.  Raises when neither works."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_build.LIB):
        _build.build_library()
    lib = ctypes.CDLL(_build.LIB)
    vp, vpp = ctypes.c_void_p, ctypes.POINTER(ctypes.c_void_p)
    lib.pn_graph_create.restype = ctypes.c_int
    lib.pn_graph_create.argtypes = [ctypes.c_char_p, ctypes.c_size_t, ctypes.c_int, ctypes.c_uint, vpp]
    for fn in (lib.pn_graph_run, lib.pn_graph_run_host, lib.pn_graph_run_static):
        fn.restype = ctypes.c_int
        fn.argtypes = [vp, vpp, ctypes.c_int, vpp, ctypes.c_int, vp]
    lib.pn_graph_destroy.restype = ctypes.c_int
    lib.pn_graph_destroy.argtypes = [vp]
    lib.pn_graph_bind.restype = ctypes.c_int
    lib.pn_graph_bind.argtypes = [vp, vpp, ctypes.c_int, vpp, ctypes.c_int, vpp]
    lib.pn_bound_run.restype = ctypes.c_int
    lib.pn_bound_run.argtypes = [vp, vp]
    lib.pn_bound_run_many.restype = ctypes.c_int
    lib.pn_bound_run_many.argtypes = [ctypes.POINTER(vp), ctypes.c_int, vp]
    lib.pn_bound_destroy.restype = ctypes.c_int
    lib.pn_bound_destroy.argtypes = [vp]
    lib.pn_graph_query.restype = ctypes.c_int
    lib.pn_graph_query.argtypes = [vp, ctypes.c_int, vp, ctypes.c_size_t]
    lib.pn_graph_codegen.restype = ctypes.c_int
    lib.pn_graph_codegen.argtypes = [vp, ctypes.c_int, ctypes.c_int, ctypes.c_char_p, ctypes.c_size_t,
                                     ctypes.POINTER(ctypes.c_size_t)]
    lib.pn_sequence_create.restype = ctypes.c_int
    lib.pn_sequence_create.argtypes = [ctypes.c_int, vpp, ctypes.POINTER(vpp), ctypes.POINTER(ctypes.c_int),
                                       ctypes.POINTER(vpp), ctypes.POINTER(ctypes.c_int), ctypes.c_uint, vpp]
    lib.pn_sequence_run.restype = ctypes.c_int
    lib.pn_sequence_run.argtypes = [vp, vp]
    lib.pn_sequence_query.restype = ctypes.c_int
    lib.pn_sequence_query.argtypes = [vp, ctypes.c_int, vp, ctypes.c_size_t]
    lib.pn_sequence_destroy.restype = ctypes.c_int
    lib.pn_sequence_destroy.argtypes = [vp]
    lib.pn_stream_probe.restype = ctypes.c_int
    lib.pn_stream_probe.argtypes = [ctypes.c_int, ctypes.POINTER(ProbeConfig), vp, vp, vp, vp, ctypes.c_size_t, vp, vp]
    lib.pn_status_string.restype = ctypes.c_char_p
    lib.pn_status_string.argtypes = [ctypes.c_int]
    lib.pn_last_error.restype = ctypes.c_char_p
    lib.pn_last_error.argtypes = []
    _lib = lib
    return lib


def _check(status: int, what: str) -> None:
    if status != PN_OK:
        lib = load_library()
        raise PnError(status, what + ": " + lib.pn_status_string(status).decode(), lib.pn_last_error().decode())


def stream_probe(mix: int, cfg: ProbeConfig, a: int, b: int, c: int, d: int, units: int, status_word: int,
                 stream: int = 0) -> None:
    """pn_stream_probe on device pointers (integers; 0 for the buffers the mix does not use)."""
    vp = ctypes.c_void_p
    _check(load_library().pn_stream_probe(mix, ctypes.byref(cfg), vp(a), vp(b), vp(c), vp(d), units, vp(status_word),
                                          vp(stream)), "pn_stream_probe")


class Graph:
    """One lowered graph (pn_graph_t).  ``desc`` is a serialized descriptor."""

    def __init__(self, desc: bytes, device: int = 0, flags: int = 0):
        self._lib = load_library()
        self._h = ctypes.c_void_p()
        _check(self._lib.pn_graph_create(desc, len(desc), device, flags, ctypes.byref(self._h)), "pn_graph_create")
        self.n_inputs = self._query(Q_N_INPUTS, 1)[0]
        self.n_outputs = self._query(Q_N_OUTPUTS, 1)[0]

    # -- pn_graph_query -----------------------------------------------------
    def _query(self, what: int, n: int) -> List[int]:
        buf = (ctypes.c_int64 * max(n, 1))()
        _check(self._lib.pn_graph_query(self._h, what, buf, ctypes.sizeof(buf)), "pn_graph_query")
        return list(buf[:n])

    def _meta(self, what: int, n: int) -> List[Tuple[int, tuple]]:
        v = self._query(what, 6 * n)
        return [(v[6 * i], tuple(v[6 * i + 2: 6 * i + 2 + v[6 * i + 1]])) for i in range(n)]

    @property
    def input_meta(self):
        return self._meta(Q_INPUT_META, self.n_inputs)

    @property
    def output_meta(self):
        return self._meta(Q_OUTPUT_META, self.n_outputs)

    @property
    def compulsory_bytes(self) -> int:
        return self._query(Q_COMPULSORY_BYTES, 1)[0]

    @property
    def n_kernels(self) -> int:
        return self._query(Q_N_KERNELS, 1)[0]

    @property
    def n_nodes(self) -> int:
        return self._query(Q_N_NODES, 1)[0]

    @property
    def bounds_status(self) -> int:
        """Status word of a FLAG_BOUNDS handle: 0 unless an access fell outside its tensor."""
        return self._query(10, 1)[0]

    @property
    def kernel_cache(self) -> Tuple[int, int]:
        """(generated kernels loaded in this process, how many of them a live handle uses)."""
        v = self._query(11, 2)
        return v[0], v[1]

    @property
    def workspace_bytes(self) -> int:
        return self._query(Q_WORKSPACE_BYTES, 1)[0]

    @property
    def kernel_info(self) -> List[dict]:
        n = self.n_kernels
        v = self._query(Q_KERNEL_INFO, 14 * n)
        keys = ["family", "grid", "block", "cluster", "smem_bytes", "vl", "ng", "chunks",
                "code_words", "stages", "rows", "row_len", "specialised", "slices"]
        return [dict(zip(keys, v[14 * i: 14 * i + 14])) for i in range(n)]

    def codegen(self, kernel: int = 0, compile: bool = False) -> str:
        """Generated CUDA source of one launch; with compile=True also compiled by NVRTC."""
        need = ctypes.c_size_t()
        _check(self._lib.pn_graph_codegen(self._h, kernel, 0, None, 0, ctypes.byref(need)), "pn_graph_codegen")
        buf = ctypes.create_string_buffer(need.value + 1)
        _check(self._lib.pn_graph_codegen(self._h, kernel, 1 if compile else 0, buf, need.value + 1, None),
               "pn_graph_codegen")
        return buf.value.decode()

    # -- pn_graph_run / pn_graph_run_host -------------------------------------
    @staticmethod
    def _ptr_array(ptrs: Sequence[int]):
        return (ctypes.c_void_p * max(len(ptrs), 1))(*[ctypes.c_void_p(int(p)) for p in ptrs])

    def run(self, input_ptrs: Sequence[int], output_ptrs: Sequence[int], stream: int = 0) -> None:
        """Enqueue one evaluation on device pointers (integers) and a cudaStream_t handle."""
        _check(self._lib.pn_graph_run(self._h, self._ptr_array(input_ptrs), len(input_ptrs),
                                      self._ptr_array(output_ptrs), len(output_ptrs),
                                      ctypes.c_void_p(stream)), "pn_graph_run")

    def bind(self, input_ptrs: Sequence[int], output_ptrs: Sequence[int]) -> "Bound":
        """pn_graph_bind: a callable `f(stream=0)` that enqueues one evaluation on these device
        pointers.  The argument checks run once, here; each call is pn_bound_run, one launch
        call per kernel."""
        return Bound(self, input_ptrs, output_ptrs)

    def run_host(self, input_ptrs: Sequence[int], output_ptrs: Sequence[int], stream: int = 0) -> None:
        """Evaluate on HOST buffers (addresses): copy in, run, copy out, wait."""
        _check(self._lib.pn_graph_run_host(self._h, self._ptr_array(input_ptrs), len(input_ptrs),
                                           self._ptr_array(output_ptrs), len(output_ptrs),
                                           ctypes.c_void_p(stream)), "pn_graph_run_host")

    def run_static(self, input_ptrs: Sequence[int], output_ptrs: Sequence[int], stream: int = 0) -> None:
        """pn_graph_run_static: the unfused evaluation with its intermediates in the library's
        fixed scratch array, for callers that may not allocate device memory.  The handle must
        have been created with FLAG_UNFUSED | FLAG_STATIC_SCRATCH.  Calls share the array:
        keep them stream-ordered."""
        _check(self._lib.pn_graph_run_static(self._h, self._ptr_array(input_ptrs), len(input_ptrs),
                                             self._ptr_array(output_ptrs), len(output_ptrs),
                                             ctypes.c_void_p(stream)), "pn_graph_run_static")

    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h:
            self._lib.pn_graph_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class BoundList:
    """Several bound launches run in order by one call (pn_bound_run_many)."""

    def __init__(self, bound: Sequence["Bound"]):
        self._keep = list(bound)
        self._n = len(self._keep)
        self._arr = (ctypes.c_void_p * max(self._n, 1))(*[b._h.value for b in self._keep])
        self._run = load_library().pn_bound_run_many

    def __call__(self, stream: int = 0) -> None:
        st = self._run(self._arr, self._n, ctypes.c_void_p(stream))
        if st != PN_OK:
            _check(st, "pn_bound_run_many")


class Bound:
    """pn_bound_t: the launches of a Graph with one set of device pointers filled in."""

    def __init__(self, graph: Graph, input_ptrs: Sequence[int], output_ptrs: Sequence[int]):
        self._lib = graph._lib
        self._graph = graph                      # the handle must outlive its bound launches
        self._h = ctypes.c_void_p()
        _check(self._lib.pn_graph_bind(graph._h, Graph._ptr_array(input_ptrs), len(input_ptrs),
                                       Graph._ptr_array(output_ptrs), len(output_ptrs), ctypes.byref(self._h)),
               "pn_graph_bind")
        self._run = self._lib.pn_bound_run

    def __call__(self, stream: int = 0, _vp=ctypes.c_void_p) -> None:
        st = self._run(self._h, _vp(stream))
        if st != PN_OK:
            _check(st, "pn_bound_run")

    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h:
            self._lib.pn_bound_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Sequence:
    """pn_sequence_t: n (graph, input pointers, output pointers) items recorded once and replayed
    with one call.  ``items`` is a list of (Graph, [input device pointers], [output device
    pointers]); with ``independent=True`` the caller states that no item touches what another
    writes, and the items may overlap on the GPU."""

    def __init__(self, items, independent: bool = False):
        self._lib = load_library()
        self._h = ctypes.c_void_p()
        self._graphs = [g for g, _, _ in items]          # the handles must outlive the sequence
        n = len(items)
        vpp = ctypes.POINTER(ctypes.c_void_p)
        gh = (ctypes.c_void_p * max(n, 1))(*[g._h for g, _, _ in items])
        ins = [Graph._ptr_array(i) for _, i, _ in items]
        outs = [Graph._ptr_array(o) for _, _, o in items]
        in_pp = (vpp * max(n, 1))(*[ctypes.cast(a, vpp) for a in ins])
        out_pp = (vpp * max(n, 1))(*[ctypes.cast(a, vpp) for a in outs])
        n_in = (ctypes.c_int * max(n, 1))(*[len(i) for _, i, _ in items])
        n_out = (ctypes.c_int * max(n, 1))(*[len(o) for _, _, o in items])
        _check(self._lib.pn_sequence_create(n, gh, in_pp, n_in, out_pp, n_out,
                                            SEQ_INDEPENDENT if independent else 0, ctypes.byref(self._h)),
               "pn_sequence_create")

    def _query(self, what: int) -> int:
        v = ctypes.c_int64()
        _check(self._lib.pn_sequence_query(self._h, what, ctypes.byref(v), 8), "pn_sequence_query")
        return int(v.value)

    @property
    def n_items(self) -> int:
        return self._query(1)

    @property
    def n_kernels(self) -> int:
        return self._query(2)

    def run(self, stream: int = 0) -> None:
        _check(self._lib.pn_sequence_run(self._h, ctypes.c_void_p(stream)), "pn_sequence_run")

    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h:
            self._lib.pn_sequence_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
