"""Host-side logic of the library, on the CPU: the shared library loads and exports what
include/pn.h declares, descriptors are validated into the documented status codes, the
lowering picks the documented kernel families, and the kernel generated for each benchmark
graph compiles for sm_100a.  No GPU is touched (handles are created plan-only)."""
import ctypes
import os
import re
import struct
import sys

import pytest

import paper_2605_29357_b200 as pn
from paper_2605_29357_b200 import binding
from pn_workloads import configs as C
from pn_workloads import descriptor as D
from pn_workloads.descriptor import GraphBuilder, Imm

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
PLAN = pn.FLAG_PLAN_ONLY


def test_library_exports_every_declared_symbol():
    lib = pn.load_library()
    header = open(os.path.join(ROOT, "include", "pn.h")).read()
    declared = set(re.findall(r"\b(pn_[a-z_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_status_strings_and_null_arguments():
    lib = pn.load_library()
    assert lib.pn_status_string(0) == b"ok"
    assert lib.pn_status_string(-4) == b"shape error"
    h = ctypes.c_void_p()
    assert lib.pn_graph_create(None, 0, 0, PLAN, ctypes.byref(h)) == -1
    assert lib.pn_graph_destroy(None) == 0
    assert lib.pn_graph_query(None, 1, None, 0) == -1


def _status(desc, flags=PLAN):
    try:
        pn.Graph(bytes(desc), 0, flags).close()
        return 0
    except pn.PnError as e:
        return e.status


def test_malformed_descriptors_are_rejected():
    good = bytearray(C.c1(M=2, N=8).desc)
    assert _status(good) == 0
    assert _status(good[:10]) == -2
    bad = good[:]; bad[0] ^= 0xFF
    assert _status(bad) == -2                                   # magic
    assert _status(good + b"\0") == -2                          # length
    bad = good[:]; struct.pack_into("<H", bad, 16 + 40 * 8, 999)
    assert _status(bad) == -3                                   # unknown opcode
    bad = good[:]; struct.pack_into("<I", bad, 16 + 40 * 8 + 4, 77)
    assert _status(bad) == -2                                   # operand id out of range
    bad = good[:]; bad[16] = 9
    assert _status(bad) == -2                                   # unknown dtype
    # a node reading a tensor that a later node produces
    g = GraphBuilder(); x = g.input(D.F32, (4,))
    t_late = g._add_tensor(D.F32, (4,), 0)
    y = g.op("add", [x, t_late], D.F32, (4,))
    g.node("neg", [x], [D.F32], [(4,)])
    g._nodes[-1].outs = [t_late]; g._tensors.pop()
    g.mark_output(y)
    assert _status(g.build()) == -2


def test_shape_and_support_errors():
    g = GraphBuilder(); a = g.input(D.F32, (4, 8)); b = g.input(D.F32, (3, 8))
    g.mark_output(g.op("add", [a, b], D.F32, (4, 8)))
    assert _status(g.build()) == -4                             # operands do not broadcast
    g = GraphBuilder(); a = g.input(D.F32, (4, 8))
    g.mark_output(g.op("sum", [a], D.F32, (8,)))
    assert _status(g.build()) == -4                             # reduction result of the wrong shape
    g = GraphBuilder(); a = g.input(D.F32, (4, 8))
    g.mark_output(g.op("argmax", [a], D.F32, (4,)))
    assert _status(g.build()) == -3                             # index results are integers
    g = GraphBuilder(); a = g.input(D.F32, (4, 0))
    g.mark_output(g.op("neg", [a], D.F32, (4, 0)))
    assert _status(g.build()) == 0                              # empty tensors: a no-op handle
    g = GraphBuilder(); ins = [g.input(D.F32, (8,)) for _ in range(13)]
    t = ins[0]
    for u in ins[1:]:
        t = g.op("add", [t, u], D.F32, (8,))
    g.mark_output(t)
    assert _status(g.build(), PLAN | pn.FLAG_ONE_KERNEL) == -5  # more inputs than a kernel takes
    cut = pn.Graph(g.build(), 0, PLAN)                          # ... so the graph is cut into two fused launches
    assert cut.n_kernels == 2 and cut.workspace_bytes > 0
    assert _status(g.build(), PLAN | pn.FLAG_UNFUSED) == 0      # and one node at a time fits anyway


FAMILY = {"c1": "pointwise", "c2": "warp-per-row", "c3": "block-per-row", "c4": "split-row",
          "c5": "block-per-row"}
FULL = {"c1": dict(M=1024, N=1024), "c2": dict(B=512, Q=512, K=512), "c3": dict(M=16384, N=4096),
        "c4": dict(M=64, N=262144), "c5": dict(M=8192, N=14336)}


def _descriptor_only(cfg, kw):
    """The full-size graph without drawing its inputs: descriptors depend on shapes only, so
    take one built at a tiny size of every free dimension and patch nothing -- instead build
    the graph at full size through a generator stub."""
    import numpy as np
    real_draw = C._draw
    C._draw = lambda rng, kind, shape, a, b, chunk=0: np.zeros(shape, dtype=np.float32)
    try:
        return C.CONFIGS[cfg](**kw)
    finally:
        C._draw = real_draw


@pytest.mark.parametrize("cfg", list(FAMILY))
def test_lowering_of_the_benchmark_graphs(cfg):
    w = _descriptor_only(cfg, FULL[cfg])
    g = pn.Graph(w.desc, 0, PLAN)
    assert g.n_kernels == 1 and g.n_nodes == w.n_nodes
    assert g.compulsory_bytes == w.compulsory_bytes
    k = g.kernel_info[0]
    assert pn.FAMILY_NAMES[k["family"]] == FAMILY[cfg]
    if cfg == "c3":   # fp32 gamma / beta re-read by every row: groups of 4 (128-bit accesses for them, 64-bit for the bf16 rows)
        assert k["vl"] == 4 and k["ng"] == 8
    else:
        assert k["vl"] * (2 if cfg in ("c2", "c5") else 4) == 16           # 128-bit accesses
    if cfg == "c4":   # 64 long rows, a single stage: independent blocks over slices of the rows
        assert k["grid"] % 64 == 0 and k["grid"] >= 8 * 148 and g.workspace_bytes > 0
        gc = pn.Graph(w.desc, 0, PLAN | pn.FLAG_FORCE_CLUSTER)   # clusters when asked for: every SM still gets work
        kc = gc.kernel_info[0]
        assert kc["cluster"] in (2, 4, 8) and kc["grid"] % kc["cluster"] == 0 and 64 * kc["cluster"] >= 148
    if cfg in ("c2", "c3"):
        assert k["chunks"] == 1                                             # row resident in registers
    gu = pn.Graph(w.desc, 0, PLAN | pn.FLAG_UNFUSED)
    assert gu.n_kernels == w.n_nodes and gu.workspace_bytes > 0
    assert [m for m in g.input_meta] == [(dt, tuple(d)) for dt, d in w.input_meta]
    assert [m for m in g.output_meta] == [(dt, tuple(d)) for dt, d in w.output_meta]


COMPULSORY = {"c1": 12591104, "c2": 537133056, "c3": 402817024, "c4": 67109632, "c5": 822194176}


@pytest.mark.parametrize("cfg", list(COMPULSORY))
def test_compulsory_bytes(cfg):
    w = _descriptor_only(cfg, FULL[cfg])
    assert w.compulsory_bytes == COMPULSORY[cfg]


@pytest.mark.parametrize("flags", [0, pn.FLAG_FORCE_SCALAR, pn.FLAG_FORCE_CLUSTER | pn.FLAG_FORCE_MULTICHUNK])
@pytest.mark.parametrize("cfg", list(FAMILY))
def test_generated_kernels_compile(cfg, flags):
    w = C.CONFIGS[cfg](**C.SMALL[cfg])
    g = pn.Graph(w.desc, 0, PLAN | flags)
    src = g.codegen(0, compile=True)
    assert "__global__ void PN_LAUNCH_BOUNDS pn_spec_" in src and "struct Spec" in src


def test_forced_families():
    w = C.c3(M=8, N=1024)
    for flag, fam in ((pn.FLAG_FORCE_WARP, "warp-per-row"), (pn.FLAG_FORCE_BLOCK, "block-per-row"),
                      (pn.FLAG_FORCE_CLUSTER, "cluster-per-row")):
        k = pn.Graph(w.desc, 0, PLAN | flag).kernel_info[0]
        assert pn.FAMILY_NAMES[k["family"]] == fam
    k = pn.Graph(w.desc, 0, PLAN | pn.FLAG_FORCE_SCALAR).kernel_info[0]
    assert k["vl"] == 1
    k = pn.Graph(w.desc, 0, PLAN | pn.FLAG_FORCE_BLOCK | pn.FLAG_FORCE_MULTICHUNK).kernel_info[0]
    assert k["chunks"] > 1
    # a row length that is not a multiple of the vector width falls back to element accesses
    k = pn.Graph(C.c3(M=4, N=1001).desc, 0, PLAN).kernel_info[0]
    assert k["vl"] == 1


# ---- index operators (Section 3.2: index-remapped loads) --------------------------------
def test_index_chain_becomes_addressing_of_one_kernel():
    w = _descriptor_only_n1()
    g = pn.Graph(w.desc, 0, PLAN)
    assert g.n_kernels == 1
    k = g.kernel_info[0]
    assert k["rows"] == 128 * 128 and k["row_len"] == 96 and k["stages"] == 2
    src = g.codegen(0, compile=True)
    m = re.search(r"static PN_DEV bool io_mapped\(.*?\n((?:.*\n)*?)\s*default: return false;", src)
    assert m and m.group(1).count("return true") == 1          # exactly the rolled input
    # rolls by +3 over 133 read from (i + 130) mod 133; source strides are those of the 133 x 133 map
    assert "IoMap{1, 128, 128, 0, 130, 130, 0, 133, 133," in src and "12768ll, 96ll}" in src
    gu = pn.Graph(w.desc, 0, PLAN | pn.FLAG_UNFUSED)
    assert gu.n_kernels > 8                                    # every index op is a copy kernel there
    for i in range(gu.n_kernels):
        gu.codegen(i, compile=True)


def _descriptor_only_n1():
    import numpy as np
    real_draw = C._draw
    C._draw = lambda rng, kind, shape, a, b, chunk=0: np.zeros(shape, dtype=np.float32)
    try:
        return C.n1()
    finally:
        C._draw = real_draw


def test_index_operator_errors():
    def one(op, in_shape, out_shape, attr, dtype_out=D.F32):
        g = GraphBuilder(); x = g.input(D.F32, in_shape)
        g.mark_output(g.op(op, [x], dtype_out, out_shape, attr=attr))
        return _status(g.build())
    assert one("roll", (4, 8), (4, 8), [0, 1]) == 0
    assert one("roll", (4, 8), (4, 8), [1, 1]) == 0             # the last dimension: a circular shift of the columns
    assert one("roll", (4, 8), (4, 8), [2, 1]) == -4            # no such dimension
    assert one("roll", (4, 8), (5, 8), [0, 1]) == -4            # a roll keeps the shape
    assert one("roll", (4, 8), (4, 8), [0, 1], D.BF16) == -3    # and the dtype
    assert one("slice", (4, 8), (3, 8), [0, 1]) == 0
    assert one("slice", (4, 8), (3, 8), [0, 2]) == -4           # 2 + 3 > 4
    assert one("slice", (4, 8), (3, 4), [0, 0]) == -4           # a slice of dimension 0 leaves the last one whole
    assert one("slice", (4, 8), (4, 4), [1, 4]) == 0            # a slice of the last dimension: the second half
    assert one("slice", (4, 8), (4, 4), [1, 5]) == -4           # 5 + 4 > 8
    assert one("view", (4, 6, 8), (3, 8, 8), [0, 0]) == 0
    assert one("view", (4, 6, 8), (3, 8, 4), [0, 0]) == -4
    # index operators read graph inputs (or chains of them), not computed values
    g = GraphBuilder(); x = g.input(D.F32, (4, 8))
    y = g.op("neg", [x], D.F32, (4, 8))
    g.mark_output(g.op("roll", [y], D.F32, (4, 8), attr=[0, 1]))
    assert _status(g.build(), PLAN | pn.FLAG_ONE_KERNEL) == -3
    assert pn.Graph(g.build(), 0, PLAN).n_kernels == 2          # cut after the computed value: the roll is then a copy of its own
    assert _status(g.build(), PLAN | pn.FLAG_UNFUSED) == 0      # one node at a time it is a plain copy
    # roll after slice on the same dimension would need a second modulus
    g = GraphBuilder(); x = g.input(D.F32, (6, 8))
    s = g.op("slice", [x], D.F32, (4, 8), attr=[0, 1])
    g.mark_output(g.op("roll", [s], D.F32, (4, 8), attr=[0, 1]))
    assert _status(g.build(), PLAN | pn.FLAG_ONE_KERNEL) == -3
    assert pn.Graph(g.build(), 0, PLAN).n_kernels == 2
    assert _status(g.build(), PLAN | pn.FLAG_UNFUSED) == 0


# ---- reductions over a leading dimension (the column-reduce family) ----------------------
def _descriptor_only_n2(**kw):
    import numpy as np
    real_draw = C._draw
    C._draw = lambda rng, kind, shape, a, b, chunk=0: np.zeros(shape, dtype=np.float32)
    try:
        return C.n2(**kw)
    finally:
        C._draw = real_draw


def test_masked_mean_pooling_lowers_to_one_column_kernel():
    w = _descriptor_only_n2()
    g = pn.Graph(w.desc, 0, PLAN)
    assert g.n_kernels == 1 and g.n_nodes == 7
    k = g.kernel_info[0]
    assert pn.FAMILY_NAMES[k["family"]] == "column-reduce" and k["stages"] == 2
    assert k["rows"] == 256 and k["row_len"] == 1024 and k["vl"] == 8      # 128-bit loads of the bf16 hidden states
    assert g.compulsory_bytes == 256 * 512 * 1024 * 2 + 256 * 512 * 8 + 256 * 1024 * 4
    src = g.codegen(0, compile=True)
    assert "pn::column_body<pn::Spec>" in src and src.count("op_accum<8>") + src.count("op_accum_u<8>") == 2   # both sums in one walk
    gu = pn.Graph(w.desc, 0, PLAN | pn.FLAG_UNFUSED)
    assert gu.n_kernels == 7
    for i in range(gu.n_kernels):
        gu.codegen(i, compile=True)
    # ragged and scalar-access shapes compile too
    for kw in (dict(B=3, S=37, Dh=203), dict(B=2, S=9, Dh=64, dense_mask=True, mask_dtype=D.I8)):
        pn.Graph(_descriptor_only_n2(**kw).desc, 0, PLAN).codegen(0, compile=True)


def test_unsupported_column_forms_are_refused():
    def status(g, extra=pn.FLAG_ONE_KERNEL):
        try:
            pn.Graph(g.build(), 0, PLAN | extra).close()
            return 0
        except pn.PnError as e:
            return e.status
    g = GraphBuilder(); x = g.input(D.F32, (4, 6, 8))
    s = g.op("sum_dim", [x], D.F32, (4, 1, 8), attr=[1, 0])
    g.mark_output(g.op("sub", [x, s], D.F32, (4, 6, 8)))             # needs a second pass over the dimension
    assert status(g) == -3
    assert pn.Graph(g.build(), 0, PLAN).n_kernels == 2               # ... which is what two launches are
    g = GraphBuilder(); x = g.input(D.F32, (4, 6, 8))
    g.mark_output(g.op("sum_dim", [x], D.F32, (4, 6), attr=[2, 0]))  # the last dimension has its own opcodes
    assert status(g) == -3
    g = GraphBuilder(); x = g.input(D.F32, (4, 6, 8))
    g.mark_output(g.op("sum_dim", [x], D.F32, (4, 7), attr=[1, 0]))
    assert status(g) == -4
    g = GraphBuilder(); x = g.input(D.F32, (4, 6, 8))
    g.mark_output(g.op("sum_dim", [x], D.F32, (4, 8), attr=[1, 0]))
    g.mark_output(g.op("sum_dim", [x], D.F32, (6, 8), attr=[0, 0]))  # two different dimensions in one graph
    assert status(g) == -3
    assert pn.Graph(g.build(), 0, PLAN).n_kernels == 2
    g = GraphBuilder(); x = g.input(D.F32, (4, 6, 8)); y = g.input(D.F32, (4, 6, 8))
    g.mark_output(g.op("cat", [x, y], D.F32, (4, 12, 8), attr=[1, 0]))   # a concatenation of two inputs: each stored into its block
    assert status(g, 0) == 0
    g = GraphBuilder(); x = g.input(D.F32, (4, 6, 8)); y = g.input(D.F32, (4, 5, 8))
    g.mark_output(g.op("cat", [x, y], D.F32, (4, 12, 8), attr=[1, 0]))   # 6 + 5 is not 12
    assert status(g, 0) == -4


def test_checked_accessors_are_compiled_in_only_on_request():
    w = C.c3(**C.SMALL["c3"])
    plain = pn.Graph(w.desc, 0, PLAN)
    checked = pn.Graph(w.desc, 0, PLAN | pn.FLAG_BOUNDS)
    assert plain.codegen(0, compile=True) == checked.codegen(0, compile=True)   # same program; the switch is a macro
    assert _status(w.desc, PLAN | pn.FLAG_BOUNDS | pn.FLAG_UNFUSED | pn.FLAG_STATIC_SCRATCH) == -1


def _create_in_child(env_extra, flags):
    """pn_graph_create (plan only) in a fresh process, so that the library resolves NVRTC under the
    given environment.  Returns (status, detail, specialised)."""
    import subprocess
    code = (
        "import sys; sys.path.insert(0, %r)\n"
        "import paper_2605_29357_b200 as pn\n"
        "from pn_workloads import configs as C\n"
        "w = C.c1(M=4, N=64)\n"
        "try:\n"
        "    g = pn.Graph(w.desc, 0, %d)\n"
        "    print('OK', g.kernel_info[0]['specialised'])\n"
        "except pn.PnError as e:\n"
        "    print('ERR', e.status, e.detail)\n" % (ROOT, flags))
    env = dict(os.environ, **env_extra)
    r = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    return r.stdout.strip().splitlines()[-1]


def test_a_create_that_cannot_specialise_fails_loudly_unless_the_interpreter_is_asked_for():
    missing = {"PN_NVRTC_PATH": "/nonexistent/libnvrtc.so.12"}
    out = _create_in_child(missing, pn.FLAG_PLAN_ONLY)
    assert out.startswith("ERR -8") and "NVRTC not found" in out and "PN_FLAG_ALLOW_INTERPRET" in out
    # asked for by name, or allowed: the handle is lowered for the interpreter kernels
    assert _create_in_child(missing, pn.FLAG_PLAN_ONLY | pn.FLAG_ALLOW_INTERPRET) == "OK 0"
    assert _create_in_child(missing, pn.FLAG_PLAN_ONLY | pn.FLAG_INTERPRET) == "OK 0"
    # with NVRTC where the toolkit puts it, the same create succeeds (plan-only handles report 0: nothing is loaded)
    assert _create_in_child({}, pn.FLAG_PLAN_ONLY).startswith("OK")
    # a run-time library that is there but is not NVRTC is refused as well
    assert _create_in_child({"PN_NVRTC_PATH": pn.library_path()}, pn.FLAG_PLAN_ONLY).startswith("ERR -8")


def test_nodes_that_reach_no_output_are_dropped():
    """A node whose result no graph output depends on is not part of f_G: it costs no launch on the
    unfused path, and what it would need (here a second softmax) is not asked of the kernel."""
    g = GraphBuilder(); x = g.input(D.F32, (4, 64))
    dead = g.op("softmax", [g.op("softmax", [x], D.F32, (4, 64))], D.F32, (4, 64))
    live = g.op("exp", [x], D.F32, (4, 64))
    g.op("add", [dead, live], D.F32, (4, 64))                     # dead as well: nothing reads it
    g.mark_output(live)
    fused = pn.Graph(g.build(), 0, PLAN | pn.FLAG_ONE_KERNEL)
    assert fused.n_kernels == 1 and fused.n_nodes == 4
    assert pn.FAMILY_NAMES[fused.kernel_info[0]["family"]] == "pointwise"
    assert pn.Graph(g.build(), 0, PLAN | pn.FLAG_UNFUSED).n_kernels == 1
