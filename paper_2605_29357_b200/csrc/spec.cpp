// spec.cpp -- specialisation of a planned launch: the bytecode of a plan is translated,
// instruction by instruction, into straight-line calls of the same op_* device functions the
// interpreter dispatches to, wrapped in the common kernel body, and compiled for sm_100a with
// NVRTC when the handle is created.  The result computes exactly what the interpreter would,
// without the per-instruction decode and with registers allocated by the compiler.
//
// NVRTC and the driver API are opened with dlopen, so that the library loads (and the
// interpreter works) on machines that have neither.  NVRTC is looked for at the toolkit's full
// path first (PN_NVRTC_PATH, then CUDA_HOME / CUDA_PATH, then /usr/local/cuda) and by its bare
// soname last, and bound locally: a process that has another NVRTC loaded under the same soname
// (a framework's bundled copy, possibly older) still gets the toolkit's.
//
// Loaded kernels live in a process-wide cache keyed by a hash of (device, source, options),
// reference-counted by the handles that use them; entries nobody uses any more are unloaded,
// least recently used first, once the cache holds more than kCacheCap modules.  With
// PN_CACHE_DIR set, compiled cubins are also kept on disk there, keyed by the same hash plus the
// NVRTC version, so that a second process pays no compilation.
#include <cuda.h>
#include <dlfcn.h>
#include <nvrtc.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>
#include <sys/stat.h>
#include <unistd.h>

#include <algorithm>
#include <map>
#include <mutex>
#include <string>
#include <tuple>
#include <vector>

#include "graph.h"
#include "spec.h"

namespace pn {

namespace {

// NVRTC options: the fixed ones plus, for experiments, whatever PN_NVRTC_FLAGS lists
// (space separated, e.g. "-DPN_SOME_SWITCH=1").
std::vector<std::string> nvrtc_options() {
  std::vector<std::string> o = {"-arch=sm_100a", "-std=c++17", "-lineinfo"};
  if (const char* e = getenv("PN_NVRTC_FLAGS")) {
    std::string cur;
    for (const char* c = e;; ++c) {
      if (*c == ' ' || *c == '\0') { if (!cur.empty()) o.push_back(cur); cur.clear(); if (!*c) break; }
      else cur.push_back(*c);
    }
  }
  return o;
}

// plan.h followed by device_lib.cuh, as text (written by the build step)
const char kDeviceSource[] =
#include "_build/device_src.inc"
    ;

struct Api {
  bool ok = false;
  std::string why;
  // nvrtc
  nvrtcResult (*CreateProgram)(nvrtcProgram*, const char*, const char*, int, const char* const*, const char* const*) = nullptr;
  nvrtcResult (*CompileProgram)(nvrtcProgram, int, const char* const*) = nullptr;
  nvrtcResult (*GetProgramLogSize)(nvrtcProgram, size_t*) = nullptr;
  nvrtcResult (*GetProgramLog)(nvrtcProgram, char*) = nullptr;
  nvrtcResult (*GetCUBINSize)(nvrtcProgram, size_t*) = nullptr;
  nvrtcResult (*GetCUBIN)(nvrtcProgram, char*) = nullptr;
  nvrtcResult (*DestroyProgram)(nvrtcProgram*) = nullptr;
  nvrtcResult (*Version)(int*, int*) = nullptr;
  int nvrtc_major = 0, nvrtc_minor = 0;
  std::string nvrtc_path;
  // driver
  CUresult (*ModuleLoadData)(CUmodule*, const void*) = nullptr;
  CUresult (*ModuleGetFunction)(CUfunction*, CUmodule, const char*) = nullptr;
  CUresult (*ModuleUnload)(CUmodule) = nullptr;
  CUresult (*FuncSetAttribute)(CUfunction, CUfunction_attribute, int) = nullptr;
  CUresult (*FuncGetAttribute)(int*, CUfunction_attribute, CUfunction) = nullptr;
  CUresult (*LaunchKernelEx)(const CUlaunchConfig*, CUfunction, void**, void**) = nullptr;
  CUresult (*OccupancyMaxActiveBlocks)(int*, CUfunction, int, size_t) = nullptr;
  CUresult (*GetErrorString)(CUresult, const char**) = nullptr;
};

template <class F>
bool sym(void* lib, const char* name, F& f, std::string& why) {
  f = reinterpret_cast<F>(dlsym(lib, name));
  if (!f) { why = std::string("symbol not found: ") + name; return false; }
  return true;
}

const Api& api() {
  static Api a;
  static std::once_flag once;
  std::call_once(once, [] {
    // where to look for NVRTC: an explicit path (then nothing else), the toolkit's directories, the soname
    std::vector<std::string> names;
    if (const char* e = getenv("PN_NVRTC_PATH")) names.push_back(e);
    else {
      for (const char* var : {"CUDA_HOME", "CUDA_PATH"})
        if (const char* e = getenv(var)) names.push_back(std::string(e) + "/lib64/libnvrtc.so.12");
      names.push_back("/usr/local/cuda/lib64/libnvrtc.so.12");
      names.push_back("libnvrtc.so.12");
      names.push_back("libnvrtc.so");
    }
    void* rt = nullptr;
    for (const std::string& n : names)
      if ((rt = dlopen(n.c_str(), RTLD_NOW | RTLD_LOCAL))) { a.nvrtc_path = n; break; }
    if (!rt) { a.why = "NVRTC not found (tried " + names.front() + (names.size() > 1 ? " and " + std::to_string(names.size() - 1) + " more" : std::string()) + ")"; return; }
    bool ok = sym(rt, "nvrtcCreateProgram", a.CreateProgram, a.why) && sym(rt, "nvrtcCompileProgram", a.CompileProgram, a.why) &&
              sym(rt, "nvrtcGetProgramLogSize", a.GetProgramLogSize, a.why) && sym(rt, "nvrtcGetProgramLog", a.GetProgramLog, a.why) &&
              sym(rt, "nvrtcGetCUBINSize", a.GetCUBINSize, a.why) && sym(rt, "nvrtcGetCUBIN", a.GetCUBIN, a.why) &&
              sym(rt, "nvrtcDestroyProgram", a.DestroyProgram, a.why) && sym(rt, "nvrtcVersion", a.Version, a.why);
    if (!ok) { a.CreateProgram = nullptr; return; }
    a.Version(&a.nvrtc_major, &a.nvrtc_minor);
    const char* cu_name = getenv("PN_LIBCUDA_PATH") ? getenv("PN_LIBCUDA_PATH") : "libcuda.so.1";
    void* cu = dlopen(cu_name, RTLD_NOW | RTLD_LOCAL);   // absent on machines without a GPU
    if (!cu) { a.why = std::string(cu_name) + " not found (the CUDA driver library)"; return; }
    ok = sym(cu, "cuModuleLoadData", a.ModuleLoadData, a.why) && sym(cu, "cuModuleGetFunction", a.ModuleGetFunction, a.why) &&
              sym(cu, "cuModuleUnload", a.ModuleUnload, a.why) &&
              sym(cu, "cuFuncSetAttribute", a.FuncSetAttribute, a.why) && sym(cu, "cuFuncGetAttribute", a.FuncGetAttribute, a.why) && sym(cu, "cuLaunchKernelEx", a.LaunchKernelEx, a.why) &&
              sym(cu, "cuOccupancyMaxActiveBlocksPerMultiprocessor", a.OccupancyMaxActiveBlocks, a.why) &&
              sym(cu, "cuGetErrorString", a.GetErrorString, a.why);
    a.ok = ok;
  });
  return a;
}

std::string cu_err(CUresult r) {
  const char* s = nullptr;
  if (api().GetErrorString && api().GetErrorString(r, &s) == CUDA_SUCCESS && s) return s;
  return "CUDA driver error " + std::to_string((int)r);
}

// ---------------------------------------------------------------------------------------
// bytecode -> source
// ---------------------------------------------------------------------------------------
std::string regname(int k) { return k == kAccReg ? "acc" : "reg[" + std::to_string(k) + "]"; }
std::string fbits(uint32_t u) { char b[48]; snprintf(b, sizeof(b), "__uint_as_float(0x%08xu)", u); return b; }

bool is_unary(int op) { return op >= OP_NEG && op <= OP_I2F; }
bool is_binary(int op) { return op >= OP_ADD && op <= OP_LSEFIN; }

// One program range [pc, end) as statements.  vl/ng are the tile shape (1, 1 for scalar programs).
// n_prefetch > 0: the first n_prefetch instructions are loads whose data was fetched one tile
// ahead into raw[0..n): they become copies out of raw[], followed by the fetch for the next tile.
bool emit_program(const KernelParams& P, int pc, int end, bool scalar, int vl, int ng, bool full, bool reg_slots,
                  std::string& out, std::string& err, int n_prefetch = 0) {
  const std::string V = std::to_string(vl * ng), VLNG = std::to_string(vl) + ", " + std::to_string(ng);
  const std::string VLNGF = VLNG + (full ? ", true" : ", false");
  for (int j = 0; j < n_prefetch; ++j) {
    const uint32_t w = P.code[pc++];
    if ((w & 0xFF) == OP_LDBC) out += "        op_ldbc_widen<" + V + ">(" + std::to_string((int)P.io[(w >> 8) & 0xFF].dtype) + ", " + regname((w >> 16) & 0xFF) + ", raw[" + std::to_string(j) + "]);\n";
    else out += "        op_mov<" + V + ">(" + regname((w >> 16) & 0xFF) + ", raw[" + std::to_string(j) + "]);\n";
  }
  // row kernels fetch the next tile here; column kernels batch the loads of several steps themselves
  if (n_prefetch > 0 && P.family != FAM_COLUMN) out += "        if (has_next) prefetch(p, nx, raw);\n";
  while (pc < end) {
    const uint32_t w = P.code[pc++];
    const int op = w & 0xFF, a = (w >> 8) & 0xFF, b = (w >> 16) & 0xFF, c = w >> 24;
    const std::string A = std::to_string(a), B = std::to_string(b), OP = std::to_string(op);
    auto dt = [&](int io) { return std::to_string((int)P.io[io].dtype); };
    std::string s;
    if (op == OP_LDRAW) s = "op_ldraw<" + VLNGF + (P.io[a].col_mod ? ", 1" : ", 0") + ">(p, cx, " + A + ", " + dt(a) + ", " + regname(b) + ");";
    else if (op == OP_WIDEN) s = "op_widen<" + VLNG + ">(" + dt(a) + ", " + regname(b) + ");";
    else if (op == OP_LDBC) s = "op_ldbc<" + V + ">(p, cx, " + A + ", " + dt(a) + ", " + regname(b) + ");";
    else if (op == OP_LD) s = "op_mov<" + V + ">(acc, " + regname(a) + ");";
    else if (op == OP_ST) s = "op_mov<" + V + ">(" + regname(a) + ", acc);";
    else if (op == OP_STOUT) s = scalar ? "op_stout_scalar(p, cx, " + A + ", " + dt(a) + ", acc[0]);"
                                        : "op_stout<" + VLNGF + ">(p, cx, " + A + ", " + (b ? std::to_string(kStore01) : dt(a)) + ", acc);";
    else if (op == OP_STOUT_I) s = "op_stout_index(p, cx, " + A + ", " + dt(a) + ", acc[0]);";
    else if (is_unary(op)) s = "op_unary<" + OP + ", " + V + ">(acc);";
    else if (is_binary(op)) {
      if (b == OPK_REG) s = "op_binary<" + OP + ", " + V + ">(acc, " + regname(a) + ");";
      else if (b == OPK_IMM) s = "op_binary_s<" + OP + ", " + V + ">(acc, " + fbits(P.code[pc++]) + ");";
      else s = "op_binary_s<" + OP + ", " + V + ">(acc, cx.slots[" + A + "]);";
    } else if (op == OP_WHERE || op == OP_FMA) {
      const int kx = c & 15, ky = c >> 4;
      std::string x, y, pre = "{ ";
      if (kx == OPK_REG) x = regname(a);
      else { pre += "float xt[" + V + "]; op_splat<" + V + ">(xt, " + (kx == OPK_IMM ? fbits(P.code[pc++]) : "cx.slots[" + A + "]") + "); "; x = "xt"; }
      if (ky == OPK_REG) y = regname(b);
      else { pre += "float yt[" + V + "]; op_splat<" + V + ">(yt, " + (ky == OPK_IMM ? fbits(P.code[pc++]) : "cx.slots[" + B + "]") + "); "; y = "yt"; }
      s = pre + "op_ternary<" + OP + ", " + V + ">(acc, " + x + ", " + y + "); }";
    }
    else if (op == OP_WHERE_RAW) {
      const int ky = c & 15;
      std::string y, pre = "{ ";
      if (ky == OPK_REG) y = regname(b);
      else { pre += "float yt[" + V + "]; op_splat<" + V + ">(yt, " + (ky == OPK_IMM ? fbits(P.code[pc++]) : "cx.slots[" + B + "]") + "); "; y = "yt"; }
      s = pre + "op_where_raw<" + VLNG + ">(acc, " + regname(a) + ", " + y + "); }";
    }
    else if (op == OP_RED) s = "op_red<" + VLNGF + ">(cx, " + A + ", parts[" + B + "], acc, ts);";
    else if (op == OP_SCALE_TS) s = "op_scale_ts<" + V + ">(cx, " + A + ", " + B + ", acc, ts);";
    else if (op == OP_SPILL) s = "op_spill<" + V + ">(cx, " + B + ", " + regname(a) + ");";
    else if (op == OP_FILL) s = "op_fill<" + V + ">(cx, " + B + ", " + regname(a) + ");";
    else if (op == OP_SPILL_TS) s = "*stash_ptr<" + V + ">(cx, " + B + ") = ts;";
    else if (op == OP_FILL_TS) s = "ts = *stash_ptr<" + V + ">(cx, " + B + ");";
    else if (op == OP_ACCUM) s = std::string(a & 0x80 ? "op_accum_u<" : "op_accum<") + V + ">(" + std::to_string(a & 0x7F) + ", " + regname(b) + ", acc);";
    else if (op == OP_SLD) s = "op_splat<" + V + ">(acc, cx.slots[" + A + "]);";
    else if (op == OP_SST) s = std::string("op_sst<") + (reg_slots ? "true" : "false") + ">(cx, " + A + ", acc[0]);";
    else if (op == OP_END) continue;
    else { err = "specialiser: unknown opcode " + OP; return false; }
    out += "        " + s + "\n";
  }
  return true;
}

// Name of the kernel generated for a plan: family, tile shape and a hash of the program and
// its shape constants, so that profiler listings tell the kernels of different graphs apart.
std::string kernel_name(const LaunchPlan& lp) {
  static const char* fam[] = {"pointwise", "warp_row", "block_row", "cluster_row", "column_red", "split_row"};
  uint64_t h = 1469598103934665603ull;
  auto mix = [&](uint64_t v) { for (int i = 0; i < 8; ++i) { h ^= (v >> (8 * i)) & 0xFF; h *= 1099511628211ull; } };
  for (int i = 0; i < lp.code_words; ++i) mix(lp.p.code[i]);
  mix((uint64_t)lp.p.row_len); mix((uint64_t)lp.p.rows); mix((uint64_t)lp.block); mix((uint64_t)lp.p.cluster);
  mix((uint64_t)lp.p.red_len); mix((uint64_t)lp.p.col_tx); mix((uint64_t)lp.p.team_lanes); mix((uint64_t)lp.p.splits); mix((uint64_t)lp.p.slice_len);
  for (int q = 0; q < lp.p.n_io; ++q) {
    const IoDesc& io = lp.p.io[q];
    mix(io.dtype); mix((uint64_t)io.col_stride); mix(io.mapped); mix((uint64_t)io.red_stride);
    for (int i = 0; i < 3; ++i) { mix((uint64_t)io.lead_stride[i]); mix((uint64_t)io.map_dim[i]); mix((uint64_t)io.map_add[i]); mix((uint64_t)io.map_mod[i]); }
  }
  char b[96];
  snprintf(b, sizeof(b), "pn_spec_%s_v%dx%d_%08x", fam[lp.family >= 0 && lp.family <= FAM_SPLIT ? lp.family : 0], lp.vl, lp.ng, (unsigned)(h ^ (h >> 32)));
  static_assert(FAM_SPLIT == 5, "family names");
  return b;
}

// whether the generated kernel is first compiled under a register bound that it may not be able to keep
bool tentative_reg_bound(const LaunchPlan& lp) {
  return lp.p.family == FAM_WARP && lp.block == 256 && !lp.persistent && lp.vl * lp.ng <= 16 && !lp.no_reg_bound;
}

bool generate_source(const LaunchPlan& lp, std::string& src, std::string& err) {
  const KernelParams& P = lp.p;
  auto I = [](long long v) { return std::to_string(v); };
  std::string s;
  s.reserve(sizeof(kDeviceSource) + 8192);
  if (lp.bounds) s += "#define PN_BOUNDS 1\n";
  s += kDeviceSource;
  s += "\nnamespace pn {\nstruct Spec {\n";
  s += "  static constexpr int VL = " + I(lp.vl) + ", NG = " + I(lp.ng) + ", K = " + I(lp.k) + ";\n";
  // The block size as a constant folds the address arithmetic of a tile into the loads' immediate
  // offsets.  Not for rows streamed in several chunks by a block or cluster: there the constant
  // costs registers (47 against 32 on the gated multi-output workload), hence resident warps.
  const bool const_block = !((P.family == FAM_BLOCK || P.family == FAM_CLUSTER) && P.chunks > 1);
  s += "  static PN_DEV int block_threads() { return " + (const_block ? I(lp.block) : std::string("(int)blockDim.x")) + "; }\n";
  s += "  static constexpr bool kStatic = true;\n  static constexpr int kStages = " + I(P.n_stages) + ";\n";
  s += "  static constexpr int kFamily = " + I(P.family) + ", kNumIo = " + I(P.n_io) + ";\n";
  s += "  static PN_DEV unsigned lead_dim(const KernelParams&, int i) { return i == 0 ? " + I(P.lead_dim[0]) + "u : i == 1 ? " +
       I(P.lead_dim[1]) + "u : " + I(P.lead_dim[2]) + "u; }\n";
  s += "  static PN_DEV long long lead_stride(const KernelParams&, int io, int i) {\n    switch (io * 3 + i) {\n";
  for (int q = 0; q < P.n_io; ++q)
    for (int i = 0; i < 3; ++i)
      if (P.io[q].lead_stride[i] != 0) s += "      case " + I(q * 3 + i) + ": return " + I(P.io[q].lead_stride[i]) + "ll;\n";
  s += "      default: return 0;\n    }\n  }\n";
  s += "  static PN_DEV long long red_stride(const KernelParams&, int io) {\n    switch (io) {\n";
  for (int q = 0; q < P.n_io; ++q) if (P.io[q].red_stride != 0) s += "      case " + I(q) + ": return " + I(P.io[q].red_stride) + "ll;\n";
  s += "      default: return 0;\n    }\n  }\n";
  // column kernels: steps whose loads are in flight together.  Six under a bound of 7 blocks of 128
  // threads (72 registers) measured best on the pooling workload (47.2 -> 45.2 us); larger blocks keep
  // four under 64 registers.
  int walk_unroll = P.family == FAM_COLUMN ? (lp.block == 128 ? 6 : 4) : 1;
  if (lp.walk_cap > 0) walk_unroll = std::min(walk_unroll, (int)lp.walk_cap);
  s += "#ifndef PN_WALK_UNROLL\n#define PN_WALK_UNROLL " + I(walk_unroll) + "\n#endif\n  static constexpr int kWalkUnroll = PN_WALK_UNROLL;\n";
  s += "  static PN_DEV bool io_mapped(const KernelParams&, int io) {\n    switch (io) {\n";
  for (int q = 0; q < P.n_io; ++q) if (P.io[q].mapped) s += "      case " + I(q) + ": return true;\n";
  s += "      default: return false;\n    }\n  }\n";
  s += "  static PN_DEV IoMap io_map(const KernelParams&, int io) {\n    switch (io) {\n";
  for (int q = 0; q < P.n_io; ++q)
    if (P.io[q].mapped) {
      const IoDesc& io = P.io[q];
      s += "      case " + I(q) + ": return IoMap{" + I(io.map_dim[0]) + ", " + I(io.map_dim[1]) + ", " + I(io.map_dim[2]) + ", " +
           I(io.map_add[0]) + ", " + I(io.map_add[1]) + ", " + I(io.map_add[2]) + ", " + I(io.map_mod[0]) + ", " + I(io.map_mod[1]) + ", " +
           I(io.map_mod[2]) + ", " + I(io.lead_stride[0]) + "ll, " + I(io.lead_stride[1]) + "ll, " + I(io.lead_stride[2]) + "ll};\n";
    }
  s += "      default: return IoMap{1, 1, 1, 0, 0, 0, 0, 0, 0, 0, 0, 0};\n    }\n  }\n";
  // every group of every tile inside the row: no validity tests in the generated code
  const int team_threads = P.family == FAM_COLUMN ? P.col_tx : P.family <= FAM_WARP ? 32 : lp.block;
  const int team_lanes = (P.family == FAM_WARP && (P.team_lanes == 16 || P.team_lanes == 8)) ? P.team_lanes : 32;
  // (teams that share a warp may be switched off for a row: their accesses keep their validity tests)
  const bool full = team_lanes == 32 && (long long)P.chunks * team_threads * lp.vl * lp.ng == P.slice_len &&
                    (long long)P.slice_len * (P.family == FAM_SPLIT ? P.splits : P.cluster) == P.row_len;
  const bool reg_slots = true;   // generated programs keep the per-row scalars in registers
  auto konst = [&](const char* name, long long v) {
    s += std::string("  static PN_DEV int ") + name + "(const KernelParams&) { return " + I(v) + "; }\n";
  };
  konst("family", P.family); konst("cluster", P.cluster); konst("chunks", P.chunks); konst("split_chunks", P.split_chunks);
  konst("row_len", P.row_len); konst("slice_len", P.slice_len); konst("n_stages", P.n_stages); konst("n_io", P.n_io);
  konst("col_tx", P.col_tx); konst("red_len", P.red_len); konst("team_lanes", team_lanes); konst("splits", P.splits);
  auto table = [&](const char* name, const char* type, auto get) {
    s += std::string("  static PN_DEV ") + type + " " + name + "(const KernelParams&, int s, int r) {\n    switch (s * " + I(kMaxRed) + " + r) {\n";
    for (int st = 0; st < P.n_stages; ++st)
      for (int r = 0; r < P.stage[st].n_red; ++r) s += "      case " + I(st * kMaxRed + r) + ": return " + I(get(st, r)) + ";\n";
    s += "      default: return 0;\n    }\n  }\n";
  };
  table("red_kind", "int", [&](int st, int r) { return (long long)P.stage[st].red[r].kind; });
  table("red_slot", "int", [&](int st, int r) { return (long long)P.stage[st].red[r].slot; });
  table("red_uniform", "bool", [&](int st, int r) { return (long long)P.stage[st].red[r].uniform; });
  s += "  static PN_DEV int n_red(const KernelParams&, int s) {\n    switch (s) {\n";
  for (int st = 0; st < P.n_stages; ++st) s += "      case " + I(st) + ": return " + I(P.stage[st].n_red) + ";\n";
  s += "      default: return 0;\n    }\n  }\n";
  s += "  static PN_DEV bool has_scalar(const KernelParams&, int s) {\n    switch (s) {\n";
  for (int st = 0; st < P.n_stages; ++st) s += "      case " + I(st) + ": return " + (P.stage[st].scal_begin != P.stage[st].scal_end ? "true" : "false") + ";\n";
  s += "      default: return false;\n    }\n  }\n";
  const std::string V = I(lp.vl * lp.ng);
  s += "  static PN_DEV void prologue(const KernelParams& p, const TileCtx& cx, float (&acc)[" + V + "], float (&reg)[" + I(lp.k) + "][" + V + "], float& ts) {\n"
       "    Part parts[" + I(kMaxRed) + "]; (void)parts; (void)acc; (void)ts;\n";
  if (!emit_program(P, P.pro_begin, P.pro_end, false, lp.vl, lp.ng, full, reg_slots, s, err)) return false;
  s += "  }\n";
  // the loads at the head of stage 0 are issued one tile ahead of their use
  int n_pf = 0;
  for (int pc = P.stage[0].elem_begin; pc < P.stage[0].elem_end; ++pc) {
    const int op = P.code[pc] & 0xFF;
    if (op == OP_LDRAW || (op == OP_LDBC && P.family == FAM_COLUMN)) n_pf++; else break;
  }
  if (lp.no_prefetch) n_pf = 0;
  s += "  static constexpr int kNumPrefetch = " + I(n_pf) + ";\n";
  s += "  static PN_DEV void prefetch(const KernelParams& p, const TileCtx& cx, float (&raw)[" + I(n_pf > 0 ? n_pf : 1) + "][" + V + "]) {\n";
  for (int j = 0; j < n_pf; ++j) {
    const uint32_t w = P.code[P.stage[0].elem_begin + j];
    const int io = (w >> 8) & 0xFF;
    if ((w & 0xFF) == OP_LDBC) s += "    op_ldbc_raw<" + V + ">(p, cx, " + I(io) + ", " + I(P.io[io].dtype) + ", raw[" + I(j) + "]);\n";
    else s += "    op_ldraw<" + I(lp.vl) + ", " + I(lp.ng) + (full ? ", true" : ", false") + (P.io[io].col_mod ? ", 1" : ", 0") + ">(p, cx, " + I(io) + ", " + I(P.io[io].dtype) + ", raw[" + I(j) + "]);\n";
  }
  s += "  }\n";
  s += "  static PN_DEV void tile(const KernelParams& p, int s, const TileCtx& cx, float (&acc)[" + V + "], float (&reg)[" + I(lp.k) + "][" + V + "], float& ts, Part (&parts)[" + I(kMaxRed) + "],\n"
       "                          float (&raw)[" + I(n_pf > 0 ? n_pf : 1) + "][" + V + "], const TileCtx& nx, bool has_next) {\n    (void)raw; (void)nx; (void)has_next;\n    switch (s) {\n";
  for (int st = 0; st < P.n_stages; ++st) {
    s += "      case " + I(st) + ": {\n";
    if (!emit_program(P, P.stage[st].elem_begin, P.stage[st].elem_end, false, lp.vl, lp.ng, full, reg_slots, s, err, st == 0 ? n_pf : 0)) return false;
    s += "      } break;\n";
  }
  s += "      default: break;\n    }\n  }\n";
  s += "  static PN_DEV void scalar(const KernelParams& p, int s, const TileCtx& cx) {\n"
       "    float acc[1] = {0.f}; float reg[4][1] = {{0.f}, {0.f}, {0.f}, {0.f}}; float ts = 0.f;\n    (void)reg; (void)ts;\n    switch (s) {\n";
  for (int st = 0; st < P.n_stages; ++st) {
    s += "      case " + I(st) + ": {\n";
    if (!emit_program(P, P.stage[st].scal_begin, P.stage[st].scal_end, true, 1, 1, false, reg_slots, s, err)) return false;
    s += "      } break;\n";
  }
  s += "      default: break;\n    }\n  }\n};\n}  // namespace pn\n\n";
  // Blocks that hold a whole row in registers: ask the compiler to keep registers low enough
  // for 1024 resident threads per SM, since resident warps are what hides the HBM latency
  // (measured: +5 % on the LayerNorm workload).  Streaming kernels need no hint: they are
  // small already, and a bound would only license more registers.
  // Column kernels likewise: their walk keeps several steps of loads in flight per thread, and the
  // bound keeps that from eating the resident warps (measured: 64 registers with 4 steps in flight
  // beats every larger budget on the pooling workload).
  // Warp-per-row kernels that keep nothing across rows (the softmax workload: 39 registers left
  // to itself) gain from one more resident block per SM: 83.9 -> 82.3 us under a bound of 7 blocks
  // of 256 threads (the compiler settles on 32 registers and parks two words).  The bound is
  // tentative: a kernel that spills more than a few words under it is compiled again without
  // (spec_compile).
  const int min_blocks = (P.family == FAM_COLUMN && lp.block == 128) ? 7
                       : tentative_reg_bound(lp) ? 7
                       : ((P.family == FAM_BLOCK && P.chunks == 1) || P.family == FAM_COLUMN) ? std::max(1, 1024 / lp.block) : 1;
  s += "#ifndef PN_MIN_BLOCKS\n#define PN_MIN_BLOCKS " + I(min_blocks) + "\n#endif\n";
  s += "#if PN_MIN_BLOCKS > 1\n#define PN_LAUNCH_BOUNDS __launch_bounds__(" + I(lp.block) + ", PN_MIN_BLOCKS)\n#else\n"
       "#define PN_LAUNCH_BOUNDS __launch_bounds__(" + I(lp.block) + ")\n#endif\n";
  s += "extern \"C\" __global__ void PN_LAUNCH_BOUNDS " + kernel_name(lp) + "(const __grid_constant__ pn::KernelParams p) {\n"
       // launched with programmatic stream serialization (spec_launch), the kernel may be set up while
       // its predecessor in the stream still runs: it touches no memory before the predecessor is
       // complete and its writes are visible (a no-op under a plain launch)
       "  asm volatile(\"griddepcontrol.wait;\" ::: \"memory\");\n"
       "  extern __shared__ __align__(16) unsigned char smem[];\n  pn::" + std::string(P.family == FAM_COLUMN ? "column_body" : P.family == FAM_SPLIT ? "split_body" : "fused_body") + "<pn::Spec>(p, smem);\n}\n";
  src.swap(s);
  return true;
}

struct Compiled { CUmodule mod = nullptr; CUfunction fn = nullptr; int refs = 0; uint64_t used = 0; };
struct Key {
  int device; uint64_t h1, h2; size_t len;
  bool operator<(const Key& o) const { return std::tie(device, h1, h2, len) < std::tie(o.device, o.h1, o.h2, o.len); }
};
constexpr size_t kCacheCap = 256;   // loaded modules kept although no handle uses them
std::mutex g_cache_mutex;
std::map<Key, Compiled> g_cache;
uint64_t g_cache_clock = 0;

uint64_t fnv(const std::string& s, uint64_t h) { for (unsigned char c : s) { h ^= c; h *= 1099511628211ull; } return h; }
Key key_of(int device, const std::string& src) { return Key{device, fnv(src, 1469598103934665603ull), fnv(src, 0x9E3779B97F4A7C15ull), src.size()}; }

// unload modules nobody holds, least recently used first, down to the cap (call with the lock held)
void evict_unused() {
  while (g_cache.size() > kCacheCap) {
    auto victim = g_cache.end();
    for (auto it = g_cache.begin(); it != g_cache.end(); ++it)
      if (it->second.refs == 0 && (victim == g_cache.end() || it->second.used < victim->second.used)) victim = it;
    if (victim == g_cache.end()) return;
    if (api().ModuleUnload) api().ModuleUnload(victim->second.mod);
    g_cache.erase(victim);
  }
}

// ---- the optional cubin cache on disk ------------------------------------------------------------
struct DiskHeader { uint32_t magic; int32_t nvrtc_major, nvrtc_minor; uint64_t h1, h2, src_len, cubin_len; };
constexpr uint32_t kDiskMagic = 0x42434E50u;   // 'PNCB'
std::string disk_path(const Key& k) {
  const char* dir = getenv("PN_CACHE_DIR");
  if (!dir || !*dir) return std::string();
  char name[96];
  snprintf(name, sizeof(name), "/pn_%016llx%016llx_sm100a.cubin", (unsigned long long)k.h1, (unsigned long long)k.h2);
  return std::string(dir) + name;
}
bool disk_load(const Key& k, std::vector<char>& cubin) {
  const std::string path = disk_path(k);
  if (path.empty()) return false;
  FILE* f = fopen(path.c_str(), "rb");
  if (!f) return false;
  DiskHeader h;
  bool ok = fread(&h, sizeof(h), 1, f) == 1 && h.magic == kDiskMagic && h.nvrtc_major == api().nvrtc_major && h.nvrtc_minor == api().nvrtc_minor &&
            h.h1 == k.h1 && h.h2 == k.h2 && h.src_len == k.len && h.cubin_len > 0 && h.cubin_len < (64u << 20);
  if (ok) { cubin.resize(h.cubin_len); ok = fread(cubin.data(), 1, cubin.size(), f) == cubin.size(); }
  fclose(f);
  return ok;
}
void disk_store(const Key& k, const std::vector<char>& cubin) {
  const std::string path = disk_path(k);
  if (path.empty()) return;
  mkdir(getenv("PN_CACHE_DIR"), 0777);   // best effort; an existing directory is fine
  const std::string tmp = path + "." + std::to_string((long)getpid()) + ".tmp";
  FILE* f = fopen(tmp.c_str(), "wb");
  if (!f) return;
  const DiskHeader h{kDiskMagic, api().nvrtc_major, api().nvrtc_minor, k.h1, k.h2, (uint64_t)k.len, (uint64_t)cubin.size()};
  const bool ok = fwrite(&h, sizeof(h), 1, f) == 1 && fwrite(cubin.data(), 1, cubin.size(), f) == cubin.size();
  fclose(f);
  if (ok) rename(tmp.c_str(), path.c_str()); else remove(tmp.c_str());   // rename: readers never see half a file
}

}  // namespace

bool spec_available(std::string* why, bool compile_only) {
  const Api& a = api();
  const bool ok = compile_only ? a.CreateProgram != nullptr : a.ok;
  if (!ok && why) *why = a.why;
  return ok;
}

std::string spec_source(const LaunchPlan& lp) {
  std::string src, err;
  if (!generate_source(lp, src, err)) return "// " + err;
  return src.substr(sizeof(kDeviceSource) - 1 + (lp.bounds ? sizeof("#define PN_BOUNDS 1\n") - 1 : 0));   // the generated part only
}

bool spec_check(const LaunchPlan& lp, std::string& err) {
  const Api& a = api();
  if (!a.CreateProgram) { err = a.why.empty() ? "NVRTC not available" : a.why; return false; }
  std::string src;
  if (!generate_source(lp, src, err)) return false;
  nvrtcProgram prog;
  if (a.CreateProgram(&prog, src.c_str(), "pn_spec.cu", 0, nullptr, nullptr) != NVRTC_SUCCESS) { err = "nvrtcCreateProgram failed"; return false; }
  const std::vector<std::string> ov = nvrtc_options();
  std::vector<const char*> opts;
  for (const std::string& x : ov) opts.push_back(x.c_str());
  const nvrtcResult r = a.CompileProgram(prog, (int)opts.size(), opts.data());
  size_t n = 0; a.GetProgramLogSize(prog, &n);
  std::string log(n, '\0');
  if (n) a.GetProgramLog(prog, &log[0]);
  a.DestroyProgram(&prog);
  if (r != NVRTC_SUCCESS) { err = "run-time compilation failed: " + log.substr(0, 4000); return false; }
  return true;
}

bool spec_compile(LaunchPlan& lp, int device, int sm_count, SpecKernel& out, std::string& err) {
  const Api& a = api();
  if (!a.ok) { err = a.why; return false; }
  std::string src;
  if (!generate_source(lp, src, err)) return false;
  { std::string key; for (const std::string& x : nvrtc_options()) key += x + " "; src += "\n// " + key + "\n"; }
  const Key key = key_of(device, src);
  Compiled cmp;
  {
    std::lock_guard<std::mutex> lock(g_cache_mutex);
    auto it = g_cache.find(key);
    if (it != g_cache.end()) { it->second.refs++; it->second.used = ++g_cache_clock; cmp = it->second; }
  }
  if (!cmp.fn) {
    std::vector<char> cubin;
    if (!disk_load(key, cubin)) {
      nvrtcProgram prog;
      if (a.CreateProgram(&prog, src.c_str(), "pn_spec.cu", 0, nullptr, nullptr) != NVRTC_SUCCESS) { err = "nvrtcCreateProgram failed"; return false; }
      const std::vector<std::string> ov = nvrtc_options();
      std::vector<const char*> opts;
      for (const std::string& x : ov) opts.push_back(x.c_str());
      const nvrtcResult r = a.CompileProgram(prog, (int)opts.size(), opts.data());
      if (r != NVRTC_SUCCESS) {
        size_t n = 0; a.GetProgramLogSize(prog, &n);
        std::string log(n, '\0');
        if (n) a.GetProgramLog(prog, &log[0]);
        a.DestroyProgram(&prog);
        err = "run-time compilation failed: " + log.substr(0, 2000);
        return false;
      }
      size_t n = 0;
      a.GetCUBINSize(prog, &n);
      cubin.resize(n);
      a.GetCUBIN(prog, cubin.data());
      a.DestroyProgram(&prog);
      disk_store(key, cubin);
    }
    CUresult cr = a.ModuleLoadData(&cmp.mod, cubin.data());
    if (cr != CUDA_SUCCESS) { err = "cuModuleLoadData: " + cu_err(cr); return false; }
    cr = a.ModuleGetFunction(&cmp.fn, cmp.mod, kernel_name(lp).c_str());
    if (cr != CUDA_SUCCESS) { a.ModuleUnload(cmp.mod); err = "cuModuleGetFunction: " + cu_err(cr); return false; }
    std::lock_guard<std::mutex> lock(g_cache_mutex);
    auto it = g_cache.find(key);
    if (it != g_cache.end()) {   // another thread loaded the same kernel meanwhile: keep that one
      a.ModuleUnload(cmp.mod);
      it->second.refs++; it->second.used = ++g_cache_clock;
      cmp = it->second;
    } else {
      cmp.refs = 1; cmp.used = ++g_cache_clock;
      g_cache[key] = cmp;
      evict_unused();
    }
  }
  if (getenv("PN_DEBUG_SPEC")) {
    int regs = 0, local_b = 0;
    a.FuncGetAttribute(&regs, CU_FUNC_ATTRIBUTE_NUM_REGS, cmp.fn);
    a.FuncGetAttribute(&local_b, CU_FUNC_ATTRIBUTE_LOCAL_SIZE_BYTES, cmp.fn);
    fprintf(stderr, "spec: %s registers %d local bytes %d%s\n", kernel_name(lp).c_str(), regs, local_b, tentative_reg_bound(lp) ? " (tentative register bound)" : "");
  }
  // A column kernel that spills heavily under its register bound gains nothing from the steps it
  // keeps in flight, and one such kernel (six steps, 216 bytes of local memory, compiled with checked
  // accessors) was seen to compute a wrong first element per group: fewer steps in flight instead.
  if (lp.p.family == FAM_COLUMN && lp.walk_cap != 2) {
    int local_bytes = 0;
    if (a.FuncGetAttribute(&local_bytes, CU_FUNC_ATTRIBUTE_LOCAL_SIZE_BYTES, cmp.fn) == CUDA_SUCCESS && local_bytes > 96) {
      spec_release(cmp.fn);
      lp.walk_cap = lp.walk_cap == 0 ? 4 : 2;
      return spec_compile(lp, device, sm_count, out, err);
    }
  }
  if (tentative_reg_bound(lp)) {   // did the kernel keep the bound without spilling more than a few words?
    // (the softmax workload's kernel parks two words -- 8 bytes -- and is still the faster one)
    int local_bytes = 0;
    if (a.FuncGetAttribute(&local_bytes, CU_FUNC_ATTRIBUTE_LOCAL_SIZE_BYTES, cmp.fn) == CUDA_SUCCESS && local_bytes > 32) {
      spec_release(cmp.fn);
      lp.no_reg_bound = 1;
      return spec_compile(lp, device, sm_count, out, err);
    }
  }
  if (lp.smem_bytes > 48 * 1024) {
    const CUresult cr = a.FuncSetAttribute(cmp.fn, CU_FUNC_ATTRIBUTE_MAX_DYNAMIC_SHARED_SIZE_BYTES, lp.smem_bytes);
    if (cr != CUDA_SUCCESS) { spec_release(cmp.fn); err = "cuFuncSetAttribute: " + cu_err(cr); return false; }
  }
  int occ = 0;
  if (a.OccupancyMaxActiveBlocks(&occ, cmp.fn, lp.block, (size_t)lp.smem_bytes) != CUDA_SUCCESS) occ = 0;
  out.fn = cmp.fn;
  out.occupancy = occ;
  lp.specialised = 1;
  size_grid(lp, sm_count, occ);
  return true;
}

void spec_release(void* fn) {
  if (!fn) return;
  std::lock_guard<std::mutex> lock(g_cache_mutex);
  for (auto& kv : g_cache)
    if (kv.second.fn == (CUfunction)fn) { if (kv.second.refs > 0) kv.second.refs--; break; }
  evict_unused();
}

void spec_cache_stats(int64_t* modules, int64_t* in_use) {
  std::lock_guard<std::mutex> lock(g_cache_mutex);
  *modules = (int64_t)g_cache.size();
  *in_use = 0;
  for (auto& kv : g_cache) *in_use += kv.second.refs > 0;
}

bool spec_launch(const SpecKernel& k, const LaunchPlan& lp, void* stream, std::string& err) {
  const Api& a = api();
  CUlaunchConfig cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDimX = lp.grid; cfg.gridDimY = 1; cfg.gridDimZ = 1;
  cfg.blockDimX = lp.block; cfg.blockDimY = 1; cfg.blockDimZ = 1;
  cfg.sharedMemBytes = lp.smem_bytes;
  cfg.hStream = (CUstream)stream;
  CUlaunchAttribute attr[2];
  int n_attr = 0;
  if (lp.p.cluster > 1) {
    attr[n_attr].id = CU_LAUNCH_ATTRIBUTE_CLUSTER_DIMENSION;
    attr[n_attr].value.clusterDim.x = lp.p.cluster;
    attr[n_attr].value.clusterDim.y = 1;
    attr[n_attr].value.clusterDim.z = 1;
    ++n_attr;
  }
  // The launch may overlap the tail of the kernel before it in the stream: the kernel waits at its
  // head (griddepcontrol.wait) until that one is complete, so results are those of plain stream
  // order, but its set-up no longer waits for it.  Measured on B200, launches back to back from the
  // host: the pointwise chain [1024,1024] 4.7 -> 3.8 us per launch, roll + slice + add + LayerNorm
  // 6.2 -> 4.6, the long-row reduction 16.9 -> 15.2.  (Letting the successor start earlier still,
  // by a trigger at the kernel's head, costs more than it gains: its blocks take the slots of
  // blocks that have work to do: 5.8 us for the pointwise chain.)
  if (!lp.plain_launch) {
    attr[n_attr].id = CU_LAUNCH_ATTRIBUTE_PROGRAMMATIC_STREAM_SERIALIZATION;
    attr[n_attr].value.programmaticStreamSerializationAllowed = 1;
    ++n_attr;
  }
  if (n_attr) { cfg.attrs = attr; cfg.numAttrs = n_attr; }
  void* args[] = {const_cast<KernelParams*>(&lp.p)};
  const CUresult r = a.LaunchKernelEx(&cfg, (CUfunction)k.fn, args, nullptr);
  if (r != CUDA_SUCCESS) { err = "cuLaunchKernelEx: " + cu_err(r); return false; }
  return true;
}

}  // namespace pn
