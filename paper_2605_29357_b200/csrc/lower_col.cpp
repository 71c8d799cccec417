// lower_col.cpp -- host lowering of graphs whose reductions run over a leading dimension
// (the masked-mean-pooling shape of the paper's second case study, Section 4.4 and Appendix H:
// two sums over the sequence dimension of [B, S, D] tensors, then a clamped division on
// [B, D]).
//
// The iteration space is [O, R, C]: O the product of the dimensions before the reduced one,
// R the reduced dimension, C the product of those after it (contiguous in memory).  A thread
// owns a tile of columns and walks R; the tensors of the graph are either "pre" values, one
// per (o, r, c) and evaluated by the stage-0 tile program at every step, or "post" values, one
// per (o, c): the reduction results and everything computed from them, evaluated once by the
// stage-1 tile program.  Reductions are OP_ACCUM instructions into tile registers that persist
// over the walk.  Post values never feed pre values (that would need a second pass over R).
#include <string>
#include <vector>

#include "../../include/pn.h"
#include "graph.h"
#include "lower_common.h"

namespace pn {

int instance_occupancy(int vl, int ng, int k, int block, int smem_bytes);  // kernels.cu

using namespace lowering;

namespace {

enum Space : char { SP_NONE = 0, SP_PRE = 1, SP_POST = 2 };

// dims of a tensor right-aligned into `rank` positions (missing leading ones are 1)
bool right_align(const Tensor& t, int rank, int64_t* out) {
  if (t.rank > rank) return false;
  for (int i = 0; i < rank; ++i) out[i] = 1;
  for (int i = 0; i < t.rank; ++i) out[rank - t.rank + i] = t.dims[i];
  return true;
}

// One group of dimensions of a tensor against the same group of the full shape: every
// dimension full (1), every dimension 1 where the full one is not (0), or a mix (-1).
int group_state(const int64_t* d, const int64_t* full, int lo, int hi) {
  bool all_full = true, all_one = true;
  for (int i = lo; i < hi; ++i) {
    if (full[i] == 1) continue;
    if (d[i] != full[i]) all_full = false;
    if (d[i] != 1) all_one = false;
    if (d[i] != 1 && d[i] != full[i]) return -1;
  }
  if (all_full) return 1;
  return all_one ? 0 : -1;
}

}  // namespace

int lower_column_graph(const Graph& g, unsigned flags, const DeviceModel& dev, LaunchPlan& lp, std::string& err) {
  const int nt = (int)g.tensors.size();
  for (int o : g.outputs)
    if (g.tensors[o].embed_parent >= 0) { err = "a result of a reduction over a leading dimension cannot be stored as an operand of a cat in the same kernel"; return PN_ERR_UNSUPPORTED_OP; }
  // ---- (1) the reduced dimension and the two spaces ----------------------------------------
  int rs = -1, dr = -1;   // rank of the reduced tensors, reduced dimension
  for (size_t ni = 0; ni < g.nodes.size(); ++ni) {
    const Node& n = g.nodes[ni];
    const std::string where = "node " + std::to_string(ni) + ": ";
    if (is_reduction(n.op) || is_composite(n.op) || is_index_op(n.op)) {
      err = where + "last-dimension reductions and index operators do not mix with reductions over a leading dimension";
      return PN_ERR_UNSUPPORTED_OP;
    }
    if (!is_dim_reduction(n.op)) continue;
    const Tensor& X = g.tensors[n.in[0]];
    if (n.in[0] >= (uint32_t)nt) { err = where + "reduction of a constant"; return PN_ERR_UNSUPPORTED_OP; }
    if (n.attr[0] < 0 || n.attr[0] >= X.rank) { err = where + "reduced dimension outside the tensor"; return PN_ERR_SHAPE; }
    if (n.attr[0] == X.rank - 1) { err = where + "the last dimension is reduced by sum / mean / amax / amin, not by their _dim forms"; return PN_ERR_UNSUPPORTED_OP; }
    if (rs < 0) { rs = X.rank; dr = (int)n.attr[0]; }
    else if (rs != X.rank || dr != n.attr[0]) { err = where + "all reductions of a graph must run over the same dimension of tensors of one rank"; return PN_ERR_UNSUPPORTED_OP; }
  }
  if (rs < 0) { err = "internal: no reduction over a leading dimension"; return PN_ERR_UNSUPPORTED_OP; }

  std::vector<char> space(nt, SP_NONE);
  std::vector<int> n_consumers(nt, 0);
  for (size_t ni = 0; ni < g.nodes.size(); ++ni) {
    const Node& n = g.nodes[ni];
    const std::string where = "node " + std::to_string(ni) + ": ";
    bool any_post = false, any_tensor = false;
    for (int k = 0; k < n.n_in; ++k) {
      if (n.in[k] >= (uint32_t)nt) continue;
      any_tensor = true;
      n_consumers[n.in[k]]++;
      any_post = any_post || space[n.in[k]] == SP_POST;
    }
    if (!any_tensor) { err = where + "a node with only constant operands is not lowered"; return PN_ERR_UNSUPPORTED_OP; }
    if (is_dim_reduction(n.op)) {
      if (any_post) { err = where + "a reduction of a reduced value needs a second pass and is not lowered"; return PN_ERR_UNSUPPORTED_OP; }
      if (space[n.in[0]] == SP_NONE) space[n.in[0]] = SP_PRE;
      space[n.out[0]] = SP_POST;
      continue;
    }
    const char sp = any_post ? SP_POST : SP_PRE;
    for (int k = 0; k < n.n_in; ++k) {
      if (n.in[k] >= (uint32_t)nt) continue;
      char& s = space[n.in[k]];
      if (s == SP_NONE) s = sp;
      else if (s != sp) {
        err = where + (sp == SP_POST ? "a value with the reduced dimension meets a reduced value: that needs a second pass and is not lowered"
                                     : "a graph input is used both before and after the reduction");
        return PN_ERR_UNSUPPORTED_OP;
      }
    }
    for (int k = 0; k < n.n_out; ++k) space[n.out[k]] = sp;
  }

  // full shapes: pre space in rs dimensions, post space in rs - 1
  int64_t Fpre[4] = {1, 1, 1, 1}, Fpost[4] = {1, 1, 1, 1};
  std::vector<std::vector<int64_t>> dims(nt, std::vector<int64_t>(4, 1));
  for (int t = 0; t < nt; ++t) {
    const Tensor& T = g.tensors[t];
    const std::string where = "tensor " + std::to_string(t) + ": ";
    if (space[t] == SP_NONE) continue;   // a graph input nothing reads (or only nodes that reach no output): takes no part
    int64_t d[4];
    if (space[t] == SP_PRE) {
      if (!right_align(T, rs, d)) { err = where + "rank above that of the reduced tensors"; return PN_ERR_SHAPE; }
      for (int i = 0; i < rs; ++i) {
        if (Fpre[i] == 1) Fpre[i] = d[i];
        else if (d[i] != 1 && d[i] != Fpre[i]) { err = where + "does not broadcast into the iteration space"; return PN_ERR_SHAPE; }
      }
    } else {
      Tensor U = T;
      if (T.rank == rs) {   // the reduced dimension kept as 1
        if (T.dims[dr] != 1) { err = where + "a reduced value keeps the reduced dimension as 1 or drops it"; return PN_ERR_SHAPE; }
        U.rank = rs - 1;
        for (int i = 0, j = 0; i < rs; ++i) if (i != dr) U.dims[j++] = T.dims[i];
      }
      if (!right_align(U, rs - 1, d)) { err = where + "rank above that of the reduced values"; return PN_ERR_SHAPE; }
      for (int i = 0; i < rs - 1; ++i) {
        if (Fpost[i] == 1) Fpost[i] = d[i];
        else if (d[i] != 1 && d[i] != Fpost[i]) { err = where + "does not broadcast into the reduced shape"; return PN_ERR_SHAPE; }
      }
    }
    for (int i = 0; i < 4; ++i) dims[t][i] = i < rs ? d[i] : 1;
  }
  for (int i = 0, j = 0; i < rs; ++i) {
    if (i == dr) continue;
    if (Fpost[j] != 1 && Fpost[j] != Fpre[i]) { err = "the reduced values do not have the shape of the reduced tensors without the reduced dimension"; return PN_ERR_SHAPE; }
    ++j;
  }
  const int64_t R = Fpre[dr];
  int64_t O = 1, C = 1;
  for (int i = 0; i < dr; ++i) O *= Fpre[i];
  for (int i = dr + 1; i < rs; ++i) C *= Fpre[i];
  if (R <= 0 || C <= 0 || O <= 0) { err = "an empty iteration space"; return PN_ERR_SHAPE; }
  if (C >= (int64_t(1) << 30) || R >= (int64_t(1) << 30) || O >= (int64_t(1) << 31)) { err = "iteration space too large"; return PN_ERR_TOO_LARGE; }
  int64_t Fdrop[4] = {1, 1, 1, 1};   // the full post shape: the pre shape without the reduced dimension
  for (int i = 0, j = 0; i < rs; ++i) if (i != dr) Fdrop[j++] = Fpre[i];

  // per-node shape rules
  for (size_t ni = 0; ni < g.nodes.size(); ++ni) {
    const Node& n = g.nodes[ni];
    const std::string where = "node " + std::to_string(ni) + ": ";
    if (is_dim_reduction(n.op)) {
      const int x = (int)n.in[0], y = (int)n.out[0];
      if (dims[x][dr] != R) { err = where + "the reduced dimension of the operand must have its full length"; return PN_ERR_SHAPE; }
      for (int i = 0, j = 0; i < rs; ++i) {
        if (i == dr) continue;
        if (dims[y][j] != dims[x][i]) { err = where + "result must have the operand's shape with the reduced dimension dropped or 1"; return PN_ERR_SHAPE; }
        ++j;
      }
    } else {
      const int rk = space[n.out[0]] == SP_PRE ? rs : rs - 1;
      int64_t b[4] = {1, 1, 1, 1};
      for (int k = 0; k < n.n_in; ++k) {
        if (n.in[k] >= (uint32_t)nt) continue;
        for (int i = 0; i < rk; ++i) {
          const int64_t v = dims[n.in[k]][i];
          if (b[i] == 1) b[i] = v;
          else if (v != 1 && v != b[i]) { err = where + "operands do not broadcast"; return PN_ERR_SHAPE; }
        }
      }
      for (int i = 0; i < rk; ++i)
        if (b[i] != dims[n.out[0]][i]) { err = where + "declared output shape is not the broadcast of the operands"; return PN_ERR_SHAPE; }
    }
  }

  // ---- io table: graph inputs and outputs as [O, R, C] / [O, C] with strides ----------------
  memset(&lp, 0, sizeof(lp));
  KernelParams& P = lp.p;
  std::vector<int> read_inputs;   // graph inputs that the computation reads
  for (int t : g.inputs) if (space[t] != SP_NONE) read_inputs.push_back(t);
  const int n_io = (int)(read_inputs.size() + g.outputs.size());
  if (n_io > kMaxIo) { err = "more graph inputs + outputs than one kernel takes (" + std::to_string(kMaxIo) + ")"; return PN_ERR_TOO_LARGE; }
  P.n_io = n_io;
  std::vector<int> io_of_tensor(nt, -1);
  std::vector<char> io_streamed(n_io, 0);
  {
    int idx = 0;
    for (int pass = 0; pass < 2; ++pass)
      for (int t : pass == 0 ? read_inputs : g.outputs) {
        IoDesc& io = P.io[idx];
        const std::string where = "tensor " + std::to_string(t) + ": ";
        io.dtype = g.tensors[t].dtype;
        const int64_t* d = dims[t].data();
        int before, after;
        int64_t own_r = 1;
        if (space[t] == SP_PRE) {
          before = group_state(d, Fpre, 0, dr); after = group_state(d, Fpre, dr + 1, rs);
          own_r = d[dr];
        } else {
          before = group_state(d, Fdrop, 0, dr); after = group_state(d, Fdrop, dr, rs - 1);
        }
        if (before < 0 || after < 0) { err = where + "broadcasts over part of the dimensions before or after the reduced one: not lowered"; return PN_ERR_UNSUPPORTED_OP; }
        const int64_t own_c = after ? C : 1;
        io.col_stride = (after || C == 1) ? 1 : 0;
        io.red_stride = (own_r != 1 || R == 1) ? own_c : 0;
        io.lead_stride[0] = io.lead_stride[1] = 0;
        io.lead_stride[2] = (before && O != 1) ? own_c * own_r : 0;
        io_streamed[idx] = space[t] == SP_PRE && before && after && own_r == R;
        if (pass == 1) {
          const bool full = before && after && (space[t] == SP_POST || own_r == R);
          if (!full) { err = "output " + where + "must have the full shape of its space"; return PN_ERR_UNSUPPORTED_OP; }
        }
        lp.io_tensor[idx] = t; lp.io_is_output[idx] = pass;
        io_of_tensor[t] = idx;
        ++idx;
      }
  }
  P.lead_dim[0] = P.lead_dim[1] = 1; P.lead_dim[2] = (uint32_t)O;
  P.rows = O; P.row_len = (int32_t)C; P.red_len = (int32_t)R;

  // ---- (2) micro-operations -----------------------------------------------------------------
  Expander ex;
  std::vector<int> tval(nt, -1);
  for (int t : read_inputs) {
    const int v = ex.new_val(VK_E, space[t] == SP_POST ? 1 : 0);
    const int q = io_of_tensor[t];
    ex.vals[v].io = q;
    ex.vals[v].bcast = P.io[q].col_stride == 0;
    ex.vals[v].uniform = P.io[q].col_stride == 0 && C != 1;
    ex.vals[v].streamed = io_streamed[q];
    ex.vals[v].integral = !dtype_is_float(g.tensors[t].dtype);
    ex.vals[v].mask8 = g.tensors[t].dtype == kI8 || g.tensors[t].dtype == kBool;
    tval[t] = v;
  }
  std::vector<RedDesc> reds;
  std::vector<int> red_val;
  std::map<std::pair<int, int>, int> red_cache;   // (kind, value) -> accumulator
  for (size_t ni = 0; ni < g.nodes.size(); ++ni) {
    const Node& n = g.nodes[ni];
    const std::string where = "node " + std::to_string(ni) + ": ";
    int in[4] = {-1, -1, -1, -1};
    for (int k = 0; k < n.n_in; ++k) {
      if (n.in[k] == kImm0) in[k] = ex.imm_val(n.imm[0]);
      else if (n.in[k] == kImm1) in[k] = ex.imm_val(n.imm[1]);
      else in[k] = tval[n.in[k]];
    }
    int res[3] = {-1, -1, -1};
    if (is_dim_reduction(n.op)) {
      const int kind = (n.op == N_AMAX_DIM) ? RED_MAX : (n.op == N_AMIN_DIM) ? RED_MIN : RED_SUM;
      const auto key = std::make_pair(kind, in[0]);
      int a;
      if (red_cache.count(key)) a = red_cache[key];
      else {
        if ((int)reds.size() >= kMaxRed) { err = where + "more reductions than the kernel takes"; return PN_ERR_TOO_LARGE; }
        a = (int)reds.size();
        const bool uni = ex.vals[in[0]].uniform;
        RedDesc rd; rd.kind = (uint8_t)kind; rd.slot = (uint8_t)a; rd.uniform = uni ? 1 : 0;   // accumulator a is tile register a
        reds.push_back(rd);
        const int v = ex.new_val(VK_E, 1);
        ex.vals[v].pinned = true;
        ex.vals[v].integral = ex.vals[in[0]].integral;
        red_val.push_back(v);
        ex.vals[v].uniform = uni;
        ex.add_op(OP_ACCUM, 0, false, {in[0]}, -1, kind | (uni ? 0x80 : 0), a);
        red_cache[key] = a;
      }
      res[0] = red_val[a];
      if (n.op == N_MEAN_DIM) res[0] = ex.pointwise(OP_DIV, {res[0], ex.imm_val((double)R)}, false);
    } else {
      const int pw = ex.expand_pointwise(g, n, in, res, err, where);
      if (pw < 0) return pw;
      if (pw == 0) { err = where + "opcode not lowered"; return PN_ERR_UNSUPPORTED_OP; }
    }
    const int fin = ex.finish_node(g, n, res, n_consumers, io_of_tensor, tval, 2, err, where);
    if (fin != PN_OK) return fin;
  }
  std::vector<Val>& vals = ex.vals;
  for (const MOp& m : ex.ops) for (int i = 0; i < m.nin; ++i) vals[m.in[i]].uses++;
  for (const MOp& m : ex.ops)
    for (int i = 0; i < m.nin; ++i)
      if (m.stage == 0 && vals[m.in[i]].stage > 0) { err = "internal: a reduced value is read before the reduction"; return PN_ERR_UNSUPPORTED_OP; }

  // ---- (3) tile shape -------------------------------------------------------------------------
  int min_esize = 8;
  bool vec8 = true, vec4 = true;
  for (int q = 0; q < n_io; ++q) {
    const IoDesc& io = P.io[q];
    if (io.col_stride == 0) continue;
    if (io_streamed[q]) min_esize = std::min(min_esize, dtype_bytes(io.dtype));
    for (int vl : {8, 4}) {
      const bool ok = C % vl == 0 && io.lead_stride[2] % vl == 0 && io.red_stride % vl == 0;
      if (vl == 8) vec8 = vec8 && ok; else vec4 = vec4 && ok;
    }
  }
  int VL = (min_esize <= 2 && vec8) ? 8 : (vec4 ? 4 : 1);
  // groups of 8 elements of a 4-byte operand read at every step are two half-used 128-bit accesses
  // (see lower.cpp): such graphs take groups of 4
  if (VL == 8 && vec4)
    for (int q = 0; q < n_io; ++q)
      if (P.io[q].col_stride != 0 && io_streamed[q] && dtype_bytes(P.io[q].dtype) >= 4) VL = 4;
  if (flags & PN_FLAG_FORCE_SCALAR) VL = 1;
  const bool spec = dev.specialise;
  // (NG, K): the interpreter's instances with four tile registers; generated kernels take one
  // 16-byte group per operand and step (the walk over R is what keeps loads in flight)
  int NG = VL == 8 ? 1 : (VL == 4 ? 2 : 8), K = 4;
  if (spec) { NG = VL == 1 ? 4 : 1; K = kSpecRegs; }
  const int t_ng = (flags >> 24) & 31;
  if (spec && t_ng && (t_ng & (t_ng - 1)) == 0 && VL * t_ng <= 32 && VL * t_ng >= 2) NG = t_ng;   // (an i64 element in flight takes two tile slots)
  if ((int)reds.size() > K - 2) { err = "more reductions than the kernel has tile registers for"; return PN_ERR_TOO_LARGE; }
  // generated kernels: 128 threads (4 walkers of a warp-wide column tile each), measured best on
  // B200 with the register bound that keeps 1024 threads resident per SM
  int block = spec ? 128 : 256;
  const int t_block = ((flags >> 20) & 15) ? 1 << ((flags >> 20) & 15) : 0;
  if (t_block >= 32 && t_block <= (spec ? 1024 : 256)) block = t_block;
  // threads along the columns: enough to cover C, at most a warp (a warp then reads 32 x 16
  // contiguous bytes per step); the rest of the block splits R
  int TX = 1;
  while (TX < 32 && (int64_t)TX * VL * NG < C) TX *= 2;
  // Few (row, column tile) items for the size of the GPU: more walkers per item first (blocks of up
  // to 512 threads, while every walker keeps a batch of steps), then narrower column tiles (down to
  // 8 threads: 128 contiguous bytes per step and item), then slices of the reduced dimension itself
  // -- a block per (item, slice), combined by the block that arrives last; partials and arrival
  // counters live in a workspace of the handle, so not for handles that may not have one -- and only
  // then blocks of 1024.  This is what keeps a small batch of long sequences, or a few columns under
  // a very long reduced dimension, from running on a handful of SMs.  Measured on B200 (bf16 sums,
  // L2-cold): [1,1M,8] 43.8 -> 26.6 us, [4,16384,64] 12.3 -> 10.3, [1,8192,4096] 24.1 -> 16.4;
  // slices where blocks of 512 already fill the GPU only cost ([64,512,1024] 14.4 -> 18.0 with two).
  // PN_TUNE_CLUSTER(n) asks for n slices, PN_FLAG_FORCE_SPLIT for at least two.
  const bool may_slice = !(flags & PN_FLAG_STATIC_SCRATCH);
  const int t_slices = may_slice ? (int)((flags >> 16) & 15) : 0;   // PN_TUNE_CLUSTER on a column kernel
  int splits = 1;
  if (spec && !t_block && t_slices <= 1) {
    const int64_t want = (int64_t)dev.sm_count * 512;   // threads for a quarter of the resident capacity
    auto threads = [&](int tx, int blk) { return O * ((C + (int64_t)tx * VL * NG - 1) / ((int64_t)tx * VL * NG)) * blk; };
    auto steps_ok = [&](int tx, int blk) { return R / (blk / tx) >= 8; };
    while (threads(TX, block) < want && block < 512 && steps_ok(TX, block * 2)) block *= 2;
    while (threads(TX, block) < want && TX > 8 && (int64_t)(TX / 2) * VL * NG * 2 <= C * 2 && steps_ok(TX / 2, block)) TX /= 2;
    if (may_slice && threads(TX, block) < want) {
      const int64_t per_walker = R / (block / TX);      // steps a walker takes over the whole of R
      int64_t s = 1;
      while (s * threads(TX, block) < want) s *= 2;     // (a power of two: [1,8192,4096] 18.5 us in 3 slices, 16.4 in 4)
      s = std::min<int64_t>(std::min<int64_t>(s, per_walker / 8), 64);
      if (s >= 2) splits = (int)s;
    }
    while (splits == 1 && threads(TX, block) < want && block < 1024 && steps_ok(TX, block * 2)) block *= 2;
  }
  const int64_t ctile = (int64_t)TX * VL * NG;
  const int64_t n_ctiles = (C + ctile - 1) / ctile;
  if (may_slice) {
    const int64_t per_walker = std::max<int64_t>(1, R / (block / TX));
    if (t_slices > 1) splits = (int)std::min<int64_t>(t_slices, per_walker);
    if ((flags & PN_FLAG_FORCE_SPLIT) && splits < 2 && per_walker >= 2) splits = 2;
    if (splits < 2 || O * n_ctiles * splits > (int64_t(1) << 30)) splits = 1;
  } else splits = 1;

  // ---- (4) code generation ----------------------------------------------------------------------
  std::vector<uint32_t> code;
  std::map<int, int> stash_of;
  int n_stash = 0;
  Gen ge(code, vals, false, K, false, stash_of, n_stash);
  for (size_t a = 0; a < reds.size(); ++a) { ge.regv[a] = red_val[a]; ge.regraw[a] = 0; }
  StageDesc stages[kMaxStages];
  memset(stages, 0, sizeof(stages));
  for (int s = 0; s < 2; ++s) {
    stages[s].elem_begin = (uint16_t)code.size();
    ge.hoist_loads(ex.ops, s, true);
    for (const MOp& m : ex.ops) {
      if (m.stage != s) continue;
      if (m.scalar) { err = "internal: scalar operation in a column kernel"; return PN_ERR_UNSUPPORTED_OP; }
      if (!ge.gen(m)) { err = ge.err; return PN_ERR_TOO_LARGE; }
    }
    ge.accv = -1;   // nothing but the accumulators crosses from the walk to the epilogue
    for (int k = (int)reds.size(); k < K; ++k) { ge.regv[k] = -1; ge.regraw[k] = 0; }
    stages[s].elem_end = stages[s].scal_begin = stages[s].scal_end = (uint16_t)code.size();
  }
  stages[0].n_red = (uint8_t)reds.size();
  for (size_t r = 0; r < reds.size(); ++r) stages[0].red[r] = reds[r];
  if ((int)code.size() > kMaxCode) { err = "bytecode longer than the kernel takes"; return PN_ERR_TOO_LARGE; }

  // ---- (5) shared memory and grid -----------------------------------------------------------------
  int off = 0;
  auto take = [&](int bytes) { const int o = off; off += (bytes + 15) / 16 * 16; return o; };
  P.sm_rowoff = take(0); P.sm_slots = take(0); P.sm_wpart = take(0); P.sm_ctapart = take(0); P.sm_stash = take(0);
  P.sm_part = take((int)reds.size() * VL * NG * block * 4);   // accumulators of every thread, for the combine over R
  if (off > dev.max_smem_per_block) { err = "accumulators do not fit in shared memory"; return PN_ERR_TOO_LARGE; }
  P.n_stages = 2;
  memcpy(P.stage, stages, sizeof(stages));
  memcpy(P.code, code.data(), code.size() * 4);
  P.slice_len = (int32_t)C;
  P.chunks = (int32_t)n_ctiles;
  P.split_chunks = 0;
  P.cluster = 1;
  P.col_tx = TX;
  P.splits = splits > 1 ? splits : 0;
  P.family = FAM_COLUMN;
  lp.family = FAM_COLUMN; lp.vl = VL; lp.ng = NG; lp.k = K;
  lp.block = block; lp.smem_bytes = off; lp.code_words = (int)code.size();
  lp.items = O * n_ctiles * (splits > 1 ? splits : 1);
  lp.teams_per_cta = 1;
  // generated kernels issue the loads of several steps of the walk before the arithmetic of the first
  lp.specialised = 0; lp.persistent = 0; lp.grid_waves = tune_waves(flags); lp.no_prefetch = (flags & PN_FLAG_NO_HOIST) ? 1 : 0;
  const int occ = (dev.have_device && !spec) ? instance_occupancy(VL, NG, K, block, off) : 0;
  size_grid(lp, dev.sm_count, occ);
  return PN_OK;
}

}  // namespace pn
