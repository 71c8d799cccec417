// lower.cpp -- host lowering of a validated graph into one fused launch.
//
// Steps: (1) shape analysis: the iteration space [rows, N] (N = last dim), which tensors
// are tile values (one element per column) and which are per-row scalars (results of
// last-dim reductions); (2) expansion of every node into tile / reduction / scalar
// micro-operations, split into stages at reduction boundaries; (3) choice of the kernel
// family and tile shape from (rows, N, dtypes, SM count) -- the per-shape cost model whose
// absence (tile shapes fixed whatever the tensor shape) the paper counts among the failure
// modes of generated passes, Section 4.4; (4) accumulator-machine code generation with register allocation;
// (5) shared-memory layout and grid.  Graphs whose reductions run over a leading dimension are
// lowered by lower_col.cpp (the column-reduce family); roll / slice / view chains on graph inputs
// become the addressing of the kernel's loads here.
#include <math.h>
#include <string.h>

#include <algorithm>
#include <map>
#include <string>
#include <vector>

#include "../../include/pn.h"
#include "graph.h"
#include "lower_common.h"

namespace pn {

int instance_occupancy(int vl, int ng, int k, int block, int smem_bytes);  // kernels.cu

using namespace lowering;


// Grid of a planned launch from the SM count and the resident CTAs per SM of its kernel:
// whole work if it fits in a few waves, else a grid-stride loop over a bounded grid.
void size_grid(LaunchPlan& lp, int sms, int occ) {
  if (occ <= 0) occ = std::max(1, 512 / lp.block);
  const int64_t resident = (int64_t)sms * occ;
  const int cluster = std::max(lp.p.cluster, 1);
  int64_t waves = lp.persistent ? 1 : 8;   // work hoisted out of the row loop wants long-lived CTAs
  if (lp.grid_waves > 0) waves = lp.grid_waves;
  if (lp.grid_waves < 0) waves = int64_t(1) << 40;
  int64_t grid;
  if (lp.family == FAM_SPLIT) { lp.grid = (int)lp.items; return; }   // one block per slice of a row, always
  if (lp.family <= FAM_WARP) grid = std::min<int64_t>((lp.items + lp.teams_per_cta - 1) / lp.teams_per_cta, resident * waves);
  else if (lp.family == FAM_BLOCK) grid = std::min<int64_t>(lp.items, resident * waves);
  else grid = std::min<int64_t>(lp.items, std::max<int64_t>(1, resident * waves / cluster)) * cluster;
  lp.grid = (int)std::max<int64_t>(grid, cluster);
}

// PN_TUNE_WAVES: 0 default, 7 one CTA per item, n: 2^(n-1) waves
int tune_waves(unsigned flags) { const int w = (flags >> 29) & 7; return w == 0 ? 0 : (w == 7 ? -1 : 1 << (w - 1)); }

namespace {

struct Config { int family, vl, ng, k, block, cluster, chunks, slice_len; bool multichunk; int lanes; int splits; };

}  // namespace

// ---------------------------------------------------------------------------------------
int lower_graph(const Graph& g, unsigned flags, const DeviceModel& dev, LaunchPlan& lp, std::string& err) {
  for (const Node& n : g.nodes)   // (a cat of several operands has been rewritten into embedded parts before any lowering)
    if (n.op == N_CAT && n.n_in != 1) { err = "internal: a cat of several operands reached the lowering"; return PN_ERR_UNSUPPORTED_OP; }
  for (const Node& n : g.nodes) if (is_dim_reduction(n.op)) return lower_column_graph(g, flags, dev, lp, err);
  const int nt = (int)g.tensors.size();
  std::vector<char> is_s(nt, 0);
  std::vector<int> n_consumers(nt, 0);
  bool has_red = false;

  // ---- (1) shapes ---------------------------------------------------------------------
  for (const Node& n : g.nodes) {
    if (is_reduction(n.op) || is_composite(n.op)) has_red = true;
    for (int k = 0; k < n.n_in; ++k) if (n.in[k] < (uint32_t)nt) n_consumers[n.in[k]]++;
  }
  // ---- index operators: roll / slice / view chains that start at a graph input are folded into
  // the addressing of that input (no data is moved) --------------------------------------
  struct IdxMap {
    int root = -1;                       // the graph input the chain starts at
    int64_t ext[3] = {1, 1, 1}, add[3] = {0, 0, 0}, mod[3] = {0, 0, 0}, stride[3] = {0, 0, 0};
    bool sliced[3] = {false, false, false};
    int64_t col_add = 0, col_mod = 0;    // the last dimension: column c of the view is column (c + col_add) mod col_mod of the root
    bool col_sliced = false;
    bool plain = true;                   // still the dense tensor itself (views only)
    bool frozen = false;                 // regrouped by a view after rolls / slices: no further index ops
  };
  std::vector<IdxMap> imap(nt);
  // which nodes only re-index: roll / slice / view, and contiguous where it follows such a chain (or a
  // graph input): it is then a view of the same shape; on a computed value it is a pointwise identity
  std::vector<char> idx_like(g.nodes.size(), 0);
  {
    std::vector<char> chained(nt, 0);
    for (int t : g.inputs) chained[t] = 1;
    for (size_t ni = 0; ni < g.nodes.size(); ++ni) {
      const Node& n = g.nodes[ni];
      const bool src_chained = n.n_in >= 1 && n.in[0] < (uint32_t)nt && chained[n.in[0]];
      idx_like[ni] = is_index_op(n.op) || (n.op == N_CONTIGUOUS && src_chained);
      if (idx_like[ni] && src_chained) chained[n.out[0]] = 1;
    }
  }
  auto plain_map = [&](int root, const Tensor& T) {
    IdxMap m; m.root = root;
    const Shape4 s = align4(T);
    int64_t st = s.d[3];
    for (int i = 2; i >= 0; --i) { m.ext[i] = s.d[i]; m.stride[i] = st; st *= s.d[i]; }
    return m;
  };
  for (int t : g.inputs) imap[t] = plain_map(t, g.tensors[t]);
  std::vector<char> by_compute(nt, 0);   // read by an arithmetic node, or a graph output
  for (size_t ni = 0; ni < g.nodes.size(); ++ni)
    if (!idx_like[ni]) for (int k = 0; k < g.nodes[ni].n_in; ++k) if (g.nodes[ni].in[k] < (uint32_t)nt) by_compute[g.nodes[ni].in[k]] = 1;
  for (int o : g.outputs) by_compute[o] = 1;
  for (size_t ni = 0; ni < g.nodes.size(); ++ni) {
    const Node& n = g.nodes[ni];
    if (!idx_like[ni]) continue;
    const std::string where = "node " + std::to_string(ni) + ": ";
    const Tensor& X = g.tensors[n.in[0]]; const Tensor& Y = g.tensors[n.out[0]];
    IdxMap m = imap[n.in[0]];
    if (m.root < 0) { err = where + "roll / slice / view apply to graph inputs (or chains of them) only"; return PN_ERR_UNSUPPORTED_OP; }
    if (Y.dtype != X.dtype) { err = where + "an index operator keeps the dtype"; return PN_ERR_UNSUPPORTED_OP; }
    if (X.rank < 1 || Y.rank < 1) { err = where + "index operators need a dimension to act on"; return PN_ERR_SHAPE; }
    // the last dimension changes only under a slice of it, or under a view of a tensor that is still dense
    const bool last_sliced = n.op == N_SLICE && (n.attr[0] == X.rank - 1 || (n.imm[0] != 0.0 && (int64_t)n.imm[0] - 1 == X.rank - 1));
    const bool dense_view = (n.op == N_VIEW || n.op == N_CONTIGUOUS) && m.plain;
    if (X.dims[X.rank - 1] != Y.dims[Y.rank - 1] && !last_sliced && !dense_view) { err = where + "the last dimension changes only under a slice of it or a view of a dense tensor"; return PN_ERR_SHAPE; }
    if (n.op == N_CONTIGUOUS && (X.rank != Y.rank || memcmp(X.dims, Y.dims, sizeof(X.dims)) != 0)) { err = where + "contiguous keeps the shape"; return PN_ERR_SHAPE; }
    if (n.op == N_VIEW || n.op == N_CONTIGUOUS) {
      if (X.numel() != Y.numel()) { err = where + "a view keeps the number of elements"; return PN_ERR_SHAPE; }
      if (m.plain) m = plain_map(m.root, Y); else m.frozen = true;
    } else {
      if (m.frozen) { err = where + "roll / slice after a view of a rolled or sliced tensor is not lowered"; return PN_ERR_UNSUPPORTED_OP; }
      // one dimension in attr (dim, shift / start); optionally a second one in imm (1 + dim, shift / start)
      int64_t dims2[2] = {n.attr[0], -1}, amt2[2] = {n.attr[1], 0};
      if (n.imm[0] != 0.0) {
        if (n.imm[0] != floor(n.imm[0]) || n.imm[1] != floor(n.imm[1]) || n.imm[0] < 1 || n.imm[0] > 4) { err = where + "second dimension of a roll / slice: imm = (1 + dim, shift / start), integers"; return PN_ERR_BAD_DESCRIPTOR; }
        dims2[1] = (int64_t)n.imm[0] - 1; amt2[1] = (int64_t)n.imm[1];
        if (dims2[1] == dims2[0]) { err = where + "a roll / slice names each dimension once"; return PN_ERR_SHAPE; }
      }
      if (X.rank != Y.rank) { err = where + "rank must be kept"; return PN_ERR_SHAPE; }
      for (int d = 0; d < X.rank; ++d)
        if (d != dims2[0] && d != dims2[1] && X.dims[d] != Y.dims[d]) { err = where + "only the rolled / sliced dimensions may change"; return PN_ERR_SHAPE; }
      for (int which = 0; which < 2; ++which) {
        const int64_t k = dims2[which];
        if (which == 1 && k < 0) break;
        if (k < 0 || k >= X.rank || X.rank > 4) { err = where + "roll / slice dimension outside the tensor"; return PN_ERR_SHAPE; }
        const int64_t Dk = X.dims[k];
        if (k == X.rank - 1) {   // the last dimension: a column offset (slice) or a circular column shift (roll)
          if (n.op == N_ROLL) {
            if (Y.dims[k] != Dk) { err = where + "a roll keeps the shape"; return PN_ERR_SHAPE; }
            if (m.col_sliced) { err = where + "roll after slice on the same dimension is not lowered"; return PN_ERR_UNSUPPORTED_OP; }
            if (Dk > 0) { m.col_add = ((m.col_add - amt2[which]) % Dk + Dk) % Dk; m.col_mod = Dk; }
          } else {
            const int64_t a = amt2[which], L = Y.dims[k];
            if (a < 0 || a + L > Dk) { err = where + "slice outside the tensor"; return PN_ERR_SHAPE; }
            m.col_add += a; m.col_sliced = true;
            if (m.col_mod) m.col_add %= m.col_mod;
          }
          continue;
        }
        const int kk = 3 - (X.rank - 1) + (int)k;
        if (n.op == N_ROLL) {
          if (Y.dims[k] != Dk) { err = where + "a roll keeps the shape"; return PN_ERR_SHAPE; }
          if (m.sliced[kk]) { err = where + "roll after slice on the same dimension is not lowered"; return PN_ERR_UNSUPPORTED_OP; }
          if (Dk > 0) { m.add[kk] = ((m.add[kk] - amt2[which]) % Dk + Dk) % Dk; m.mod[kk] = Dk; }
        } else {
          const int64_t a = amt2[which], L = Y.dims[k];
          if (a < 0 || a + L > Dk) { err = where + "slice outside the tensor"; return PN_ERR_SHAPE; }
          m.add[kk] += a; m.ext[kk] = L; m.sliced[kk] = true;
          if (m.mod[kk]) m.add[kk] %= m.mod[kk];
        }
      }
      m.plain = false;
    }
    imap[n.out[0]] = m;
  }
  // tensors that exist only to be re-indexed take no part in the iteration space
  std::vector<char> index_only(nt, 0);
  for (int t = 0; t < nt; ++t) index_only[t] = imap[t].root >= 0 && !by_compute[t];

  for (size_t ni = 0; ni < g.nodes.size(); ++ni) {   // per-row scalars
    const Node& n = g.nodes[ni];
    if (idx_like[ni]) continue;
    if (is_reduction(n.op)) is_s[n.out[0]] = 1;
    else if (n.op == N_LAYER_NORM) { for (int k = 1; k < n.n_out; ++k) is_s[n.out[k]] = 1; }
    else if (!is_composite(n.op)) {
      bool any_t = false, all_s = true;
      for (int k = 0; k < n.n_in; ++k) {
        if (n.in[k] >= (uint32_t)nt) continue;
        any_t = true;
        all_s = all_s && is_s[n.in[k]];
      }
      if (!any_t) { err = "a node with only constant operands is not lowered"; return PN_ERR_UNSUPPORTED_OP; }
      if (all_s) is_s[n.out[0]] = 1;
    }
  }
  Shape4 F{{1, 1, 1, 1}};
  bool have_full = false;
  for (const Node& n : g.nodes) {
    if (is_reduction(n.op) || is_composite(n.op)) {
      const Shape4 s = align4(g.tensors[n.in[0]]);
      if (!have_full) { F = s; have_full = true; }
      else if (memcmp(&F, &s, sizeof(s)) != 0) { err = "all reductions of a graph must act on the same shape"; return PN_ERR_SHAPE; }
    }
  }
  for (int t = 0; t < nt; ++t) {
    if (is_s[t] || index_only[t]) continue;
    const Shape4 s = align4(g.tensors[t]);
    if (has_red) {
      for (int i = 0; i < 4; ++i)
        if (s.d[i] != 1 && s.d[i] != F.d[i]) { err = "tensor " + std::to_string(t) + " does not broadcast into the iteration space"; return PN_ERR_SHAPE; }
    } else if (!bcast_into(F, s)) { err = "tensor " + std::to_string(t) + ": shapes do not broadcast"; return PN_ERR_SHAPE; }
  }
  const int64_t rows = F.d[0] * F.d[1] * F.d[2];
  const int64_t N = F.d[3];
  if (N <= 0) { err = "the last dimension is empty"; return PN_ERR_SHAPE; }
  if (N >= (int64_t(1) << 30)) { err = "last dimension too long"; return PN_ERR_TOO_LARGE; }
  for (size_t ni = 0; ni < g.nodes.size(); ++ni) {   // per-node shape rules
    const Node& n = g.nodes[ni];
    if (idx_like[ni]) continue;   // checked with the chains above
    const std::string where = "node " + std::to_string(ni) + ": ";
    auto row_shaped = [&](const Tensor& t, const Tensor& src) {
      if (t.rank == src.rank - 1) { for (int i = 0; i < t.rank; ++i) if (t.dims[i] != src.dims[i]) return false; return true; }
      if (t.rank == src.rank) { for (int i = 0; i + 1 < t.rank; ++i) if (t.dims[i] != src.dims[i]) return false; return t.rank > 0 && t.dims[t.rank - 1] == 1; }
      return false;
    };
    if (is_reduction(n.op) || is_composite(n.op)) {
      const Tensor& src = g.tensors[n.in[0]];
      if (src.rank < 1) { err = where + "reduction of a rank-0 tensor"; return PN_ERR_SHAPE; }
      if (is_s[n.in[0]]) { err = where + "reduction of a per-row result"; return PN_ERR_UNSUPPORTED_OP; }
      if (is_reduction(n.op)) {
        if (!row_shaped(g.tensors[n.out[0]], src)) { err = where + "result must have the input's shape with the last dim dropped or 1"; return PN_ERR_SHAPE; }
        if ((n.op == N_ARGMAX || n.op == N_ARGMIN) && g.tensors[n.out[0]].dtype != kI64 && g.tensors[n.out[0]].dtype != kI32) {
          err = where + "argmax / argmin results must be i32 or i64"; return PN_ERR_UNSUPPORTED_OP;
        }
      } else {
        const Tensor& y = g.tensors[n.out[0]];
        if (y.rank != src.rank || memcmp(y.dims, src.dims, sizeof(int64_t) * 4) != 0) { err = where + "output shape differs from the input's"; return PN_ERR_SHAPE; }
        for (int k = 1; k < n.n_out; ++k)
          if (!row_shaped(g.tensors[n.out[k]], src)) { err = where + "mean / rstd must have the per-row shape"; return PN_ERR_SHAPE; }
      }
    } else {
      Shape4 b{{1, 1, 1, 1}};
      for (int k = 0; k < n.n_in; ++k)
        if (n.in[k] < (uint32_t)nt && !bcast_into(b, align4(g.tensors[n.in[k]]))) { err = where + "operands do not broadcast"; return PN_ERR_SHAPE; }
      const Shape4 o = align4(g.tensors[n.out[0]]);
      if (memcmp(&b, &o, sizeof(o)) != 0) { err = where + "declared output shape is not the broadcast of the operands"; return PN_ERR_SHAPE; }
    }
  }
  for (int o : g.outputs) {
    if (is_s[o]) continue;
    const Shape4 s = align4(g.tensors[o]);
    if (memcmp(&s, &F, sizeof(s)) != 0) { err = "output tensor " + std::to_string(o) + " must have the full iteration shape or be a per-row result"; return PN_ERR_UNSUPPORTED_OP; }
  }

  // ---- io table ------------------------------------------------------------------------
  memset(&lp, 0, sizeof(lp));
  KernelParams& P = lp.p;
  // input-like entries: graph inputs read directly, and re-indexed views of graph inputs
  std::vector<int> in_like;
  for (int t = 0; t < nt; ++t)
    if (imap[t].root >= 0 && by_compute[t] && ((g.tensors[t].role & 1) || g.tensors[t].producer >= 0)) in_like.push_back(t);
  const int n_io = (int)(in_like.size() + g.outputs.size());
  if (n_io > kMaxIo) { err = "more graph inputs + outputs than one kernel takes (" + std::to_string(kMaxIo) + ")"; return PN_ERR_TOO_LARGE; }
  P.n_io = n_io;
  std::vector<int> io_of_tensor(nt, -1), in_io_of_tensor(nt, -1);
  std::vector<char> io_streamed(n_io, 0);
  bool any_mapped = false;
  {
    int idx = 0;
    auto add_io = [&](int t, bool is_out) -> bool {
      IoDesc& io = P.io[idx];
      const Tensor& T = g.tensors[t];
      io.dtype = T.dtype;
      if (is_s[t]) {   // one element per row, dense over the leading dims
        io.is_row_scalar = 1; io.col_stride = 0;
        io.lead_stride[2] = 1; io.lead_stride[1] = F.d[2]; io.lead_stride[0] = F.d[2] * F.d[1];
      } else {
        const Shape4 s = align4(T);
        int64_t st = 1, strides[4];
        bool full = true;
        for (int i = 3; i >= 0; --i) { strides[i] = (s.d[i] == 1 && F.d[i] != 1) ? 0 : st; st *= s.d[i]; full = full && s.d[i] == F.d[i]; }
        for (int i = 0; i < 3; ++i) io.lead_stride[i] = F.d[i] == 1 ? 0 : strides[i];
        io.col_stride = (s.d[3] == 1 && N != 1) ? 0 : 1;
        io_streamed[idx] = full;
      }
      lp.io_offset[idx] = 0;
      if (is_out && T.embed_parent >= 0) {   // stored as a block of a larger tensor: the parent's strides, the block's start
        if (is_s[t]) return false;
        int64_t st = 1, ps[4];
        for (int i = 3; i >= 0; --i) { ps[i] = st; st *= T.embed_dims[i]; }
        for (int i = 0; i < 3; ++i) io.lead_stride[i] = F.d[i] == 1 ? 0 : ps[i];
        for (int i = 0; i < 4; ++i) lp.io_offset[idx] += T.embed_off[i] * ps[i];
      }
      if (!is_out && !imap[t].plain) {   // read through rolls / slices: own coordinates, source strides
        const IdxMap& m = imap[t];
        const Shape4 s = align4(T);
        if (m.ext[0] * m.ext[1] * m.ext[2] != rows || s.d[3] != N) return false;
        io.mapped = 1; io.col_stride = 1; io_streamed[idx] = 1; any_mapped = true;
        for (int i = 0; i < 3; ++i) {
          io.lead_stride[i] = m.stride[i];
          io.map_dim[i] = (int32_t)std::max<int64_t>(m.ext[i], 1); io.map_add[i] = (int32_t)m.add[i]; io.map_mod[i] = (int32_t)m.mod[i];
        }
        if (m.col_mod) { io.col_add = (int32_t)m.col_add; io.col_mod = (int32_t)m.col_mod; }   // rolled columns wrap in the kernel
        else lp.io_offset[idx] += m.col_add;                                                     // sliced columns: the row starts later
      }
      lp.io_tensor[idx] = is_out ? t : imap[t].root; lp.io_is_output[idx] = is_out;
      if (is_out) io_of_tensor[t] = idx; else in_io_of_tensor[t] = idx;
      ++idx;
      return true;
    };
    for (int t : in_like)
      if (!add_io(t, false)) { err = "tensor " + std::to_string(t) + ": a rolled / sliced input must cover the whole iteration space"; return PN_ERR_UNSUPPORTED_OP; }
    for (int t : g.outputs)
      if (!add_io(t, true)) { err = "tensor " + std::to_string(t) + ": a per-row result cannot be an operand of a cat"; return PN_ERR_UNSUPPORTED_OP; }
  }
  // collapse leading dims that every io walks contiguously (or broadcasts) together
  int64_t lead_dim[3] = {F.d[0], F.d[1], F.d[2]};
  for (int pass = 0; pass < 2; ++pass) {
    for (int i = 1; i >= 0; --i) {   // try merging dim i into dim i+1
      if (lead_dim[i] == 1) continue;
      bool ok = true;
      if (lead_dim[i + 1] != 1)
        for (int q = 0; q < n_io && ok; ++q) ok = P.io[q].mapped || P.io[q].lead_stride[i] == P.io[q].lead_stride[i + 1] * lead_dim[i + 1];
      if (!ok) continue;
      for (int q = 0; q < n_io; ++q) {
        IoDesc& io = P.io[q];
        if (io.mapped) continue;   // splits the row index by its own extents
        if (lead_dim[i + 1] == 1) io.lead_stride[i + 1] = io.lead_stride[i];
        io.lead_stride[i] = 0;
      }
      lead_dim[i + 1] *= lead_dim[i]; lead_dim[i] = 1;
    }
  }
  for (int i = 0; i < 3; ++i) if (lead_dim[i] > 0xFFFFFFFFll) { err = "leading dimension too large"; return PN_ERR_TOO_LARGE; }
  int64_t eff_rows = rows, eff_N = N;
  // a purely pointwise graph whose tensors all have the full shape is one long row
  if (!has_red && !any_mapped && rows > 1 && rows * N < (int64_t(1) << 30) && lead_dim[0] == 1 && lead_dim[1] == 1) {
    bool flat = true;
    for (int q = 0; q < n_io; ++q) flat = flat && P.io[q].col_stride == 1 && P.io[q].lead_stride[2] == N;
    if (flat) { eff_N = rows * N; eff_rows = 1; lead_dim[2] = 1; for (int q = 0; q < n_io; ++q) P.io[q].lead_stride[2] = 0; }
  }
  for (int i = 0; i < 3; ++i) P.lead_dim[i] = (uint32_t)std::max<int64_t>(lead_dim[i], 1);
  P.rows = eff_rows;
  P.row_len = (int32_t)eff_N;

  // ---- (2) micro-operations --------------------------------------------------------------
  Expander ex;
  std::vector<Val>& vals = ex.vals;
  std::vector<MOp>& ops = ex.ops;
  int& n_slots = ex.n_slots;
  std::vector<int> tval(nt, -1);
  std::vector<std::vector<RedDesc>> stage_reds(kMaxStages);
  std::map<std::pair<int, int>, int> red_cache;   // (kind, value) -> first slot
  auto new_val = [&](ValKind k, int stage) { return ex.new_val(k, stage); };
  auto new_slot = [&](int n) { return ex.new_slot(n); };
  auto add_op = [&](int op, int stage, bool scalar, std::initializer_list<int> in, int out, int a0 = 0, int a1 = 0) {
    ex.add_op(op, stage, scalar, in, out, a0, a1);
  };
  for (int t : in_like) {
    const int v = new_val(VK_E, 0);
    const int q = in_io_of_tensor[t];
    vals[v].io = q;
    vals[v].bcast = P.io[q].col_stride == 0;
    vals[v].streamed = io_streamed[q];
    vals[v].invariant = !P.io[q].mapped && P.io[q].lead_stride[0] == 0 && P.io[q].lead_stride[1] == 0 && P.io[q].lead_stride[2] == 0;
    vals[v].integral = !dtype_is_float(g.tensors[t].dtype);
    vals[v].mask8 = g.tensors[t].dtype == kI8 || g.tensors[t].dtype == kBool;
    tval[t] = v;
  }
  std::vector<char> feeds_var(nt, 0);
  for (const Node& n : g.nodes) if (n.op == N_VAR) feeds_var[n.in[0]] = 1;

  auto pointwise = [&](int vmop, std::initializer_list<int> in, bool integral) { return ex.pointwise(vmop, in, integral); };
  auto slot_val = [&](int slot, int stage, bool int_bits) { return ex.slot_val(slot, stage, int_bits); };
  auto imm_val = [&](double x) { return ex.imm_val(x); };
  // reduction of tile value x; returns the first of its 3 slots, -1 / -2 when a budget is hit
  auto reduce = [&](int kind, int x, int* e_out) -> int {
    const int s = vals[x].stage;
    auto key = std::make_pair(kind, x);
    if (kind != RED_SOFTMAX && red_cache.count(key)) return red_cache[key];
    if (s >= kMaxStages - 1) return -1;
    if ((int)stage_reds[s].size() >= kMaxRed) return -2;
    const int base = new_slot(3);
    RedDesc rd; rd.kind = (uint8_t)kind; rd.slot = (uint8_t)base; rd.uniform = 0;
    const int ridx = (int)stage_reds[s].size();
    stage_reds[s].push_back(rd);
    int e = -1;
    if (kind == RED_SOFTMAX) { e = new_val(VK_E, s); vals[e].has_ts = true; }
    add_op(OP_RED, s, false, {x}, e, kind, ridx);
    if (e_out) *e_out = e;
    red_cache[key] = base;
    return base;
  };

  int softmax_count = 0;
  for (size_t ni = 0; ni < g.nodes.size(); ++ni) {
    const Node& n = g.nodes[ni];
    const std::string where = "node " + std::to_string(ni) + ": ";
    int in[4] = {-1, -1, -1, -1};
    for (int k = 0; k < n.n_in; ++k) {
      if (n.in[k] == kImm0) in[k] = imm_val(n.imm[0]);
      else if (n.in[k] == kImm1) in[k] = imm_val(n.imm[1]);
      else in[k] = tval[n.in[k]];
    }
    if (idx_like[ni]) {
      const int t = n.out[0];
      if (g.tensors[t].role & 2) {
        if (tval[t] < 0) { err = where + "internal: re-indexed output without a value"; return PN_ERR_UNSUPPORTED_OP; }
        add_op(OP_STOUT, 0, false, {tval[t]}, -1, io_of_tensor[t], 0);
      }
      continue;
    }
    int res[3] = {-1, -1, -1};
    const double Nd = (double)N;
    const int pw = ex.expand_pointwise(g, n, in, res, err, where);
    if (pw < 0) return pw;
    if (pw == 1) {   // a pointwise node: done
    } else if (is_reduction(n.op) || is_composite(n.op)) {
      const int x = in[0];
      if (vals[x].kind != VK_E) { err = where + "reduction of a per-row value"; return PN_ERR_UNSUPPORTED_OP; }
      const int s1 = vals[x].stage + 1;
      int base = 0;
      auto bad = [&](int b) {
        if (b == -1) { err = where + "more reduction-dependent stages than the kernel takes"; return true; }
        if (b == -2) { err = where + "more reductions in one stage than the kernel takes"; return true; }
        return false;
      };
      switch (n.op) {
        case N_SUM: base = reduce(RED_SUM, x, nullptr); if (bad(base)) return PN_ERR_TOO_LARGE; res[0] = slot_val(base, s1, false); break;
        case N_AMAX: base = reduce(RED_MAX, x, nullptr); if (bad(base)) return PN_ERR_TOO_LARGE; res[0] = slot_val(base, s1, false); break;
        case N_AMIN: base = reduce(RED_MIN, x, nullptr); if (bad(base)) return PN_ERR_TOO_LARGE; res[0] = slot_val(base, s1, false); break;
        case N_ARGMAX: base = reduce(RED_ARGMAX, x, nullptr); if (bad(base)) return PN_ERR_TOO_LARGE; res[0] = slot_val(base + 1, s1, true); break;
        case N_ARGMIN: base = reduce(RED_ARGMIN, x, nullptr); if (bad(base)) return PN_ERR_TOO_LARGE; res[0] = slot_val(base + 1, s1, true); break;
        case N_MEAN:
          if (feeds_var[n.in[0]]) { base = reduce(RED_MEANVAR, x, nullptr); if (bad(base)) return PN_ERR_TOO_LARGE; res[0] = slot_val(base + 1, s1, false); }
          else { base = reduce(RED_SUM, x, nullptr); if (bad(base)) return PN_ERR_TOO_LARGE; res[0] = pointwise(OP_DIV, {slot_val(base, s1, false), imm_val(Nd)}, false); }
          break;
        case N_VAR: {
          base = reduce(RED_MEANVAR, x, nullptr); if (bad(base)) return PN_ERR_TOO_LARGE;
          res[0] = pointwise(OP_DIV, {slot_val(base + 2, s1, false), imm_val(Nd - (double)n.attr[0])}, false);
          break;
        }
        case N_LOGSUMEXP: case N_LOG_SOFTMAX: {
          base = reduce(RED_LSE, x, nullptr); if (bad(base)) return PN_ERR_TOO_LARGE;
          const int lse = pointwise(OP_LSEFIN, {slot_val(base, s1, false), slot_val(base + 1, s1, false)}, false);
          res[0] = n.op == N_LOGSUMEXP ? lse : pointwise(OP_SUB, {x, lse}, false);
          break;
        }
        case N_SOFTMAX: {
          if (++softmax_count > 1) { err = where + "more than one softmax per graph is not lowered"; return PN_ERR_UNSUPPORTED_OP; }
          int e = -1;
          base = reduce(RED_SOFTMAX, x, &e); if (bad(base)) return PN_ERR_TOO_LARGE;
          const int inv = pointwise(OP_RECIP, {slot_val(base + 1, s1, false)}, false);
          const int r = new_val(VK_E, s1);
          add_op(OP_SCALE_TS, s1, false, {e}, r, base, vals[inv].slot);
          res[0] = r;
          break;
        }
        case N_LAYER_NORM: {
          base = reduce(RED_MEANVAR, x, nullptr); if (bad(base)) return PN_ERR_TOO_LARGE;
          const int mean = slot_val(base + 1, s1, false);
          const int var = pointwise(OP_DIV, {slot_val(base + 2, s1, false), imm_val(Nd)}, false);
          const int ve = pointwise(OP_ADD, {var, imm_val(n.imm[0])}, false);
          const int rstd = pointwise(OP_RSQRT, {ve}, false);
          int y = pointwise(OP_SUB, {x, mean}, false);
          y = pointwise(OP_MUL, {y, rstd}, false);
          if (n.n_in > 1) y = pointwise(OP_MUL, {y, in[1]}, false);
          if (n.n_in > 2) y = pointwise(OP_ADD, {y, in[2]}, false);
          res[0] = y; res[1] = mean; res[2] = rstd;
          break;
        }
        case N_RMS_NORM: {
          const int sq = pointwise(OP_SQUARE, {x}, false);
          base = reduce(RED_SUM, sq, nullptr); if (bad(base)) return PN_ERR_TOO_LARGE;
          const int ms = pointwise(OP_DIV, {slot_val(base, s1, false), imm_val(Nd)}, false);
          const int me = pointwise(OP_ADD, {ms, imm_val(n.imm[0])}, false);
          const int r = pointwise(OP_RSQRT, {me}, false);
          int y = pointwise(OP_MUL, {x, r}, false);
          if (n.n_in > 1) y = pointwise(OP_MUL, {y, in[1]}, false);
          res[0] = y;
          break;
        }
      }
    } else { err = where + "opcode not lowered"; return PN_ERR_UNSUPPORTED_OP; }

    const int fin = ex.finish_node(g, n, res, n_consumers, io_of_tensor, tval, kMaxStages, err, where);
    if (fin != PN_OK) return fin;
  }
  if (n_slots > kMaxSlots) { err = "more per-row scalars than the kernel takes"; return PN_ERR_TOO_LARGE; }
  for (const MOp& m : ops) for (int i = 0; i < m.nin; ++i) vals[m.in[i]].uses++;
  int n_stages = 1;
  for (const MOp& m : ops) n_stages = std::max(n_stages, m.stage + 1);
  if (n_stages > kMaxStages) { err = "more reduction-dependent stages than the kernel takes"; return PN_ERR_TOO_LARGE; }

  bool cross_stage = false;   // a tile value made in one stage and read in a later one: the row must stay resident
  for (const MOp& m : ops) for (int i = 0; i < m.nin; ++i)
    if (!m.scalar && vals[m.in[i]].kind == VK_E && vals[m.in[i]].stage < m.stage) cross_stage = true;

  // ---- (3) family and tile shape ---------------------------------------------------------
  int min_esize = 8;
  bool vec8 = true, vec4 = true;
  for (int q = 0; q < n_io; ++q) {
    const IoDesc& io = P.io[q];
    if (io.is_row_scalar || io.col_stride == 0) continue;
    if (io_streamed[q]) min_esize = std::min(min_esize, dtype_bytes(io.dtype));
    for (int vl : {8, 4}) {
      bool ok = eff_N % vl == 0 && lp.io_offset[q] % vl == 0 && io.col_add % vl == 0 && io.col_mod % vl == 0;
      for (int i = 0; i < 3; ++i) ok = ok && io.lead_stride[i] % vl == 0;
      if (vl == 8) vec8 = vec8 && ok; else vec4 = vec4 && ok;
    }
  }
  int VL = (min_esize <= 2 && vec8) ? 8 : (vec4 ? 4 : 1);
  const bool spec = dev.specialise;
  // A group of 8 elements of a 4-byte operand is two 128-bit accesses 32 bytes apart from lane to
  // lane: each touches every 128-byte line of the warp's span and uses half of it, so the operand
  // costs twice the L1 wavefronts.  Measured on the residual + LayerNorm workload (bf16 rows, fp32
  // gamma and beta re-read by every row): the L1 data pipe at 74 % with groups of 8, and 73.7 ->
  // 66.4 us with groups of 4 (the 2-byte rows then move in 64-bit accesses, which stay whole).
  // Groups of 8 are kept where such operands are loaded once per thread, not per row: the
  // warp-per-row kernels, which pin row-invariant operands in registers.
  if (VL == 8 && vec4) {
    bool wide_per_row = false, wide_varying = false;
    for (int q = 0; q < n_io; ++q) {
      const IoDesc& io = P.io[q];
      if (io.is_row_scalar || io.col_stride == 0 || dtype_bytes(io.dtype) < 4) continue;
      wide_per_row = true;
      if (io.mapped || io.lead_stride[0] != 0 || io.lead_stride[1] != 0 || io.lead_stride[2] != 0 || lp.io_is_output[q]) wide_varying = true;
    }
    const bool pinned_in_warp = has_red && spec && !wide_varying && eff_N <= 32 * 64 &&
                                !(flags & (PN_FLAG_FORCE_BLOCK | PN_FLAG_FORCE_CLUSTER | PN_FLAG_FORCE_MULTICHUNK | PN_FLAG_NO_HOIST));
    if (wide_per_row && !pinned_in_warp) VL = 4;
  }
  if (flags & PN_FLAG_FORCE_SCALAR) VL = 1;
  std::vector<std::pair<int, int>> ng_opts;   // (NG, K): the 8-element tile first
  if (VL == 8) ng_opts = {{1, 4}, {2, 2}};
  else if (VL == 4) ng_opts = {{2, 4}, {4, 2}};
  else ng_opts = {{8, 4}};
  if (spec) for (auto& o : ng_opts) o.second = kSpecRegs;   // a generated kernel pays only for live registers

  std::vector<Config> cands;
  const int sms = dev.sm_count;
  auto chunks_of = [&](int64_t len, int T, int ng) { const int64_t cap = (int64_t)T * VL * ng; return (int)((len + cap - 1) / cap); };
  if (!has_red) {
    // A generated kernel on a problem too small to give every SM several blocks takes one group
    // per thread: twice the blocks, spread more evenly (measured: 4.28 -> 4.03 us on the 12.6 MB
    // pointwise chain; at 768 MB two groups per thread reach the copy rate).
    if (spec && VL > 1 && ng_opts.front().first > 1) {
      const int64_t blocks = (eff_rows * chunks_of(eff_N, 32, ng_opts.front().first) + 7) / 8;
      if (blocks < 8ll * sms) cands.push_back(Config{FAM_POINTWISE, VL, 1, kSpecRegs, 256, 1, chunks_of(eff_N, 32, 1), (int)eff_N, false});
    }
    for (auto o : ng_opts) cands.push_back(Config{FAM_POINTWISE, VL, o.first, o.second, 256, 1, chunks_of(eff_N, 32, o.first), (int)eff_N, false});
  } else {
    const bool fw = flags & PN_FLAG_FORCE_WARP, fb = flags & PN_FLAG_FORCE_BLOCK, fc = flags & PN_FLAG_FORCE_CLUSTER;
    const bool fm = flags & PN_FLAG_FORCE_MULTICHUNK;
    const bool fs = flags & PN_FLAG_FORCE_SPLIT;
    const bool any_force = fw || fb || fc || fs;
    const bool few_rows = eff_rows < 2ll * sms;
    // the interpreter's 16-element-tile instances are built for at most 256 threads
    auto tile_ok = [&](int T, int ng) { return spec || !(T > 256 && VL * ng > 8); };
    // one chunk per thread.  Generated kernels (measured on B200 over row lengths 256..8192,
    // LayerNorm and softmax graphs): a warp per row while the row fits in 64 two-byte (32
    // four-byte) elements per lane -- no block barrier at all -- and beyond that a block of
    // N / 32 threads holding 32 (16) elements each, when the epilogue needs the row again.
    if (spec && !fm && !fc && !fs && VL > 1) {
      const int v_warp = min_esize <= 2 ? 64 : 32, v_block = min_esize <= 2 ? 32 : 16;
      if (!fb)
        for (int ng = 1; VL * ng <= v_warp; ng *= 2)
          if (32ll * VL * ng >= eff_N) {
            // rows of at most 16 (8) groups: two (four) of them share a warp, so that most lanes work
            const int lanes = ng > 1 ? 32 : (8ll * VL >= eff_N ? 8 : (16ll * VL >= eff_N ? 16 : 32));
            cands.push_back(Config{FAM_WARP, VL, ng, kSpecRegs, 256, 1, 1, (int)eff_N, false, lanes});
            break;
          }
      if (!fw && cands.empty() && cross_stage)   // rows that need no residency stream in chunks instead
        for (int T : {64, 128, 256, 512})
          if ((int64_t)T * v_block >= eff_N) { cands.push_back(Config{FAM_BLOCK, VL, v_block / VL, kSpecRegs, T, 1, 1, (int)eff_N, false}); break; }
    }
    // Few long rows whose elements are needed once (a single stage): independent blocks over slices
    // of the rows, in memory order, meeting per row through partials in device memory (generated
    // kernels; needs a workspace, so not for handles that may not allocate).  About 32 KB of a
    // four-byte input per block (128 bytes in flight per thread) measured best on B200; smaller
    // slices when the rows are so few that the SMs would not all get several blocks.
    if (spec && VL > 1 && n_stages == 1 && !cross_stage && !(flags & PN_FLAG_STATIC_SCRATCH) &&
        ((!any_force && !fm && few_rows && cands.empty()) || fs)) {   // (rows short enough for a warp stay with it)
      // (blocks of 128 once there are thousands of slices: [256, 262144] 46.7 -> 45.0 us; slower below that)
      const int T = eff_rows * ((eff_N + 256ll * 32 - 1) / (256ll * 32)) >= 8192 ? 128 : 256;
      for (int ng : {8, 4, 2, 1}) {
        if (VL * ng > 32) continue;
        const int64_t tile = (int64_t)T * VL * ng;
        int seg_chunks = 1;
        while ((eff_N + tile * seg_chunks - 1) / (tile * seg_chunks) > 1024) seg_chunks *= 2;   // at most 1024 partials per row
        const int64_t slice = tile * seg_chunks;
        const int64_t S = (eff_N + slice - 1) / slice;
        if (S < 2 && !fs) continue;
        if (eff_rows * S > (int64_t(1) << 30)) continue;
        if (eff_rows * S < 4ll * sms && ng > 1) continue;   // too few blocks: smaller slices
        Config c{FAM_SPLIT, VL, ng, kSpecRegs, T, 1, seg_chunks, (int)slice, false, 32, (int)S};
        cands.push_back(c);
        break;
      }
    }
    // the smallest team that holds the row in one of the interpreter's tile shapes
    if (!fm && !fc && !fs) {
      for (int T : {32, 64, 128, 256, 512}) {
        if ((fw && T != 32) || (fb && T == 32)) continue;
        for (auto o : ng_opts)
          if (tile_ok(T, o.first) && (int64_t)T * VL * o.first >= eff_N)
            cands.push_back(Config{T == 32 ? FAM_WARP : FAM_BLOCK, VL, o.first, o.second, T == 32 ? 256 : T, 1, 1, (int)eff_N, false});
      }
    }
    // several chunks per thread
    if (fw)
      for (auto o : ng_opts) {
        const int ch = chunks_of(eff_N, 32, o.first);
        cands.push_back(Config{FAM_WARP, VL, o.first, o.second, 256, 1, ch, (int)eff_N, ch > 1});
      }
    if ((!any_force && !few_rows) || fb) {
      std::vector<Config> mc;
      for (int T : fm ? std::vector<int>{64} : std::vector<int>{256, 512})
        for (auto o : ng_opts) {
          if (!tile_ok(T, o.first)) continue;
          const int ch = chunks_of(eff_N, T, o.first);
          mc.push_back(Config{FAM_BLOCK, VL, o.first, o.second, T, 1, ch, (int)eff_N, ch > 1});
        }
      std::stable_sort(mc.begin(), mc.end(), [&](const Config& a, const Config& b) {
        return (int64_t)a.chunks * a.block * a.vl * a.ng < (int64_t)b.chunks * b.block * b.vl * b.ng;   // least padding first
      });
      cands.insert(cands.end(), mc.begin(), mc.end());
    }
    if ((!any_force && few_rows) || fc || cands.empty()) {
      std::vector<std::pair<int, int>> cl_opts = ng_opts;
      if (spec && !fm) std::reverse(cl_opts.begin(), cl_opts.end());   // more bytes in flight per thread
      // the fewest CTAs per row that still put at least one CTA on every SM
      std::vector<int> cl_sizes = {2, 4, 8};
      std::stable_sort(cl_sizes.begin(), cl_sizes.end(), [&](int a, int b) {
        const bool fa = eff_rows * a >= sms, fb2 = eff_rows * b >= sms;
        return fa != fb2 ? fa : (fa ? a < b : a > b);
      });
      for (int C : cl_sizes)
        for (auto o : cl_opts) {
          const int T = fm ? 64 : (spec && (eff_N + C - 1) / C >= 2ll * 512 * VL * o.first) ? 512 : 256;
          int64_t slice = (eff_N + C - 1) / C;
          slice = (slice + VL - 1) / VL * VL;
          if (slice * (C - 1) >= eff_N) continue;                              // a CTA would get no columns
          if (!fc && !fm && slice < (int64_t)T * VL * o.first) continue;     // keep every CTA busy
          const int ch = chunks_of(slice, T, o.first);
          cands.push_back(Config{FAM_CLUSTER, VL, o.first, o.second, T, C, ch, (int)slice, ch > 1});
        }
      for (auto o : ng_opts) {   // rows too short to split: plain blocks
        const int ch = chunks_of(eff_N, 256, o.first);
        cands.push_back(Config{FAM_BLOCK, VL, o.first, o.second, 256, 1, ch, (int)eff_N, ch > 1});
      }
    }
  }

  // tuning overrides: keep only the candidates that match, or add the asked-for shape
  {
    const int t_cluster = (flags >> 16) & 15, t_block = ((flags >> 20) & 15) ? 1 << ((flags >> 20) & 15) : 0, t_ng = (flags >> 24) & 31;
    if ((t_cluster || t_block || t_ng) && !cands.empty()) {
      std::vector<Config> extra;
      for (Config c : cands) {
        if (t_ng) {
          bool ok = spec && (t_ng & (t_ng - 1)) == 0 && VL * t_ng <= 128;   // generated kernels take any power of two
          for (auto o : ng_opts) ok = ok || o.first == t_ng;
          if (!ok) continue;
          c.ng = t_ng;
          for (auto o : ng_opts) if (o.first == t_ng) c.k = o.second;
        }
        if (t_block && c.family != FAM_WARP && c.family != FAM_POINTWISE) c.block = t_block;
        if (t_cluster && c.family == FAM_CLUSTER) c.cluster = t_cluster;
        if (t_cluster && c.family == FAM_BLOCK && has_red) { c.family = FAM_CLUSTER; c.cluster = t_cluster; }
        if (c.block < 32 || c.block > 1024 || (c.cluster != 1 && c.cluster != 2 && c.cluster != 4 && c.cluster != 8)) continue;
        if (!spec && c.block > 256 && c.vl * c.ng > 8) continue;
        if (c.family == FAM_SPLIT) {   // PN_TUNE_CLUSTER(n) on a split-row kernel: n tiles per slice
          const int64_t tile = (int64_t)c.block * VL * c.ng;
          int seg_chunks = t_cluster ? t_cluster : 1;
          while ((eff_N + tile * seg_chunks - 1) / (tile * seg_chunks) > 1024) seg_chunks *= 2;
          c.cluster = 1; c.chunks = seg_chunks; c.slice_len = (int)(tile * seg_chunks);
          c.splits = (int)((eff_N + c.slice_len - 1) / c.slice_len);
          c.multichunk = false;
          if (eff_rows * c.splits > (int64_t(1) << 30)) continue;
          extra.push_back(c);
          continue;
        }
        const int team = c.family <= FAM_WARP ? 32 : c.block;
        int64_t slice = (eff_N + c.cluster - 1) / c.cluster;
        slice = (slice + VL - 1) / VL * VL;
        if (c.cluster > 1 && slice * (c.cluster - 1) >= eff_N) continue;
        c.slice_len = (int)slice;
        c.chunks = chunks_of(slice, team, c.ng);
        c.multichunk = c.family != FAM_POINTWISE && c.chunks > 1;
        extra.push_back(c);
      }
      if (!extra.empty()) cands = extra;
    }
  }

  // ---- (4) code generation: first candidate whose program fits -----------------------------
  std::string gen_err = "no kernel configuration fits this graph";
  for (const Config& cf : cands) {
    std::vector<Val> v2 = vals;
    std::vector<uint32_t> code;
    std::map<int, int> stash_of;
    int n_stash = 0;
    StageDesc stages[kMaxStages];
    memset(stages, 0, sizeof(stages));
    bool ok = true;
    Gen ge(code, v2, false, cf.k, cf.multichunk, stash_of, n_stash);
    // rows held in one chunk per thread: the operands that do not depend on the row are loaded
    // once, before the row loop (generated kernels only: they have the registers for it)
    const bool pin = spec && cf.chunks == 1 && cf.family == FAM_WARP && !(flags & PN_FLAG_NO_HOIST);
    const uint16_t pro_begin = (uint16_t)code.size();
    if (pin) ge.pin_invariants(ops, 4);
    const uint16_t pro_end = (uint16_t)code.size();
    const bool persistent = pro_end > pro_begin;
    for (int s = 0; s < n_stages && ok; ++s) {
      stages[s].elem_begin = (uint16_t)code.size();
      ge.hoist_loads(ops, s);
      for (const MOp& m : ops) {
        if (m.stage != s || m.scalar) continue;
        if (!ge.gen(m)) { ok = false; gen_err = ge.err; break; }
      }
      if (ok && !ge.end_stage()) { ok = false; gen_err = ge.err; }
      stages[s].elem_end = (uint16_t)code.size();
      stages[s].scal_begin = (uint16_t)code.size();
      Gen gs(code, v2, true, 4, false, stash_of, n_stash);
      for (const MOp& m : ops) {
        if (m.stage != s || !m.scalar || !ok) continue;
        if (!gs.gen(m)) { ok = false; gen_err = gs.err; }
      }
      stages[s].scal_end = (uint16_t)code.size();
      stages[s].n_red = (uint8_t)stage_reds[s].size();
      for (size_t r = 0; r < stage_reds[s].size(); ++r) stages[s].red[r] = stage_reds[s][r];
    }
    if (!ok) continue;
    if ((int)code.size() > kMaxCode) { gen_err = "bytecode longer than the kernel takes"; continue; }
    if (n_stash > kMaxStash) { gen_err = "too many tile values cross a reduction"; continue; }

    // ---- (5) shared memory and grid ------------------------------------------------------
    const int lanes = (cf.family == FAM_WARP && (cf.lanes == 16 || cf.lanes == 8)) ? cf.lanes : 32;
    const int teams = cf.family <= FAM_WARP ? cf.block / lanes : 1;
    int off = 0;
    auto take = [&](int bytes) { const int o = off; off += (bytes + 15) / 16 * 16; return o; };
    P.sm_rowoff = take(teams * kMaxIo * 8);
    P.sm_slots = take(teams * kMaxSlots * 4);
    P.sm_part = take(has_red && !spec ? kMaxRed * 3 * cf.block * 4 : 0);   // generated kernels keep their partials in registers
    P.sm_wpart = take(has_red ? 2 * 32 * kMaxRed * 3 * 4 : 0);   // two alternating buffers
    P.sm_ctapart = take(cf.cluster > 1 ? 2 * kMaxRed * 3 * 4 : 0);
    const int64_t stash_floats = (int64_t)n_stash * cf.chunks * cf.vl * cf.ng * cf.block;
    if (off + stash_floats * 4 > dev.max_smem_per_block) { gen_err = "the row does not fit in shared memory for its epilogue"; continue; }
    P.sm_stash = take((int)(stash_floats * 4));
    P.stash_floats = (int32_t)stash_floats;
    P.n_stages = n_stages;
    P.pro_begin = pro_begin; P.pro_end = pro_end;
    memcpy(P.stage, stages, sizeof(stages));
    memset(P.code, 0, sizeof(P.code));
    memcpy(P.code, code.data(), code.size() * 4);
    P.slice_len = cf.slice_len;
    P.chunks = cf.chunks;
    P.split_chunks = cf.family == FAM_POINTWISE;
    P.cluster = cf.cluster;
    P.team_lanes = lanes;
    P.splits = cf.family == FAM_SPLIT ? cf.splits : 0;
    lp.family = cf.family; lp.vl = cf.vl; lp.ng = cf.ng; lp.k = cf.k;
    lp.block = cf.block; lp.smem_bytes = off; lp.code_words = (int)code.size();
    P.family = cf.family;
    lp.items = P.split_chunks ? eff_rows * cf.chunks : (cf.family == FAM_SPLIT ? eff_rows * cf.splits : eff_rows);
    lp.teams_per_cta = teams;
    lp.specialised = 0;
    lp.persistent = persistent ? 1 : 0;
    lp.grid_waves = tune_waves(flags);
    // long rows split over a cluster run few, long-lived threads: there the first stage's loads
    // are issued one tile ahead (elsewhere the extra registers cost more than they bring)
    lp.no_prefetch = cf.family == FAM_SPLIT ? 1 : ((flags & PN_FLAG_PREFETCH) || (cf.family == FAM_CLUSTER && cf.chunks > 1 && !(flags & PN_FLAG_NO_HOIST))) ? 0 : 1;
    int occ = (dev.have_device && !spec) ? instance_occupancy(cf.vl, cf.ng, cf.k, cf.block, off) : 0;
    size_grid(lp, sms, occ);
    return PN_OK;
  }
  err = gen_err;
  return PN_ERR_TOO_LARGE;
}

}  // namespace pn
