// descriptor.cpp -- decode and validate a serialized computational graph
// G = (V, E, tau, sigma) (Definition 3.1): tensor table = sigma (+ dtypes), node table = tau
// and E.  Everything a later stage indexes with is range-checked here.
#include <string.h>

#include <string>
#include <vector>

#include "../../include/pn.h"
#include "graph.h"

namespace pn {

namespace {

struct Arity { int lo, hi, outs_lo, outs_hi; };

bool arity_of(uint16_t op, Arity& a) {
  if (op >= N_NEG && op <= N_ERF) { a = {1, 1, 1, 1}; return true; }
  if (op >= N_ADD && op <= N_NE) { a = {2, 2, 1, 1}; return true; }
  if (op == N_WHERE || op == N_CLAMP || op == N_FMA) { a = {3, 3, 1, 1}; return true; }
  if (op >= N_SUM && op <= N_LOGSUMEXP) { a = {1, 1, 1, 1}; return true; }
  if (op >= N_SUM_DIM && op <= N_AMIN_DIM) { a = {1, 1, 1, 1}; return true; }
  if (op == N_CAT) { a = {1, 4, 1, 1}; return true; }
  if (op == N_SOFTMAX || op == N_LOG_SOFTMAX) { a = {1, 1, 1, 1}; return true; }
  if (op == N_LAYER_NORM) { a = {1, 3, 1, 3}; return true; }
  if (op == N_RMS_NORM) { a = {1, 2, 1, 1}; return true; }
  if ((op >= N_ROLL && op <= N_VIEW) || op == N_CONTIGUOUS) { a = {1, 1, 1, 1}; return true; }
  return false;
}

template <class T>
T rd(const unsigned char* p) { T v; memcpy(&v, p, sizeof(T)); return v; }

}  // namespace

int parse_descriptor(const void* desc, size_t bytes, Graph& g, std::string& err) {
  const unsigned char* p = static_cast<const unsigned char*>(desc);
  if (bytes < 16) { err = "descriptor shorter than its 16-byte header"; return PN_ERR_BAD_DESCRIPTOR; }
  const uint32_t magic = rd<uint32_t>(p);
  const uint16_t version = rd<uint16_t>(p + 4);
  const uint32_t n_t = rd<uint32_t>(p + 8), n_n = rd<uint32_t>(p + 12);
  if (magic != 0x31474E50u) { err = "bad magic"; return PN_ERR_BAD_DESCRIPTOR; }
  if (version != 1) { err = "unsupported descriptor version"; return PN_ERR_BAD_DESCRIPTOR; }
  if (n_t == 0 || n_t > 4096 || n_n > 4096) { err = "tensor / node count out of range"; return PN_ERR_BAD_DESCRIPTOR; }
  if (bytes != 16 + 40ull * n_t + 64ull * n_n) { err = "descriptor length does not match its tables"; return PN_ERR_BAD_DESCRIPTOR; }

  g.tensors.assign(n_t, Tensor());
  g.nodes.assign(n_n, Node());
  g.inputs.clear();
  g.outputs.clear();
  const unsigned char* q = p + 16;
  for (uint32_t i = 0; i < n_t; ++i, q += 40) {
    Tensor& t = g.tensors[i];
    const std::string where = "tensor " + std::to_string(i) + ": ";
    t.dtype = q[0]; t.role = q[1]; t.rank = q[2];
    if (t.dtype > kI64) { err = where + "unknown dtype"; return PN_ERR_BAD_DESCRIPTOR; }
    if (t.rank > 4) { err = where + "rank above 4"; return PN_ERR_BAD_DESCRIPTOR; }
    if (t.role > 3) { err = where + "bad role bits"; return PN_ERR_BAD_DESCRIPTOR; }
    for (int d = 0; d < 4; ++d) t.dims[d] = 1;
    for (int d = 0; d < t.rank; ++d) {
      const int64_t v = rd<int64_t>(q + 8 + 8 * d);
      if (v < 0 || v > (int64_t(1) << 40)) { err = where + "bad dimension"; return PN_ERR_BAD_DESCRIPTOR; }
      t.dims[d] = v;
    }
    if ((t.role & 1) && (t.role & 2)) { err = where + "a graph input cannot also be a graph output"; return PN_ERR_UNSUPPORTED_OP; }
    if (t.role & 1) g.inputs.push_back((int)i);
    if (t.role & 2) g.outputs.push_back((int)i);
  }
  if (g.outputs.empty()) { err = "graph has no output"; return PN_ERR_BAD_DESCRIPTOR; }

  for (uint32_t i = 0; i < n_n; ++i, q += 64) {
    Node& n = g.nodes[i];
    const std::string where = "node " + std::to_string(i) + ": ";
    n.op = rd<uint16_t>(q); n.n_in = q[2]; n.n_out = q[3];
    Arity a;
    if (!arity_of(n.op, a)) { err = where + "unknown opcode " + std::to_string(n.op); return PN_ERR_UNSUPPORTED_OP; }
    if (n.n_in < a.lo || n.n_in > a.hi || n.n_out < a.outs_lo || n.n_out > a.outs_hi) {
      err = where + "operand count does not fit its opcode"; return PN_ERR_BAD_DESCRIPTOR;
    }
    for (int k = 0; k < 4; ++k) n.in[k] = rd<uint32_t>(q + 4 + 4 * k);
    for (int k = 0; k < 3; ++k) n.out[k] = rd<uint32_t>(q + 20 + 4 * k);
    n.imm[0] = rd<double>(q + 32); n.imm[1] = rd<double>(q + 40);
    n.attr[0] = rd<int64_t>(q + 48); n.attr[1] = rd<int64_t>(q + 56);
    for (int k = 0; k < n.n_in; ++k) {
      const uint32_t s = n.in[k];
      if (s == kImm0 || s == kImm1) continue;
      if (s >= n_t) { err = where + "operand id out of range"; return PN_ERR_BAD_DESCRIPTOR; }
      const Tensor& t = g.tensors[s];
      if (!(t.role & 1) && t.producer < 0) {
        err = where + "reads tensor " + std::to_string(s) + " before it is produced (nodes must be in topological order)";
        return PN_ERR_BAD_DESCRIPTOR;
      }
    }
    for (int k = 0; k < n.n_out; ++k) {
      const uint32_t o = n.out[k];
      if (o >= n_t) { err = where + "output id out of range"; return PN_ERR_BAD_DESCRIPTOR; }
      Tensor& t = g.tensors[o];
      if (t.role & 1) { err = where + "writes a graph input"; return PN_ERR_BAD_DESCRIPTOR; }
      if (t.producer >= 0) { err = "tensor " + std::to_string(o) + " is produced twice"; return PN_ERR_BAD_DESCRIPTOR; }
      t.producer = (int)i;
    }
  }
  for (int o : g.outputs)
    if (g.tensors[o].producer < 0) { err = "output tensor " + std::to_string(o) + " is never produced"; return PN_ERR_BAD_DESCRIPTOR; }
  return PN_OK;
}

int expand_concatenations(Graph& g, std::string& err) {
  bool any = false;
  for (const Node& n : g.nodes) any = any || (n.op == N_CAT && n.n_in > 1);
  if (!any) return PN_OK;
  std::vector<Node> nodes;
  for (size_t ni = 0; ni < g.nodes.size(); ++ni) {
    const Node n = g.nodes[ni];
    if (!(n.op == N_CAT && n.n_in > 1)) { nodes.push_back(n); continue; }
    const std::string where = "node " + std::to_string(ni) + ": ";
    const int y = (int)n.out[0];
    const Tensor Y = g.tensors[y];
    const int64_t dim = n.attr[0];
    if (dim < 0 || dim >= Y.rank) { err = where + "cat dimension outside the tensor"; return PN_ERR_SHAPE; }
    int64_t pd[4] = {1, 1, 1, 1};
    for (int i = 0; i < Y.rank; ++i) pd[4 - Y.rank + i] = Y.dims[i];
    int64_t at = 0;
    for (int k = 0; k < n.n_in; ++k) {
      if (n.in[k] >= g.tensors.size()) { err = where + "cat of a constant"; return PN_ERR_UNSUPPORTED_OP; }
      const Tensor X = g.tensors[n.in[k]];
      if (X.rank != Y.rank || X.dtype != Y.dtype) { err = where + "the operands of a cat have the rank and dtype of its result"; return X.rank != Y.rank ? PN_ERR_SHAPE : PN_ERR_UNSUPPORTED_OP; }
      for (int i = 0; i < Y.rank; ++i)
        if (i != dim && X.dims[i] != Y.dims[i]) { err = where + "the operands of a cat differ from its result in the cat dimension only"; return PN_ERR_SHAPE; }
      Tensor part = X;
      part.role = 0; part.producer = (int)nodes.size();
      part.assembled = false;
      part.embed_parent = y;
      for (int i = 0; i < 4; ++i) { part.embed_dims[i] = pd[i]; part.embed_off[i] = 0; }
      part.embed_off[4 - Y.rank + dim] = at;
      at += X.dims[dim];
      g.tensors.push_back(part);
      Node c;
      c.op = N_CONTIGUOUS; c.n_in = 1; c.n_out = 1;
      c.in[0] = n.in[k]; c.out[0] = (uint32_t)g.tensors.size() - 1;
      nodes.push_back(c);
    }
    if (at != Y.dims[dim]) { err = where + "the operands of a cat do not add up to its result along the cat dimension"; return PN_ERR_SHAPE; }
    g.tensors[y].assembled = true;
    g.tensors[y].producer = -1;
  }
  g.nodes.swap(nodes);
  for (size_t ni = 0; ni < g.nodes.size(); ++ni)   // producers by the new numbering
    for (int k = 0; k < g.nodes[ni].n_out; ++k) g.tensors[g.nodes[ni].out[k]].producer = (int)ni;
  return PN_OK;
}

// Nodes whose results reach no graph output take no part in f_G: they are dropped before any
// lowering (fused, they would cost nothing anyway; as a launch of their own they would have
// nothing to store).  A part of a cat result counts as used when the result is.
void prune_dead_nodes(Graph& g) {
  std::vector<char> used(g.tensors.size(), 0);
  for (size_t t = 0; t < g.tensors.size(); ++t) used[t] = (g.tensors[t].role & 2) != 0;
  std::vector<char> live(g.nodes.size(), 0);
  for (int pass = 0; pass < 2; ++pass)   // (a second pass: a cat result read by a node listed before its parts' stores)
    for (int ni = (int)g.nodes.size() - 1; ni >= 0; --ni) {
      const Node& n = g.nodes[ni];
      bool need = false;
      for (int k = 0; k < n.n_out; ++k) {
        const Tensor& T = g.tensors[n.out[k]];
        need = need || used[n.out[k]] || (T.embed_parent >= 0 && used[T.embed_parent]);
      }
      if (!need) continue;
      live[ni] = 1;
      for (int k = 0; k < n.n_in; ++k) if (n.in[k] < g.tensors.size()) used[n.in[k]] = 1;
    }
  bool all = true;
  for (char c : live) all = all && c;
  if (all) return;
  std::vector<Node> nodes;
  for (size_t ni = 0; ni < g.nodes.size(); ++ni) if (live[ni]) nodes.push_back(g.nodes[ni]);
  g.nodes.swap(nodes);
  // the tensors only dead nodes touched leave the table too (the lowering looks at every tensor)
  std::vector<char> keep(g.tensors.size(), 0);
  for (size_t t = 0; t < g.tensors.size(); ++t) keep[t] = g.tensors[t].role != 0;
  for (const Node& n : g.nodes) {
    for (int k = 0; k < n.n_in; ++k) if (n.in[k] < g.tensors.size()) keep[n.in[k]] = 1;
    for (int k = 0; k < n.n_out; ++k) {
      keep[n.out[k]] = 1;
      if (g.tensors[n.out[k]].embed_parent >= 0) keep[g.tensors[n.out[k]].embed_parent] = 1;
    }
  }
  std::vector<int> new_id(g.tensors.size(), -1);
  std::vector<Tensor> tensors;
  for (size_t t = 0; t < g.tensors.size(); ++t)
    if (keep[t]) { new_id[t] = (int)tensors.size(); tensors.push_back(g.tensors[t]); }
  for (Tensor& T : tensors) { T.producer = -1; if (T.embed_parent >= 0) T.embed_parent = new_id[T.embed_parent]; }
  g.tensors.swap(tensors);
  for (size_t ni = 0; ni < g.nodes.size(); ++ni) {
    Node& n = g.nodes[ni];
    for (int k = 0; k < n.n_in; ++k) if (n.in[k] < new_id.size()) n.in[k] = (uint32_t)new_id[n.in[k]];
    for (int k = 0; k < n.n_out; ++k) { n.out[k] = (uint32_t)new_id[n.out[k]]; g.tensors[n.out[k]].producer = (int)ni; }
  }
  for (int& t : g.inputs) t = new_id[t];
  for (int& t : g.outputs) t = new_id[t];
}

}  // namespace pn
