// descriptor.cpp -- decode and validate a serialized computational graph
// G = (V, E, tau, sigma) (Definition 3.1): tensor table = sigma (+ dtypes), node table = tau
// and E.  Everything a later stage indexes with is range-checked here.
#include <string.h>

#include <string>

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

}  // namespace pn
