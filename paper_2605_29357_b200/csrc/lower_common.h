// lower_common.h -- pieces shared by the lowerings of the kernel families: the values and
// micro-operations a graph is expanded into, and the accumulator-machine code generator with
// its register allocation.
#pragma once
#include <math.h>
#include <string.h>

#include <algorithm>
#include <map>
#include <string>
#include <vector>

#include "../../include/pn.h"
#include "graph.h"

namespace pn {
namespace lowering {

enum ValKind { VK_E, VK_S, VK_IMM };

struct Val {
  ValKind kind = VK_E;
  int stage = 0;
  int io = -1;          // tile value that is a graph input not loaded yet
  bool bcast = false;   // that input has col_stride 0
  bool streamed = false;// that input has one element per element of the iteration space
  bool invariant = false;// that input is the same for every row (all leading strides 0)
  bool pinned = false;  // loaded once before the row loop into a register of its own
  float imm = 0.f;
  int slot = -1;        // per-row scalar: its shared-memory slot
  bool int_bits = false;// slot holds int32 bits (argmax / argmin)
  bool has_ts = false;  // exp(x - m_tile) of a softmax: travels with the tile scalar
  bool integral = false;// known to hold integer / 0-1 values
  bool boolean = false; // known to hold exactly 0.0f or 1.0f
  bool mask8 = false;   // graph input stored as int8 / bool
  bool uniform = false; // column kernels: the same value in every column of a tile
  int uses = 0;
};

struct MOp {
  int op = OP_END;      // VM opcode
  int stage = 0;
  bool scalar = false;
  int nin = 0;
  int in[3] = {-1, -1, -1};
  int out = -1;
  int aux0 = 0, aux1 = 0;
};

struct Shape4 { int64_t d[4]; };

inline Shape4 align4(const Tensor& t) {
  Shape4 s{{1, 1, 1, 1}};
  for (int i = 0; i < t.rank; ++i) s.d[4 - t.rank + i] = t.dims[i];
  return s;
}

inline bool bcast_into(Shape4& acc, const Shape4& s) {
  for (int i = 0; i < 4; ++i) {
    if (acc.d[i] == s.d[i] || s.d[i] == 1) continue;
    if (acc.d[i] == 1) { acc.d[i] = s.d[i]; continue; }
    return false;
  }
  return true;
}

inline int vm_unary(uint16_t op) {
  switch (op) {
    case N_NEG: return OP_NEG; case N_ABS: return OP_ABS; case N_EXP: return OP_EXP; case N_LOG: return OP_LOG;
    case N_SQRT: return OP_SQRT; case N_RSQRT: return OP_RSQRT; case N_RECIP: return OP_RECIP;
    case N_TANH: return OP_TANH; case N_SIGMOID: return OP_SIGMOID; case N_SILU: return OP_SILU;
    case N_GELU_TANH: return OP_GELU_TANH; case N_GELU_ERF: return OP_GELU_ERF; case N_RELU: return OP_RELU;
    case N_SQUARE: return OP_SQUARE; case N_ERF: return OP_ERF;
  }
  return -1;
}
inline int vm_binary(uint16_t op) {
  switch (op) {
    case N_ADD: return OP_ADD; case N_SUB: return OP_SUB; case N_MUL: return OP_MUL; case N_DIV: return OP_DIV;
    case N_MAX: return OP_MAX; case N_MIN: return OP_MIN; case N_GT: return OP_GT; case N_GE: return OP_GE;
    case N_LT: return OP_LT; case N_LE: return OP_LE; case N_EQ: return OP_EQ; case N_NE: return OP_NE;
  }
  return -1;
}
// opcode computing op(y, x) when acc holds y instead of x
inline int swapped(int op) {
  switch (op) {
    case OP_SUB: return OP_RSUB; case OP_RSUB: return OP_SUB; case OP_DIV: return OP_RDIV; case OP_RDIV: return OP_DIV;
    case OP_GT: return OP_LT; case OP_LT: return OP_GT; case OP_GE: return OP_LE; case OP_LE: return OP_GE;
    default: return op;  // commutative
  }
}

// ---------------------------------------------------------------------------------------
// code generation for one program (tile program of a stage, or a per-row scalar program)
// ---------------------------------------------------------------------------------------
struct Gen {
  std::vector<uint32_t>& code;
  std::vector<Val>& vals;
  const bool scalar;
  const int K;
  const bool multichunk;
  int accv = -1;
  std::vector<int> regv;
  std::vector<char> regraw;
  std::map<int, int>& stash_of;   // value -> stash index (shared over the stages)
  int& n_stash;
  std::string err;

  Gen(std::vector<uint32_t>& c, std::vector<Val>& v, bool sc, int k, bool mc, std::map<int, int>& so, int& ns)
      : code(c), vals(v), scalar(sc), K(k), multichunk(mc), regv(k, -1), regraw(k, 0), stash_of(so), n_stash(ns) {}

  void emit(int op, int a = 0, int b = 0, int c = 0) {
    code.push_back((uint32_t)op | ((uint32_t)a << 8) | ((uint32_t)b << 16) | ((uint32_t)c << 24));
  }
  void emit_f(float f) { uint32_t u; memcpy(&u, &f, 4); code.push_back(u); }
  int find_reg(int v) const { for (int k = 0; k < K; ++k) if (regv[k] == v) return k; return -1; }
  int free_reg() {
    for (int k = 0; k < K; ++k) if (regv[k] < 0) return k;
    for (int k = 0; k < K; ++k) if (vals[regv[k]].uses <= 0 && !vals[regv[k]].pinned) { regv[k] = -1; regraw[k] = 0; return k; }
    err = "expression needs more tile registers than the kernel instance has";
    return -1;
  }
  int n_free() const { int n = 0; for (int k = 0; k < K; ++k) n += regv[k] < 0; return n; }
  void widen_if_raw(int k) { if (regraw[k]) { emit(OP_WIDEN, vals[regv[k]].io, k); regraw[k] = 0; } }
  void drop_dead() {
    for (int k = 0; k < K; ++k) if (regv[k] >= 0 && vals[regv[k]].uses <= 0 && !vals[regv[k]].pinned) { regv[k] = -1; regraw[k] = 0; }
    if (accv >= 0 && vals[accv].uses <= 0) accv = -1;
  }
  bool save_acc() {   // acc is about to be overwritten
    if (accv < 0 || vals[accv].uses <= 0 || find_reg(accv) >= 0) return true;
    if (vals[accv].kind != VK_E) return true;   // scalars live in their slots
    const int k = free_reg();
    if (k < 0) return false;
    emit(OP_ST, k); regv[k] = accv; regraw[k] = 0;
    return true;
  }
  void load_input(int v, int target) {   // target = kAccReg names acc
    const Val& x = vals[v];
    if (x.bcast) emit(OP_LDBC, x.io, target);
    else { emit(OP_LDRAW, x.io, target); emit(OP_WIDEN, x.io, target); }
  }
  bool place_in_acc(int v) {
    if (accv == v) return true;
    if (!save_acc()) return false;
    const Val& x = vals[v];
    if (x.kind == VK_S) { emit(OP_SLD, x.slot); accv = v; return true; }
    if (x.kind == VK_IMM) { err = "constant-only subexpression is not lowered"; return false; }
    const int k = find_reg(v);
    if (k >= 0) { widen_if_raw(k); emit(OP_LD, k); }
    else if (stash_of.count(v)) { emit(OP_FILL, kAccReg, stash_of[v]); if (x.has_ts) emit(OP_FILL_TS, 0, stash_of[v] + 1); }
    else if (x.io >= 0) load_input(v, kAccReg);
    else { err = "internal: tile value has no location"; return false; }
    accv = v;
    return true;
  }
  struct Src { int idx = 0, kind = OPK_REG; float imm = 0.f; };
  bool src_operand(int v, Src& s) {
    const Val& x = vals[v];
    if (x.kind == VK_IMM) { s.kind = OPK_IMM; s.imm = x.imm; return true; }
    if (x.kind == VK_S) { s.kind = OPK_SLOT; s.idx = x.slot; return true; }
    int k = find_reg(v);
    if (k >= 0) { widen_if_raw(k); s.idx = k; return true; }
    k = free_reg();
    if (k < 0) return false;
    if (accv == v) emit(OP_ST, k);
    else if (stash_of.count(v)) emit(OP_FILL, k, stash_of[v]);
    else if (x.io >= 0) load_input(v, k);
    else { err = "internal: tile operand has no location"; return false; }
    regv[k] = v; regraw[k] = 0; s.idx = k;
    return true;
  }
  // after an op consumed `v` from acc: keep a copy if others still need it
  bool keep_if_live(int v) {
    if (vals[v].kind != VK_E || vals[v].uses <= 0 || find_reg(v) >= 0 || stash_of.count(v)) return true;
    const int k = free_reg();
    if (k < 0) return false;
    emit(OP_ST, k); regv[k] = v; regraw[k] = 0;
    return true;
  }
  void result(int r) {
    accv = r;
    if (scalar && r >= 0 && vals[r].kind == VK_S) emit(OP_SST, vals[r].slot);
    drop_dead();
  }
  bool is_tile(int v) const { return vals[v].kind == (scalar ? VK_S : VK_E); }

  bool gen(const MOp& m) {
    switch (m.op) {
      case OP_STOUT: case OP_STOUT_I: {
        if (!place_in_acc(m.in[0])) return false;
        vals[m.in[0]].uses--;
        emit(m.op, m.aux0, m.aux1);
        drop_dead();
        return true;
      }
      case OP_ACCUM: {   // reg[aux1] (op)= acc; acc itself is left as it is
        if (!place_in_acc(m.in[0])) return false;
        vals[m.in[0]].uses--;
        emit(OP_ACCUM, m.aux0, m.aux1);
        drop_dead();
        return true;
      }
      case OP_RED: {
        if (!place_in_acc(m.in[0])) return false;
        vals[m.in[0]].uses--;
        if (m.aux0 == RED_SOFTMAX) {
          if (!keep_if_live(m.in[0])) return false;
          emit(OP_RED, m.aux0, m.aux1);
          result(m.out);
        } else {
          emit(OP_RED, m.aux0, m.aux1);
          drop_dead();
        }
        return true;
      }
      case OP_SCALE_TS: {
        if (!place_in_acc(m.in[0])) return false;
        vals[m.in[0]].uses--;
        if (!keep_if_live(m.in[0])) return false;
        emit(OP_SCALE_TS, m.aux0, m.aux1);
        result(m.out);
        return true;
      }
      case OP_WHERE: case OP_FMA: {
        int x = m.in[0], X = m.in[1], Y = m.in[2];
        // a mask read straight from an int8 / bool input and used only here is tested as bytes
        if (m.op == OP_WHERE && !scalar && vals[x].kind == VK_E && vals[x].io >= 0 && vals[x].mask8 && !vals[x].bcast &&
            vals[x].uses == 1 && accv != x && !stash_of.count(x) && vals[X].kind == VK_E && X != x && Y != x) {
          int k = find_reg(x);
          if (k < 0 || regraw[k]) {
            if (!place_in_acc(X)) return false;
            if (k < 0) {
              k = free_reg();
              if (k < 0) return false;
              emit(OP_LDRAW, vals[x].io, k);
              regv[k] = x; regraw[k] = 1;
            }
            Src sy;
            if (!src_operand(Y, sy)) return false;
            // (the copy that keeps X alive is made while the other operands still count as used: their
            // registers must not be handed out before the instruction that reads them)
            vals[X].uses--;
            if (!keep_if_live(X)) return false;
            vals[x].uses--; vals[Y].uses--;
            emit(OP_WHERE_RAW, k, sy.idx, sy.kind);
            if (sy.kind == OPK_IMM) emit_f(sy.imm);
            result(m.out);
            return true;
          }
        }
        if (m.op == OP_FMA && !is_tile(x) && is_tile(X)) std::swap(x, X);
        if (vals[x].kind == VK_IMM) { err = "where / fma with a constant first operand is not lowered"; return false; }
        if (!place_in_acc(x)) return false;
        Src sx, sy;
        if (!src_operand(X, sx) || !src_operand(Y, sy)) return false;
        vals[x].uses--;
        if (!keep_if_live(x)) return false;
        vals[X].uses--; vals[Y].uses--;
        emit(m.op, sx.idx, sy.idx, sx.kind | (sy.kind << 4));
        if (sx.kind == OPK_IMM) emit_f(sx.imm);
        if (sy.kind == OPK_IMM) emit_f(sy.imm);
        result(m.out);
        return true;
      }
      default: break;
    }
    if (m.nin == 1) {   // unary
      if (!place_in_acc(m.in[0])) return false;
      vals[m.in[0]].uses--;
      if (!keep_if_live(m.in[0])) return false;
      emit(m.op);
      result(m.out);
      return true;
    }
    // binary
    int op = m.op, x = m.in[0], y = m.in[1];
    const bool xt = is_tile(x), yt = is_tile(y);
    if ((!xt && yt) || (xt && yt && accv == y && accv != x)) { std::swap(x, y); op = swapped(op); }
    if (vals[x].kind == VK_IMM) { err = "constant-only subexpression is not lowered"; return false; }
    if (!place_in_acc(x)) return false;
    Src s;
    if (!src_operand(y, s)) return false;
    vals[x].uses--;
    if (!keep_if_live(x)) return false;
    vals[y].uses--;
    emit(op, s.idx, s.kind);
    if (s.kind == OPK_IMM) emit_f(s.imm);
    result(m.out);
    return true;
  }

  // Issue the loads of this stage's inputs before any arithmetic, so that they are all in
  // flight together; the large (streamed) operands first.
  // also_bcast: the one-element loads of last-dim-broadcast operands are issued there too.
  void hoist_loads(const std::vector<MOp>& ops, int stage, bool also_bcast = false) {
    if (scalar) return;
    for (int pass = 0; pass < (also_bcast ? 3 : 2); ++pass)
      for (const MOp& m : ops) {
        if (m.stage != stage || m.scalar) continue;
        for (int i = 0; i < m.nin; ++i) {
          const int v = m.in[i];
          if (v < 0 || vals[v].kind != VK_E || vals[v].io < 0) continue;
          if (vals[v].bcast != (pass == 2)) continue;
          if (pass < 2 && vals[v].streamed != (pass == 0)) continue;
          if (find_reg(v) >= 0 || accv == v || stash_of.count(v)) continue;
          if (n_free() <= 1) return;
          const int k = free_reg();
          if (pass == 2) { emit(OP_LDBC, vals[v].io, k); regv[k] = v; regraw[k] = 0; }
          else { emit(OP_LDRAW, vals[v].io, k); regv[k] = v; regraw[k] = 1; }
        }
      }
  }

  // Before the row loop: load (and widen) the operands that are the same for every row, each
  // into a register that keeps it for the whole kernel.  Leaves `reserve` registers free.
  void pin_invariants(const std::vector<MOp>& ops, int reserve) {
    for (const MOp& m : ops) {
      if (m.scalar) continue;
      for (int i = 0; i < m.nin; ++i) {
        const int v = m.in[i];
        if (v < 0 || vals[v].kind != VK_E || vals[v].io < 0 || !vals[v].invariant || vals[v].pinned) continue;
        if (n_free() <= reserve) return;
        const int k = free_reg();
        load_input(v, k);
        regv[k] = v; regraw[k] = 0; vals[v].pinned = true;
      }
    }
  }

  // End of a stage: tile values still needed later stay in registers (one chunk per thread)
  // or are parked in shared memory (several chunks per thread).
  bool end_stage() {
    if (scalar) { accv = -1; return true; }
    if (!multichunk) return save_acc();
    auto park = [&](int v, int k) {
      stash_of[v] = n_stash; emit(OP_SPILL, k, n_stash); n_stash++;
      if (vals[v].has_ts) { emit(OP_SPILL_TS, 0, n_stash); n_stash++; }
    };
    if (accv >= 0 && vals[accv].uses > 0 && vals[accv].kind == VK_E && find_reg(accv) < 0 && !stash_of.count(accv))
      park(accv, kAccReg);
    for (int k = 0; k < K; ++k) {
      const int v = regv[k];
      if (v >= 0 && vals[v].pinned) continue;
      if (v >= 0 && vals[v].uses > 0 && !stash_of.count(v)) { widen_if_raw(k); park(v, k); }
      regv[k] = -1; regraw[k] = 0;
    }
    accv = -1;
    return true;
  }
};

// ---------------------------------------------------------------------------------------
// expansion of graph nodes into micro-operations: the part every family shares
// ---------------------------------------------------------------------------------------
struct Expander {
  std::vector<Val> vals;
  std::vector<MOp> ops;
  int n_slots = 0;

  int new_val(ValKind k, int stage) { Val v; v.kind = k; v.stage = stage; vals.push_back(v); return (int)vals.size() - 1; }
  int new_slot(int n) { const int s = n_slots; n_slots += n; return s; }
  void add_op(int op, int stage, bool scalar, std::initializer_list<int> in, int out, int a0 = 0, int a1 = 0) {
    MOp m; m.op = op; m.stage = stage; m.scalar = scalar; m.nin = 0;
    for (int v : in) m.in[m.nin++] = v;
    m.out = out; m.aux0 = a0; m.aux1 = a1; ops.push_back(m);
  }
  // a pointwise micro-operation: a tile operation in the latest stage of its operands, or a
  // per-row scalar operation when no operand is a tile value
  int pointwise(int vmop, std::initializer_list<int> in, bool integral) {
    bool any_e = false, uni = true; int stage = 0;
    for (int v : in) { any_e |= vals[v].kind == VK_E; stage = std::max(stage, vals[v].stage); uni = uni && (vals[v].uniform || vals[v].kind == VK_IMM); }
    const bool sc = !any_e;
    const int r = new_val(sc ? VK_S : VK_E, stage);
    vals[r].integral = integral;
    vals[r].uniform = uni;
    if (sc) vals[r].slot = new_slot(1);
    add_op(vmop, sc ? stage - 1 : stage, sc, in, r);
    return r;
  }
  int slot_val(int slot, int stage, bool int_bits) { const int v = new_val(VK_S, stage); vals[v].slot = slot; vals[v].int_bits = int_bits; return v; }
  int imm_val(double x) { const int v = new_val(VK_IMM, 0); vals[v].imm = (float)x; return v; }

  // unary, cast, binary, where, fma, clamp, and cat of one operand (the identity).  Returns 1 when
  // the node was one of these (res[0] is its value), 0 when it is another kind of node, or a
  // negative pn_status with `err` set.
  int expand_pointwise(const Graph& g, const Node& n, int (&in)[4], int (&res)[3], std::string& err, const std::string& where) {
    const Tensor& T0 = g.tensors[n.out[0]];
    if (vm_unary(n.op) >= 0) {
      if (vals[in[0]].int_bits) in[0] = pointwise(OP_I2F, {in[0]}, true);
      res[0] = pointwise(vm_unary(n.op), {in[0]}, false);
    } else if (n.op == N_CAST) {
      const bool src_int = vals[in[0]].integral;
      if (vals[in[0]].int_bits) {   // an index held as int32 bits
        res[0] = dtype_is_float(T0.dtype) ? pointwise(OP_I2F, {in[0]}, true) : in[0];
        if (T0.dtype == kBool) res[0] = pointwise(OP_NEZ, {pointwise(OP_I2F, {in[0]}, true)}, true);
      }
      else if (dtype_is_float(T0.dtype)) res[0] = in[0];
      else if (T0.dtype == kBool) {
        res[0] = (vals[in[0]].boolean || (src_int && g.tensors[n.in[0]].dtype == kBool)) ? in[0] : pointwise(OP_NEZ, {in[0]}, true);
        vals[res[0]].boolean = true;
      }
      else res[0] = src_int ? in[0] : pointwise(OP_TRUNC, {in[0]}, true);
    } else if (vm_binary(n.op) >= 0) {
      for (int k = 0; k < 2; ++k) if (vals[in[k]].int_bits) in[k] = pointwise(OP_I2F, {in[k]}, true);
      res[0] = pointwise(vm_binary(n.op), {in[0], in[1]}, n.op >= N_GT);
      vals[res[0]].boolean = n.op >= N_GT;
    } else if (n.op == N_WHERE || n.op == N_FMA) {
      for (int k = 0; k < 3; ++k) if (vals[in[k]].int_bits) in[k] = pointwise(OP_I2F, {in[k]}, true);
      res[0] = pointwise(n.op == N_WHERE ? OP_WHERE : OP_FMA, {in[0], in[1], in[2]}, false);
    } else if (n.op == N_CLAMP) {
      for (int k = 0; k < 3; ++k) if (vals[in[k]].int_bits) in[k] = pointwise(OP_I2F, {in[k]}, true);
      const int lo = pointwise(OP_MAX, {in[0], in[1]}, false);
      res[0] = pointwise(OP_MIN, {lo, in[2]}, false);
    } else if (n.op == N_CONTIGUOUS) {   // on a computed value: the identity
      if (g.tensors[n.in[0]].numel() != T0.numel() || g.tensors[n.in[0]].dtype != T0.dtype) { err = where + "contiguous keeps shape and dtype"; return PN_ERR_SHAPE; }
      if (vals[in[0]].kind == VK_IMM) { err = where + "contiguous of a constant"; return PN_ERR_UNSUPPORTED_OP; }
      res[0] = in[0];
    } else if (n.op == N_CAT) {
      if (n.n_in != 1) { err = where + "cat of several operands is not lowered (one operand is the identity)"; return PN_ERR_UNSUPPORTED_OP; }
      if (g.tensors[n.in[0]].numel() != T0.numel()) { err = where + "cat of one operand keeps its shape"; return PN_ERR_SHAPE; }
      if (vals[in[0]].kind == VK_IMM) { err = where + "cat of a constant"; return PN_ERR_UNSUPPORTED_OP; }
      res[0] = in[0];
    } else {
      return 0;
    }
    return 1;
  }

  // After a node's values are known: a declared 16-bit float result is rounded for its
  // consumers, and results that are graph outputs are stored.
  int finish_node(const Graph& g, const Node& n, const int (&res)[3], const std::vector<int>& n_consumers,
                  const std::vector<int>& io_of_tensor, std::vector<int>& tval, int max_stages, std::string& err, const std::string& where) {
    for (int k = 0; k < n.n_out; ++k) {
      const int t = n.out[k];
      const Tensor& T = g.tensors[t];
      int v = res[k];
      if (v < 0) { err = where + "internal: missing result"; return PN_ERR_UNSUPPORTED_OP; }
      if (vals[v].stage >= max_stages) { err = where + "more reduction-dependent stages than the kernel takes"; return PN_ERR_TOO_LARGE; }
      // a declared 16-bit float intermediate is rounded for its consumers
      if ((T.dtype == kBF16 || T.dtype == kF16) && n_consumers[t] > 0 && !vals[v].integral && vals[v].kind != VK_IMM)
        v = pointwise(T.dtype == kBF16 ? OP_RND_BF16 : OP_RND_F16, {v}, false);
      tval[t] = v;
      if (T.role & 2) {
        if (vals[v].kind == VK_IMM) { err = where + "constant output"; return PN_ERR_UNSUPPORTED_OP; }
        if (vals[v].int_bits && dtype_is_float(T.dtype)) v = pointwise(OP_I2F, {v}, true);
        const bool sc = vals[v].kind == VK_S;
        if (vals[v].int_bits && T.dtype != kI64 && T.dtype != kI32) { err = where + "index results must be stored as i32 or i64"; return PN_ERR_UNSUPPORTED_OP; }
        const int zero_one = (!sc && vals[v].boolean && (T.dtype == kI8 || T.dtype == kBool)) ? 1 : 0;
        add_op(vals[v].int_bits ? OP_STOUT_I : OP_STOUT, sc ? vals[v].stage - 1 : vals[v].stage, sc, {v}, -1, io_of_tensor[t], zero_one);
      }
    }
    return PN_OK;
  }
};

}  // namespace lowering
}  // namespace pn
