// graph.h -- host-side representation of a parsed descriptor, and the lowering entry points.
#pragma once
#include <stddef.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "plan.h"

namespace pn {

// opcodes of descriptor format version 1
enum NodeOp : uint16_t {
  N_NEG = 1, N_ABS, N_EXP, N_LOG, N_SQRT, N_RSQRT, N_RECIP, N_TANH, N_SIGMOID, N_SILU,
  N_GELU_TANH, N_GELU_ERF, N_RELU, N_CAST, N_SQUARE, N_ERF,
  N_ADD = 32, N_SUB, N_MUL, N_DIV, N_MAX, N_MIN, N_GT, N_GE, N_LT, N_LE, N_EQ, N_NE,
  N_WHERE = 64, N_CLAMP, N_FMA,
  N_SUM = 96, N_MEAN, N_VAR, N_AMAX, N_AMIN, N_ARGMAX, N_ARGMIN, N_LOGSUMEXP,
  N_SUM_DIM = 104, N_MEAN_DIM, N_AMAX_DIM, N_AMIN_DIM,   // over one leading dimension, attr[0] = dim
  N_SOFTMAX = 128, N_LOG_SOFTMAX, N_LAYER_NORM, N_RMS_NORM,
  N_ROLL = 160, N_SLICE, N_VIEW,   // index operators on leading dimensions
  N_CAT = 163,                     // concatenation along attr[0]
  N_CONTIGUOUS = 164               // the identity on values (dense layout is what every tensor has)
};

constexpr uint32_t kImm0 = 0xFFFFFFFFu, kImm1 = 0xFFFFFFFEu;

struct Tensor {
  uint8_t dtype = 0;
  uint8_t role = 0;        // bit0 input, bit1 output
  int rank = 0;
  int64_t dims[4] = {1, 1, 1, 1};
  int producer = -1;       // node index, -1 for graph inputs
  // A concatenation of several operands is not computed: each operand is stored straight into its
  // block of the result.  `assembled`: this tensor is such a result (no node of its own produces it;
  // it is complete once its parts are stored).  `embed_parent` >= 0: this tensor is such a part: it
  // lives inside tensor embed_parent, whose dims (aligned to 4) are embed_dims, at embed_off.
  bool assembled = false;
  int embed_parent = -1;
  int64_t embed_dims[4] = {1, 1, 1, 1};
  int64_t embed_off[4] = {0, 0, 0, 0};
  int64_t numel() const { int64_t n = 1; for (int i = 0; i < rank; ++i) n *= dims[i]; return n; }
};

struct Node {
  uint16_t op = 0;
  int n_in = 0, n_out = 0;
  uint32_t in[4] = {0, 0, 0, 0};
  uint32_t out[3] = {0, 0, 0};
  double imm[2] = {0, 0};
  int64_t attr[2] = {0, 0};
};

struct Graph {
  std::vector<Tensor> tensors;
  std::vector<Node> nodes;
  std::vector<int> inputs, outputs;   // tensor ids in pointer-array order
};

inline int dtype_bytes(int dt) {
  switch (dt) { case kF32: case kI32: return 4; case kF16: case kBF16: return 2; case kI64: return 8; default: return 1; }
}
inline bool dtype_is_float(int dt) { return dt == kF32 || dt == kF16 || dt == kBF16; }
inline bool is_reduction(uint16_t op) { return op >= N_SUM && op <= N_LOGSUMEXP; }
inline bool is_dim_reduction(uint16_t op) { return op >= N_SUM_DIM && op <= N_AMIN_DIM; }
inline bool is_composite(uint16_t op) { return op >= N_SOFTMAX && op <= N_RMS_NORM; }
inline bool is_index_op(uint16_t op) { return op >= N_ROLL && op <= N_VIEW; }

// Returns a pn_status value (see pn.h).
int parse_descriptor(const void* desc, size_t bytes, Graph& g, std::string& err);

// Replaces every cat of several operands by one `contiguous` node per operand whose result is
// embedded in the cat's output (see Tensor::embed_parent).  Returns a pn_status value.
int expand_concatenations(Graph& g, std::string& err);

// Drops the nodes whose results reach no graph output (after expand_concatenations).
void prune_dead_nodes(Graph& g);

struct DeviceModel {      // what the lowering needs to know about the GPU
  int sm_count = 148;
  int max_smem_per_block = 227 * 1024;
  bool have_device = false;   // occupancy queries allowed
  bool specialise = false;    // lower for a generated kernel (many tile registers, loop-invariant
                              // operand loads hoisted, larger tiles) rather than for the interpreter
};

// Lower a whole graph into one fused launch.  Returns a pn_status value.
int lower_graph(const Graph& g, unsigned flags, const DeviceModel& dev, LaunchPlan& out, std::string& err);

// The same for a graph whose reductions run over a leading dimension (lower_col.cpp).
int lower_column_graph(const Graph& g, unsigned flags, const DeviceModel& dev, LaunchPlan& out, std::string& err);

// Grid size of a planned launch given the SM count and its kernel's resident CTAs per SM.
void size_grid(LaunchPlan& lp, int sms, int occ);
int tune_waves(unsigned flags);   // the PN_TUNE_WAVES field of the create flags as LaunchPlan::grid_waves

}  // namespace pn
