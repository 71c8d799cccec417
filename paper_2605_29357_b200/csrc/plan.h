// plan.h -- what the host lowering hands to the kernels: a tile bytecode program, the
// addressing of every graph input / output, and the launch shape.  Plain structs only;
// included by host (.cpp) and device (.cu) code.
#pragma once
#ifndef __CUDACC_RTC__
#include <stdint.h>
#else   // run-time compilation has no standard headers: the fixed-width types by hand
typedef signed char int8_t;
typedef unsigned char uint8_t;
typedef short int16_t;
typedef unsigned short uint16_t;
typedef int int32_t;
typedef unsigned int uint32_t;
typedef long long int64_t;
typedef unsigned long long uint64_t;
typedef unsigned long size_t;
#endif

namespace pn {

constexpr int kMaxIo = 12;      // graph inputs + outputs of one kernel
constexpr int kMaxCode = 224;   // 32-bit bytecode words of one kernel
constexpr int kMaxStages = 4;   // reduction-separated stages
constexpr int kMaxRed = 4;      // reductions accumulated in one stage
constexpr int kMaxSlots = 48;   // per-row scalar slots
constexpr int kMaxStash = 6;    // tile values parked in shared memory across stages
constexpr int kAccReg = 31;     // register operand id that names the accumulator tile
constexpr int kSpecRegs = 12;   // tile registers of a generated kernel (only live ones cost anything)

// Storage types (same numbering as the descriptor).
enum DType : uint8_t { kF32 = 0, kF16 = 1, kBF16 = 2, kI8 = 3, kBool = 4, kI32 = 5, kI64 = 6 };
// store-only pseudo type: an int8 / bool tensor written from values known to be 0.0f or 1.0f
constexpr int kStore01 = 16;

// Tile bytecode.  One instruction acts on the whole register tile of a thread.  The
// machine has an accumulator tile `acc`, K tile registers, a per-tile scalar `ts`, and
// reads per-row scalars from shared-memory slots.  Word layout: op | a<<8 | b<<16 | c<<24;
// an immediate operand occupies the following word (fp32 bits).
enum Op : uint8_t {
  OP_END = 0,
  // memory
  OP_LDRAW,   // a = io, b = reg (kAccReg = acc): issue the loads of a tile, storage bits as they are
  OP_WIDEN,   // a = io (for its dtype), b = reg: storage bits -> fp32 in place
  OP_LDBC,    // a = io, b = reg: last-dim-broadcast operand, one element splat over the tile
  OP_LD,      // acc = reg[a]
  OP_ST,      // reg[a] = acc
  OP_STOUT,   // a = io: narrow acc and store it; b = 1: the values are known to be 0 or 1
  // unary on acc
  OP_NEG, OP_ABS, OP_EXP, OP_LOG, OP_SQRT, OP_RSQRT, OP_RECIP, OP_TANH, OP_SIGMOID, OP_SILU,
  OP_GELU_TANH, OP_GELU_ERF, OP_RELU, OP_SQUARE, OP_ERF,
  OP_RND_BF16, OP_RND_F16,  // round to a narrow float and back (a declared narrow intermediate)
  OP_TRUNC,                 // float -> integer value, toward zero
  OP_NEZ,                   // x != 0 -> 1 / 0
  OP_I2F,                   // value holding int32 bits -> float (scalar programs)
  // binary: acc = acc (op) src, src = operand(a, kind b)
  OP_ADD, OP_SUB, OP_RSUB, OP_MUL, OP_DIV, OP_RDIV, OP_MAX, OP_MIN,
  OP_GT, OP_GE, OP_LT, OP_LE, OP_EQ, OP_NE,
  OP_LSEFIN,  // acc = isinf(acc) ? acc : acc + log(src)
  // ternary: X = operand(a, kind c&15), Y = operand(b, kind c>>4)
  OP_WHERE,   // acc = acc != 0 ? X : Y
  OP_FMA,     // acc = acc * X + Y
  OP_WHERE_RAW, // acc = C != 0 ? acc : Y; C = reg a holding the unwidened bytes of an int8 / bool
              // tensor, Y = operand(b, kind c&15)
  // reductions over the tile into the thread's partial state
  OP_RED,      // a = RedKind, b = reduction index within the stage
  OP_SCALE_TS, // acc *= exp(ts - slot[a]) * slot[b]   (softmax epilogue)
  // parking tile values in shared memory across stages (rows of several chunks per thread)
  OP_SPILL, OP_FILL,        // a = reg (kAccReg = acc), b = stash index
  OP_SPILL_TS, OP_FILL_TS,  // b = stash index
  // scalar programs only
  OP_SLD,     // acc = slot[a]
  OP_SST,     // slot[a] = acc
  OP_STOUT_I, // a = io: store the int32 bits held in acc as an integer (argmax / argmin)
  // column kernels (reductions over a leading dimension)
  OP_ACCUM,   // a = RedKind (sum / max / min), b = reg: reg = reg (op) acc, element by element;
              // a | 0x80: acc holds one value in all its elements, only element 0 is accumulated
  OP_COUNT_
};

enum OperandKind : uint8_t { OPK_REG = 0, OPK_IMM = 1, OPK_SLOT = 2 };

// Reductions.  Each keeps a 3-float partial (a, b, c) per thread and combines associatively.
enum RedKind : uint8_t {
  RED_SUM = 0,     // a = sum
  RED_MAX,         // a = max                     (NaN wins)
  RED_MIN,         // a = min
  RED_ARGMAX,      // a = max, b = int bits of its lowest column
  RED_ARGMIN,
  RED_LSE,         // a = running max M, b = sum of exp(x - M)
  RED_SOFTMAX,     // as RED_LSE; also leaves exp(x - m_tile) in acc and m_tile in ts
  RED_MEANVAR      // a = count, b = mean, c = sum of squared deviations
};

enum Family : int32_t { FAM_POINTWISE = 0, FAM_WARP = 1, FAM_BLOCK = 2, FAM_CLUSTER = 3, FAM_COLUMN = 4, FAM_SPLIT = 5 };

struct IoDesc {
  void* base;              // device pointer; filled in per run
  int64_t lead_stride[3];  // elements per step of each collapsed leading dim; 0 = broadcast
  int32_t col_stride;      // 1, or 0 when the last dim is broadcast
  uint8_t dtype;
  uint8_t is_row_scalar;   // per-row result tensor (one element per row)
  uint8_t mapped;          // an input read through roll / slice / view: the row index is split by
                           // map_dim (row-major) into coordinates c_d, and the row starts at
                           // sum_d ((c_d + map_add[d]) mod map_mod[d]) * lead_stride[d]  (mod 0 = none)
  uint8_t pad[1];
  int32_t map_dim[3];
  int32_t map_add[3];
  int32_t map_mod[3];
  int32_t col_add, col_mod;// an input rolled along the last dimension: column c is read at (c + col_add) mod col_mod
                           // (col_mod 0 = none; a slice of the last dimension is an offset of the base instead)
  int32_t pad2;
  int64_t red_stride;      // column kernels: elements per step of the reduced dimension; 0 = broadcast
  int64_t numel;           // elements of the tensor behind this entry (checked accessors)
};

struct RedDesc {
  uint8_t kind;
  uint8_t slot;   // first of the 3 slots receiving the combined (a, b, c)
  uint8_t uniform;// column kernels: the reduced value is the same in every column of a tile (it comes
                  // from operands broadcast over the columns): one element is accumulated, then copied
};

struct StageDesc {
  uint16_t elem_begin, elem_end;   // tile program [begin, end) in code[]
  uint16_t scal_begin, scal_end;   // per-row scalar program run after the stage's combine
  uint8_t n_red;
  uint8_t pad[3];
  RedDesc red[kMaxRed];
};

struct KernelParams {
  IoDesc io[kMaxIo];
  int32_t n_io;
  int32_t n_stages;
  int32_t family;          // Family
  int32_t pad0;
  uint32_t lead_dim[3];    // collapsed leading dims of the iteration space (unused = 1)
  int64_t rows;            // product of the leading dims
  int32_t row_len;         // N
  int32_t slice_len;       // columns one CTA covers (N unless a cluster splits the row)
  int32_t chunks;          // chunks per slice: ceil(slice_len / (team_threads * VL * NG))
  int32_t split_chunks;    // pointwise graphs: every (row, chunk) is its own work item
  int32_t cluster;         // CTAs per cluster (1 unless FAM_CLUSTER)
  int32_t stash_floats;    // floats of parked tile values per CTA
  // column kernels: the iteration space is [rows, red_len, row_len], reduced over the middle
  // dimension.  A CTA is col_tx threads along the columns by blockDim.x / col_tx along the reduced
  // dimension; stage 0 runs per (row, step, column tile) and ends in OP_ACCUM into tile registers
  // 0 .. n_red-1, stage 1 runs once per (row, column tile) on the combined registers.
  int32_t red_len;
  int32_t col_tx;
  int64_t item_begin, item_end;   // item_end > 0: this launch does the work items [item_begin, item_end) only
                                  // (rows, or (row, chunk) / (row, column tile) pairs in launch order)
  uint32_t* status;        // checked accessors (PN_FLAG_BOUNDS): bit q is set when an access to io entry q
                           // fell outside its tensor; null when checking is off
  int32_t team_lanes;      // warp-per-row kernels: lanes per row (32, or 16 / 8 when short rows share a warp)
  int32_t splits;          // FAM_SPLIT: independent thread blocks per row, each reducing slice_len columns; their
                           // partials meet in split_part and the block that arrives last at a row combines them
  int32_t pad1[3];
  float* split_part;       // FAM_SPLIT: [rows][splits][reductions of stage 0][3] floats, device memory of the handle
  uint32_t* split_ticket;  // FAM_SPLIT: [rows] arrival counters, zero between launches
  uint16_t pro_begin, pro_end;   // tile program run once per thread before the row loop: loads of
                                 // operands that are the same for every row (generated kernels only)
  // shared-memory layout, byte offsets into dynamic shared memory
  int32_t sm_rowoff, sm_part, sm_wpart, sm_slots, sm_ctapart, sm_stash;
  StageDesc stage[kMaxStages];
  uint32_t code[kMaxCode];
};

// One kernel launch as planned by the lowering.
struct LaunchPlan {
  KernelParams p;
  int32_t family;
  int32_t vl, ng, k;       // template instance: vector length, groups per tile, tile registers
  int32_t grid, block, smem_bytes;
  int32_t code_words;
  int64_t items;           // rows, or rows * chunks for pointwise graphs
  int32_t teams_per_cta;
  int32_t specialised;     // 1 when the launch uses a kernel generated for this program
  int32_t persistent;      // 1: grid = resident CTAs, each looping over many rows
  int32_t grid_waves;      // tuning override: the grid is at most this many times the resident CTAs (0 = the default rule,
                           // -1 = one CTA per work item whatever their number)
  int32_t no_prefetch;     // 1: generated kernels issue no loads ahead of the tile in hand
  int32_t bounds;          // 1: the generated kernel is compiled with checked accessors
  int32_t plain_launch;    // 1: launch in plain stream order (no overlap of the set-up with the predecessor's tail)
  int32_t walk_cap;        // column kernels: at most this many steps of the walk in flight (0 = the default)
  int32_t no_reg_bound;    // 1: compile the generated kernel without the tentative register bound (it spilled)
  int64_t io_offset[kMaxIo];   // elements between the start of the tensor's storage and this entry's first element
                               // (non-zero for an output stored as a block of a larger tensor: an operand of a cat)
  int32_t io_tensor[kMaxIo];   // tensor id behind each io entry
  int32_t io_is_output[kMaxIo];
};

}  // namespace pn
