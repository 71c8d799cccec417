/*
 * pn.h -- C ABI of the fused-subgraph executor for NVIDIA B200 (sm_100a).
 *
 * The library runs a "long-tail fusible subgraph" -- a DAG of pointwise operators
 * with broadcasting, optional reductions (over the last dimension, or over one leading
 * dimension), and a normalisation / scaling epilogue -- as ONE pass over HBM instead of
 * one kernel per operator.  The input is the paper's computational graph G = (V, E, tau, sigma)
 * (Definition 3.1: operator nodes, data dependencies, an operator type per node and a
 * static output shape per node), serialised as a descriptor.  What a handle computes
 * is f_G; a fused execution is acceptable when it equals the per-operator evaluation
 * within a tolerance (Definition 3.2, Eq. 1).  One handle serves one shape / dtype
 * instance of a graph, as in the paper's task formulation (Section 3.1).
 *
 * All functions are thread-safe with respect to different handles.  Nothing throws
 * or aborts across this boundary: every failure is a negative pn_status, with a
 * thread-local detail message available from pn_last_error().
 *
 * Descriptor format, version 1 (little-endian):
 *   header  16 B : u32 magic 0x31474E50 ('PNG1') | u16 version = 1 | u16 0
 *                  | u32 n_tensors | u32 n_nodes
 *   tensor  40 B : u8 dtype | u8 role (bit0 graph input, bit1 graph output) | u8 rank (<= 4)
 *                  | u8 0 | u32 0 | i64 dims[4]
 *   node    64 B : u16 opcode | u8 n_in (<= 4) | u8 n_out (1..3) | u32 in[4] | u32 out[3]
 *                  | f64 imm[2] | i64 attr[2]
 * Tensor ids are table positions.  Graph inputs / outputs are the tensors carrying the
 * role bit, in table order: that order is the order of the pointer arrays passed to
 * pn_graph_run.  An operand slot equal to 0xFFFFFFFF / 0xFFFFFFFE names imm[0] / imm[1].
 * Nodes are listed in topological order.  All tensors are dense, row-major, last
 * dimension contiguous; operands broadcast by NumPy's size-1 rules.  Reductions and
 * composites act over the last dimension; their per-row results have the input's
 * shape with the last dimension dropped or kept as 1.
 *
 * Opcodes: 1 neg, 2 abs, 3 exp, 4 log, 5 sqrt, 6 rsqrt, 7 recip, 8 tanh, 9 sigmoid,
 * 10 silu, 11 gelu_tanh, 12 gelu_erf, 13 relu, 14 cast (to the output tensor's dtype),
 * 15 square, 16 erf; 32 add, 33 sub, 34 mul, 35 div, 36 max, 37 min, 38 gt, 39 ge,
 * 40 lt, 41 le, 42 eq, 43 ne; 64 where(c, a, b), 65 clamp(x, lo, hi), 66 fma(a, b, c);
 * 96 sum, 97 mean, 98 var (attr[0] = correction), 99 amax, 100 amin, 101 argmax,
 * 102 argmin (lowest index on ties; i32 / i64 result), 103 logsumexp; 128 softmax,
 * 129 log_softmax, 130 layer_norm(x[, gamma[, beta]]) -> y[, mean, rstd] with
 * imm[0] = eps, 131 rms_norm(x[, gamma]) with imm[0] = eps.
 * Reductions over ONE LEADING dimension (the masked-mean-pooling shape of the paper's second
 * case study, Section 4.4): 104 sum_dim, 105 mean_dim, 106 amax_dim, 107 amin_dim with
 * attr[0] = the reduced dimension (not the last one); the result has the operand's shape with
 * that dimension dropped or kept as 1.  A graph may hold several of them over the same
 * dimension, a pointwise chain before them and one after them on the reduced values; a reduced
 * value cannot flow back into a tensor that still has the reduced dimension.
 * Index operators (the index-remapped loads of the paper's first case study, Section 4.4): 160
 * roll (attr = dim, shift), 161 slice (attr = dim, start; length from the output shape), 162 view
 * (regroups leading dimensions; of a tensor that is still dense, any dimensions).  A roll or slice
 * over two dimensions at once, as graph traces have them, gives the second one in
 * imm = (1 + dim, shift / start); imm[0] = 0 means one dimension.  They act on any dimension of
 * graph inputs, or of chains of index operators that start at one, and cost no data movement: the
 * fused kernel computes the source row instead (idx = (S + i - shift) mod S); along the last
 * dimension a slice is an offset of the row's start and a roll a circular shift of the columns
 * (whole 128-bit groups when shift and row length allow it, element by element otherwise), so the
 * two halves of a gated activation are two views of one input.  On a computed value an index
 * operator starts a launch of its own.  164 contiguous: the identity on values (every
 * tensor here is dense already); after a chain of index operators it is one more link of the chain,
 * on a computed value a pointwise identity.  163 cat (attr[0] = dim, up to 4 operands of the
 * result's dtype): with one operand it is the identity, as graph traces contain it; with several it
 * is not computed at all: every operand is stored straight into its block of the result by the
 * kernel that produces it (an output-address remap), operands of different shapes by a launch
 * each, and a node that reads the result runs in a later launch.
 * Arithmetic is fp32 in registers whatever the storage types; integer and boolean
 * tensors take part as exact small integers / predicates; a node whose declared
 * output dtype is bf16 / f16 is rounded to it (nearest even) for its consumers.
 */
#ifndef PN_H_
#define PN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct pn_graph pn_graph_t; /* opaque handle */
typedef int pn_status;

/*
 * Status codes.  The paper sorts the ways a rewritten graph can fail into three categories
 * (Section 3.5: accuracy, compilation, runtime).  Here a "compilation" failure is any negative
 * status of pn_graph_create (the graph could not be parsed, lowered or compiled: codes -2 .. -5,
 * -8, and -9 with the compiler's log), a "runtime" failure any negative status of a run call
 * (codes -1, -6, -7, -9), and an "accuracy" failure is not a status at all: it is what the
 * tolerance rule of Eq. 1 detects when outputs are compared (the tests, and the report module).
 */
enum {
  PN_OK = 0,
  PN_ERR_INVALID_ARG = -1,    /* null pointer, bad enum, bad size                       */
  PN_ERR_BAD_DESCRIPTOR = -2, /* malformed bytes, ids out of range, not topological     */
  PN_ERR_UNSUPPORTED_OP = -3, /* unknown opcode, or an operator / dtype mix not lowered */
  PN_ERR_SHAPE = -4,          /* broadcast mismatch, reduction result of the wrong shape */
  PN_ERR_TOO_LARGE = -5,      /* exceeds the bytecode, register, I/O or stage budget    */
  PN_ERR_ALIGNMENT = -6,      /* a device pointer is less aligned than the plan needs   */
  PN_ERR_COUNT = -7,          /* n_inputs / n_outputs differ from the descriptor        */
  PN_ERR_DEVICE = -8,         /* no such device, or not an sm_100 part                  */
  PN_ERR_CUDA = -9            /* a CUDA call failed; text in pn_last_error()            */
};

/* dtype codes of the descriptor */
enum { PN_F32 = 0, PN_F16 = 1, PN_BF16 = 2, PN_I8 = 3, PN_BOOL = 4, PN_I32 = 5, PN_I64 = 6 };

/* create-time flags */
enum {
  PN_FLAG_UNFUSED = 1u << 0,      /* one kernel per node, intermediates in a workspace   */
  PN_FLAG_PLAN_ONLY = 1u << 1,    /* no CUDA call at all: lower for a B200, allow query  */
  PN_FLAG_FORCE_WARP = 1u << 4,   /* row kernels: one warp per row                        */
  PN_FLAG_FORCE_BLOCK = 1u << 5,  /* row kernels: one thread block per row                */
  PN_FLAG_FORCE_CLUSTER = 1u << 6,/* row kernels: one thread-block cluster per row        */
  PN_FLAG_FORCE_SCALAR = 1u << 7, /* element-wise (unvectorised) memory accesses          */
  PN_FLAG_FORCE_MULTICHUNK = 1u << 8,/* smallest tile: rows span several chunks per thread */
  PN_FLAG_INTERPRET = 1u << 9,    /* run the bytecode on the interpreter kernels built into the
                                     library instead of a kernel specialised for the graph */
  PN_FLAG_NO_HOIST = 1u << 10,    /* do not move row-invariant operand loads out of the row loop */
  PN_FLAG_PREFETCH = 1u << 11,    /* generated kernels: issue the first stage's loads one tile
                                     ahead (costs registers; off by default)                 */
  PN_FLAG_STATIC_SCRATCH = 1u << 12,/* with PN_FLAG_UNFUSED: allocate no workspace; the handle
                                     is run with pn_graph_run_static only                    */
  PN_FLAG_PLAIN_LAUNCH = 1u << 2, /* launch the generated kernels in plain stream order.  By default they
                                     are launched with programmatic stream serialization: a kernel is
                                     set up while its predecessor in the stream still runs and waits
                                     at its head until that one is complete -- the same results, about
                                     a microsecond less per launch for kernels of a few microseconds */
  PN_FLAG_ONE_KERNEL = 1u << 3,   /* a graph that does not fit one kernel (a bytecode, register, scalar,
                                     I/O or stage budget; a combination the fused lowering does not
                                     take) is refused with PN_ERR_TOO_LARGE / PN_ERR_UNSUPPORTED_OP
                                     instead of being cut into several fused launches          */
  PN_FLAG_FORCE_SPLIT = 1u << 15, /* row kernels: independent blocks over slices of a row, combined
                                     through partials in a workspace of the handle (single-stage
                                     graphs, generated kernels); kernels that reduce over a
                                     leading dimension: at least two slices of that dimension  */
  PN_FLAG_ALLOW_INTERPRET = 1u << 14,/* a create that cannot specialise kernels (NVRTC or the driver
                                     library cannot be opened) normally fails with PN_ERR_DEVICE;
                                     with this flag it runs on the interpreter kernels instead  */
  PN_FLAG_BOUNDS = 1u << 13       /* checked accessors: every global access of the kernels is tested
                                     against the extent of its tensor; one that falls outside is
                                     skipped and recorded in a status word on the device (4 bytes
                                     owned by the handle), read with PN_Q_BOUNDS_STATUS.  A debugging
                                     aid at some cost in speed; a correct build always reads 0   */
};
/* Size of the fixed scratch array behind pn_graph_run_static. */
#define PN_STATIC_SCRATCH_BYTES (32ll << 20)
/* Tuning overrides of the lowering's own choices, for measurements and tests: OR them into
 * `flags`.  A value of 0 leaves the choice to the lowering; an impossible one is ignored. */
#define PN_TUNE_CLUSTER(n) (((unsigned)(n) & 15u) << 16)      /* CTAs per cluster: 2, 4, 8; split-row kernels: tiles per
                                                                 slice; column-reduce kernels: slices of the reduced
                                                                 dimension (2..15)                */
#define PN_TUNE_BLOCK_LOG2(n) (((unsigned)(n) & 15u) << 20)   /* threads per block = 1 << n     */
#define PN_TUNE_GROUPS(n) (((unsigned)(n) & 31u) << 24)       /* vector groups per thread tile  */
#define PN_TUNE_WAVES(n) (((unsigned)(n) & 7u) << 29)         /* grid <= 2^(n-1) x the resident CTAs; 7: one CTA per work item */

/* pn_graph_query selectors; each writes int64 values into `out` */
enum {
  PN_Q_N_INPUTS = 1,        /* 1 value                                                   */
  PN_Q_N_OUTPUTS = 2,       /* 1 value                                                   */
  PN_Q_INPUT_META = 3,      /* per input 6 values: dtype, rank, dims[4]                  */
  PN_Q_OUTPUT_META = 4,     /* per output 6 values                                       */
  PN_Q_COMPULSORY_BYTES = 5,/* 1 value: every input read once + every output written once */
  PN_Q_N_KERNELS = 6,       /* 1 value: launches per pn_graph_run (1 when fused)         */
  PN_Q_N_NODES = 7,         /* 1 value: operator nodes in the descriptor                 */
  PN_Q_WORKSPACE_BYTES = 8, /* 1 value: device memory owned by the handle                */
  PN_Q_BOUNDS_STATUS = 10,  /* 1 value, PN_FLAG_BOUNDS handles only: bit q set when an access to the
                               q-th input / output entry of a launch fell outside its tensor;
                               waits for the device                                        */
  PN_Q_KERNEL_CACHE = 11,   /* 2 values, process-wide: generated kernels now loaded, and how many of
                               them a live handle uses                                      */
  PN_Q_KERNEL_INFO = 9      /* per kernel 14 values: family (0 pointwise, 1 warp-per-row,
                               2 block-per-row, 3 cluster-per-row, 5 split-row, 4 column-reduce: rows =
                               the dimensions before the reduced one, row length = those after
                               it), grid, block, cluster,
                               dynamic smem bytes, vector length, groups per tile, chunks
                               per row slice, bytecode words, stages, rows, row length,
                               specialised (1) or interpreted (0), slices (split-row: of a row;
                               column-reduce: of the reduced dimension; else 0)          */
};

/*
 * pn_graph_create -- parse, validate and lower a graph (the host side of running G of
 * Definition 3.1; the lowering picks a kernel family and tile per shape: the hardware
 * cost model whose absence -- one tile shape kept whatever the tensor shape -- the paper counts
 * among the failure modes of generated passes, Section 4.4).
 *   desc, desc_bytes : HOST pointer to the descriptor; copied, caller may free it.
 *   device           : CUDA device ordinal the handle is bound to.
 *   flags            : PN_FLAG_* bits.
 *   out              : receives the handle; set to NULL on failure.
 * A graph that exceeds what one kernel takes (the paper's fusible subgraphs run to 35 operators,
 * its classical ones to 62: Section 3.3) is cut into the cheapest sequence of fused launches --
 * consecutive runs of nodes, the tensors that cross a cut written once to a workspace of the handle
 * and read once; cheapest by bytes moved, then by launches -- unless PN_FLAG_ONE_KERNEL asks for the
 * refusal.  PN_Q_N_KERNELS tells the number of launches, PN_Q_WORKSPACE_BYTES the workspace.
 * Allocates device memory for the workspace of such cuts, of PN_FLAG_UNFUSED (the intermediates
 * between all nodes) and of split-row kernels (partials and arrival counters of rows reduced by
 * several independent blocks) -- owned by the handle and released by pn_graph_destroy.  Launches
 * no kernel.
 * Unless PN_FLAG_INTERPRET is given, the bytecode of each launch is also translated into a
 * kernel of its own and compiled for sm_100a with NVRTC (a few hundred ms per distinct
 * kernel).  Loaded kernels are shared through a process-wide cache, reference-counted by the
 * handles that use them; unused ones are unloaded, least recently used first, beyond 256.  With
 * the environment variable PN_CACHE_DIR set, compiled kernels are also kept in that directory
 * (keyed by a hash of the source, the NVRTC version and sm_100a) and a later process loads them
 * without compiling.  NVRTC is looked for at PN_NVRTC_PATH, else under CUDA_HOME / CUDA_PATH /
 * /usr/local/cuda, else by soname.  If NVRTC or the driver library cannot be opened the create
 * FAILS with PN_ERR_DEVICE and the reason, unless PN_FLAG_INTERPRET or PN_FLAG_ALLOW_INTERPRET
 * was given (the interpreter kernels are more than ten times slower); PN_Q_KERNEL_INFO tells
 * which kind a handle runs.  The calling thread's current device is left as it was.
 * Two more environment variables are aids for measurement and debugging: PN_NVRTC_FLAGS adds
 * options to the run-time compilation (e.g. -DPN_MIN_BLOCKS=6, the resident blocks per SM the
 * register allocation aims at), PN_DEBUG_PARTITION prints to stderr how a graph was cut into
 * launches and why the runs that were tried did not lower, PN_DEBUG_SPEC the registers and local
 * memory of every generated kernel as it is loaded.
 */
pn_status pn_graph_create(const void* desc, size_t desc_bytes, int device, unsigned flags,
                          pn_graph_t** out);

/*
 * pn_graph_run -- enqueue one evaluation of f_G (Definition 3.1) on `stream`.
 *   inputs  : HOST array of n_inputs DEVICE pointers, descriptor input order; read-only.
 *   outputs : HOST array of n_outputs DEVICE pointers, descriptor output order; every
 *             element of every output is overwritten.
 *   stream  : a cudaStream_t (NULL = the default stream).
 * Asynchronous: returns after the launch(es).  No allocation, no host synchronisation.
 * Stream order holds as for any kernel launch; the generated kernels are, unless
 * PN_FLAG_PLAIN_LAUNCH was given, set up while the kernel before them in the stream still runs and
 * touch no memory until that kernel is complete and its writes are visible.
 * Pointers must be aligned to 16 bytes unless the handle was created with
 * PN_FLAG_FORCE_SCALAR (then to the element size); otherwise PN_ERR_ALIGNMENT.  Inputs
 * and outputs must not overlap, not even exactly: the kernels read inputs through the
 * read-only data path, which does not see a kernel's own writes.  The library never retains or
 * frees user memory.  The handle itself is only read, so runs of one fused handle may be issued
 * from several threads and streams at once; runs of a handle that has a workspace
 * (PN_Q_WORKSPACE_BYTES > 0: unfused handles, graphs cut into several launches, rows or a reduced
 * leading dimension split over independent blocks) share that workspace and must be stream-ordered by the caller.  The launch
 * goes to the handle's device whatever device the calling thread has current, and that choice
 * is left as it was.  A graph any of whose inputs or outputs has zero elements runs as a no-op.
 */
pn_status pn_graph_run(pn_graph_t* g, const void* const* inputs, int n_inputs,
                       void* const* outputs, int n_outputs, void* stream);

/*
 * pn_graph_bind / pn_bound_run / pn_bound_destroy -- the same evaluation of f_G (Definition 3.1)
 * with the per-call work done once.  The paper finds fixed per-call overhead to be what sinks
 * small graphs (Table 6); for a fused kernel of a few microseconds the argument checks and the
 * marshalling of a 4 KB parameter block are that kind of cost.  pn_graph_bind runs the checks of
 * pn_graph_run on one set of pointers and stores the filled-in launch parameters in a bound
 * object; pn_bound_run(b, stream) is then one launch call per kernel and nothing else.
 *   g, inputs, outputs : as for pn_graph_run; the DEVICE pointers are recorded, the caller keeps
 *                        the buffers alive and unmoved while the bound object is used.
 *   out                : receives the bound object (HOST memory owned by the library); NULL on
 *                        failure.  It must be destroyed before its handle.
 * Errors of pn_graph_bind: those of pn_graph_run; PN_ERR_INVALID_ARG for a PN_FLAG_STATIC_SCRATCH
 * handle.  pn_bound_run: PN_ERR_INVALID_ARG for NULL, PN_ERR_CUDA for a failed launch.  A bound
 * object is immutable: pn_bound_run may be called from several threads at once (the workspace
 * rule of pn_graph_run applies).  Asynchronous, no allocation at run time, capturable in a CUDA
 * graph like pn_graph_run.
 * pn_bound_run_many(bound, n, stream): the launches of n bound objects, in the order of the HOST
 * array `bound`, on one stream, in one call -- for many small subgraphs whose pointers are known
 * but which are not worth a CUDA graph; stops at the first failure and returns its status (the
 * launches before it stay enqueued).  n = 0 is a no-op.
 */
typedef struct pn_bound pn_bound_t;
pn_status pn_graph_bind(pn_graph_t* g, const void* const* inputs, int n_inputs, void* const* outputs,
                        int n_outputs, pn_bound_t** out);
pn_status pn_bound_run(pn_bound_t* b, void* stream);
pn_status pn_bound_run_many(pn_bound_t* const* bound, int n, void* stream);
pn_status pn_bound_destroy(pn_bound_t* b);

/*
 * pn_graph_run_host -- the same evaluation of f_G (Definition 3.1) for callers whose
 * tensors live in HOST memory: copies each input to the device, runs, copies each output
 * back and waits.  `inputs` / `outputs` are HOST arrays of HOST pointers to dense buffers
 * of the sizes the descriptor states (pinned memory lets the copies run at full speed).
 * Staging buffers are allocated on first use and owned by the handle.  When the inputs are
 * large (tens of MB) and the work of a fused handle can be cut along its outermost dimension,
 * the call works in pieces: the copy in of one piece, the kernel on the piece before and the
 * copy out of the one before that run at the same time, on two copy streams of the handle's
 * own beside `stream`, so that both directions of the host link are busy; tensors without the
 * outermost dimension (broadcast operands) are copied whole first.  The results are the same
 * bits as in one piece.  The call returns when everything has arrived.
 */
pn_status pn_graph_run_host(pn_graph_t* g, const void* const* inputs, int n_inputs,
                            void* const* outputs, int n_outputs, void* stream);

/*
 * pn_graph_run_static -- the unfused evaluation (one kernel per node) without any allocation.
 * The paper has no counterpart to this call; it exists for a class of callers.
 *
 * Who needs it: code that runs after its process has stopped allocating device memory --
 * a serving loop whose framework took all free HBM into its own pool at start-up (a late
 * cudaMalloc there fails, or succeeds only by stalling every stream, since it synchronises
 * the device), or a worker that is handed a fixed memory budget and may not grow it.  Such
 * a caller cannot create an ordinary PN_FLAG_UNFUSED handle, whose workspace for the
 * intermediates between the per-node kernels comes from cudaMalloc.
 *
 * What it does instead: the intermediates go into one fixed array of
 * PN_STATIC_SCRATCH_BYTES (32 MiB) that is part of the library's device image.  A GPU starts
 * holding that array when the library's device code for it is first loaded there -- which
 * pn_graph_create does for a handle with PN_FLAG_STATIC_SCRATCH -- and holds it until the
 * process exits.
 *   g       : a handle created with PN_FLAG_UNFUSED | PN_FLAG_STATIC_SCRATCH.  That create is
 *             the set-up step and the one place that may fail for lack of memory: it allocates
 *             no workspace, but it looks up the array's device address (cudaGetSymbolAddress,
 *             once per device, with that device current), and under the CUDA runtime's lazy
 *             loading that lookup is what reserves the 32 MiB on the device.  Do it while the
 *             process may still allocate, and before any stream capture begins.  Combine the
 *             flags with PN_FLAG_INTERPRET if the create must not load generated kernels
 *             either.  pn_graph_run, pn_graph_run_host and pn_graph_bind refuse such a handle.
 *   inputs, outputs, stream : as for pn_graph_run (HOST arrays of DEVICE pointers that the
 *             caller owns; the same alignment and no-overlap rules, checked by the same code).
 * Errors: PN_ERR_TOO_LARGE when the graph's intermediates need more than
 * PN_STATIC_SCRATCH_BYTES (pn_graph_query PN_Q_WORKSPACE_BYTES tells how much);
 * PN_ERR_INVALID_ARG for a handle without the two flags; otherwise as pn_graph_run.
 * The call itself uses no cudaMalloc, cudaFree or other allocating routine, looks nothing up,
 * and leaves the free device memory exactly as it found it.
 *
 * All calls, from all handles and threads, share the one array per device and it keeps
 * whatever the last call left: nothing has to start at zero (each intermediate is fully
 * written before it is read), but two calls whose kernels overlap on the GPU -- different
 * streams, no ordering between them -- race on it.  Order them.
 */
pn_status pn_graph_run_static(pn_graph_t* g, const void* const* inputs, int n_inputs,
                              void* const* outputs, int n_outputs, void* stream);

/*
 * Sequences: many small evaluations replayed with one call.
 *
 * The paper traces 61.5 % of the end-to-end slowdowns it measures under a graph compiler to
 * fixed per-call overhead on graphs of fewer than 15 nodes: about 0.14 ms of dispatch per call
 * while the kernels themselves got faster (Table 6, root-cause decomposition).  A fused kernel
 * of a few microseconds meets the same kind of cost in the host's launch path.  A sequence
 * pays it once: pn_sequence_create runs the pointer checks and records the launches of all its
 * items into a CUDA graph; pn_sequence_run replays them with a single launch call, the kernels
 * running back to back on the GPU.
 *
 * pn_sequence_create
 *   n                : number of items (> 0).
 *   graphs           : HOST array of n handles, all bound to one device; a handle may appear
 *                      several times.  The handles must outlive the sequence.
 *   inputs, outputs  : HOST arrays of n pointers to HOST arrays of DEVICE pointers, per item
 *                      as for pn_graph_run; n_inputs / n_outputs give their lengths.  The
 *                      device pointers are recorded: the sequence reads and writes exactly
 *                      those buffers at every run; the caller keeps them alive.
 *   flags            : 0: the items run in order, each after the one before (outputs of one
 *                      may be inputs of the next).  PN_SEQ_INDEPENDENT: the caller states that
 *                      no item reads or writes what another writes; items are then recorded on
 *                      parallel branches and small kernels may overlap on the GPU.
 *   out              : receives the sequence; NULL on failure.
 * Creates streams and events for the recording and releases them before it returns; allocates
 * no device memory of its own.  Errors: those of pn_graph_run for any item (the message names
 * the item); PN_ERR_DEVICE for handles of different devices; PN_ERR_INVALID_ARG for a
 * PN_FLAG_STATIC_SCRATCH handle, or for an unfused handle that appears twice in an
 * independent sequence (its runs share one workspace).
 *
 * pn_sequence_run -- enqueue one replay on `stream` (a cudaStream_t); asynchronous.  Replays of
 * one sequence, and a replay and a direct run of an unfused handle it contains, must be
 * stream-ordered by the caller.
 * pn_sequence_query -- PN_SQ_N_ITEMS / PN_SQ_N_KERNELS: one int64 into `out` (HOST memory).
 * pn_sequence_destroy -- release the sequence (not its handles); NULL is accepted.
 */
typedef struct pn_sequence pn_sequence_t;
enum { PN_SEQ_INDEPENDENT = 1u << 0 };
enum { PN_SQ_N_ITEMS = 1, PN_SQ_N_KERNELS = 2 };
pn_status pn_sequence_create(int n, pn_graph_t* const* graphs, const void* const* const* inputs,
                             const int* n_inputs, void* const* const* outputs, const int* n_outputs,
                             unsigned flags, pn_sequence_t** out);
pn_status pn_sequence_run(pn_sequence_t* s, void* stream);
pn_status pn_sequence_query(const pn_sequence_t* s, int what, void* out, size_t out_bytes);
pn_status pn_sequence_destroy(pn_sequence_t* s);

/* pn_graph_destroy -- end of the life of one instance of G (Definition 3.1; Section 3.1: one handle
 * per shape / dtype instance): releases the handle, its workspace, staging buffers and status word,
 * and gives its kernels back to the process-wide cache.  Bound launches and sequences made from
 * the handle must be destroyed first.  NULL is accepted. */
pn_status pn_graph_destroy(pn_graph_t* g);

/*
 * pn_graph_query -- introspection for tests and benchmarks (the kernel count is the
 * paper's "kernels N -> 1" figure of Table 2).  Writes int64 values as listed beside
 * each PN_Q_* selector into `out` (HOST memory, out_bytes large enough, else
 * PN_ERR_INVALID_ARG).
 */
pn_status pn_graph_query(const pn_graph_t* g, int what, void* out, size_t out_bytes);

/*
 * pn_graph_codegen -- the CUDA source generated for launch `kernel` of a handle (the
 * translation of its bytecode; the device library it is compiled against is not repeated).
 * Copies at most out_bytes - 1 characters plus a terminator into `out` (HOST memory; may be
 * NULL with out_bytes 0) and stores the full length in *needed if that is not NULL.  With
 * compile != 0 the source is also compiled for sm_100a with NVRTC, without loading it: this
 * needs no GPU and returns PN_ERR_CUDA with the compiler's log on failure.  The paper has no
 * counterpart: an aid for tests and for reading what the specialiser made of a graph.
 */
pn_status pn_graph_codegen(const pn_graph_t* g, int kernel, int compile, char* out, size_t out_bytes,
                           size_t* needed);

/*
 * pn_stream_probe -- a streaming kernel that only moves bytes, for the roofline: the rate it
 * reaches in a given read : write mix is the ceiling that a fused kernel of the same mix can be
 * judged against (the paper times whole subgraphs, Appendix C's protocol, and has no counterpart
 * to a bandwidth ceiling; this call is a measuring aid, not part of evaluating f_G).
 *   mix    : PN_MIX_READ   read a                      (a long-row reduction)
 *            PN_MIX_WRITE  write c
 *            PN_MIX_1_1    read a, write c             (softmax, a plain copy)
 *            PN_MIX_2_1    read a and b, write c       (residual + LayerNorm)
 *            PN_MIX_4_3    read a and b, write c and d (two 2-byte inputs, a 2-byte and a 1-byte output)
 *   cfg    : HOST pointer; how to move them (see the struct).
 *   a, b, c: DEVICE buffers of units * 16 bytes each; d of units * 8 bytes; those the mix does not
 *            use may be NULL.  All aligned to 16 bytes; owned by the caller; a, b are only read.
 *   units  : 16-byte units per array.
 *   status_word : DEVICE pointer to 4 zeroed bytes (aligned to 16): bit 0 / 1 set when a bounded
 *            wait of the bulk loader's producer / consumers ran out (the kernel then stops early,
 *            after its copies in flight have landed); always 0 for the other loaders.
 *   stream : a cudaStream_t.  Asynchronous; allocates nothing.
 * Errors: PN_ERR_INVALID_ARG / PN_ERR_ALIGNMENT / PN_ERR_TOO_LARGE for a bad configuration,
 * PN_ERR_CUDA for a failed launch.
 */
enum { PN_MIX_READ = 0, PN_MIX_WRITE = 1, PN_MIX_1_1 = 2, PN_MIX_2_1 = 3, PN_MIX_4_3 = 4 };
enum {
  PN_PROBE_LDG = 0,         /* 128-bit loads through the read-only path                      */
  PN_PROBE_LDG_NOALLOC = 1, /* the same, not allocating in L1                                */
  PN_PROBE_BULK = 2         /* 1-D bulk copies into a shared-memory ring (mbarrier completion;
                               one extra producer warp per block; this GPU's memory only)    */
};
typedef struct pn_probe_config {
  int loader;           /* PN_PROBE_*                                                         */
  int streaming_stores; /* 1: stores carry the evict-first hint                               */
  int layout;           /* direct loaders: 0 grid-stride over units, 1 a contiguous range per block,
                           2 runs of tile_units units taken by the blocks in turn, 3 (PN_MIX_READ only)
                           strips: the array as rows of tile_units units, a block owning strip_units
                           units by rows_per_block rows, its block / strip_units walkers going down
                           the rows (the pattern of a reduction over a leading dimension; the grid
                           follows from the sizes)                                              */
  int block;            /* threads that load / store per block (multiple of 32, <= 992)       */
  int unroll;           /* direct loaders: units in flight per thread (1, 2, 4, 8)            */
  int grid;             /* blocks                                                             */
  int stages;           /* bulk loader: ring depth (2..16)                                    */
  int tile_units;       /* bulk loader: units per array per stage (32..4096); layout 2: the run length;
                           layout 3: units per row                                              */
  int strip_units;      /* layout 3: units a strip is wide                                    */
  int rows_per_block;   /* layout 3: rows a strip is long                                     */
} pn_probe_config;
pn_status pn_stream_probe(int mix, const pn_probe_config* cfg, const void* a, const void* b, void* c, void* d,
                          size_t units, void* status_word, void* stream);

/* pn_status_string -- static text for a status code (the failure classes of Section 3.5 as mapped
 * beside the status enum above); never NULL. */
const char* pn_status_string(pn_status s);

/* pn_last_error -- detail of the calling thread's most recent failure ("" if none): for a
 * "compilation" failure (Section 3.5) the node and the rule it broke, or the run-time compiler's
 * log; for a "runtime" failure the argument or the CUDA error.  The pointer stays valid until the
 * same thread's next failing call. */
const char* pn_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* PN_H_ */
