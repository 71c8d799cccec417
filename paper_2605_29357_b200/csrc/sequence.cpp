// sequence.cpp -- pn_sequence_*: many small evaluations bound into one replayable launch.
//
// The paper attributes 61.5 % of the end-to-end slowdowns it measures under a graph compiler to
// fixed per-call overhead on small graphs (Table 6, the root-cause decomposition: about 0.14 ms
// of dispatch per call while the kernels themselves are faster).  For a fused kernel of a few
// microseconds the host's launch path is the same kind of cost.  A sequence records the launches
// of n (handle, pointers) pairs once into a CUDA graph and replays them with one call: the
// pointer checks, the parameter marshalling and the per-kernel launch calls are paid at create
// time, and the kernels run back to back on the GPU.
#include <cuda_runtime.h>

#include <new>
#include <string>
#include <vector>

#include "../../include/pn.h"
#include "handle.h"

using namespace pn;

struct pn_sequence {
  int device = 0;
  int n_items = 0;
  int n_kernels = 0;
  cudaGraph_t graph = nullptr;
  cudaGraphExec_t exec = nullptr;
};

namespace {

constexpr int kLanes = 8;   // capture streams of an independent sequence

struct Capture {   // what a create in progress holds, released on every path out
  cudaStream_t lane[kLanes] = {};
  cudaEvent_t fork = nullptr, join[kLanes] = {};
  bool capturing = false;
  ~Capture() {
    if (capturing) { cudaGraph_t g = nullptr; cudaStreamEndCapture(lane[0], &g); if (g) cudaGraphDestroy(g); }
    for (cudaStream_t s : lane) if (s) cudaStreamDestroy(s);
    if (fork) cudaEventDestroy(fork);
    for (cudaEvent_t e : join) if (e) cudaEventDestroy(e);
  }
};

pn_status cuda_fail(const char* what, cudaError_t e) { return fail(PN_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e)); }

}  // namespace

extern "C" {
#pragma GCC visibility push(default)

pn_status pn_sequence_create(int n, pn_graph_t* const* graphs, const void* const* const* inputs, const int* n_inputs,
                             void* const* const* outputs, const int* n_outputs, unsigned flags, pn_sequence_t** out) {
  if (out) *out = nullptr;
  if (!out || n <= 0 || !graphs || !inputs || !n_inputs || !outputs || !n_outputs) return fail(PN_ERR_INVALID_ARG, "null argument or empty sequence");
  if (flags & ~(unsigned)PN_SEQ_INDEPENDENT) return fail(PN_ERR_INVALID_ARG, "unknown sequence flag");
  for (int i = 0; i < n; ++i) {
    if (!graphs[i]) return fail(PN_ERR_INVALID_ARG, "item " + std::to_string(i) + ": null handle");
    if (graphs[i]->plan_only) return fail(PN_ERR_DEVICE, "item " + std::to_string(i) + ": handle was created with PN_FLAG_PLAN_ONLY");
    if (graphs[i]->device != graphs[0]->device) return fail(PN_ERR_DEVICE, "all handles of a sequence must be bound to one device");
    if (graphs[i]->flags & PN_FLAG_STATIC_SCRATCH) return fail(PN_ERR_INVALID_ARG, "item " + std::to_string(i) + ": static-scratch handles are not recorded");
  }
  const bool independent = (flags & PN_SEQ_INDEPENDENT) != 0;
  if (independent)   // the workspace of a handle (intermediates, partials, arrival counters) is shared by its runs: two of them may not overlap
    for (int i = 0; i < n; ++i)
      for (int j = 0; j < i; ++j)
        if (graphs[i] == graphs[j] && graphs[i]->workspace_bytes > 0)
          return fail(PN_ERR_INVALID_ARG, "a handle that has a workspace appears twice in an independent sequence (items " + std::to_string(j) + " and " + std::to_string(i) + " would share its workspace)");
  pn_sequence* s = new (std::nothrow) pn_sequence();
  if (!s) return fail(PN_ERR_INVALID_ARG, "out of host memory");
  s->device = graphs[0]->device;
  s->n_items = n;
  DeviceScope scope(s->device);   // the caller's current device is put back on every path out
  cudaError_t e = scope.err;
  if (e != cudaSuccess) { delete s; return cuda_fail("cudaSetDevice", e); }

  Capture c;
  const int lanes = independent ? (n < kLanes ? n : kLanes) : 1;
  for (int l = 0; l < lanes; ++l) {
    e = cudaStreamCreateWithFlags(&c.lane[l], cudaStreamNonBlocking);
    if (e != cudaSuccess) { delete s; return cuda_fail("cudaStreamCreate", e); }
    if (l > 0) {
      e = cudaEventCreateWithFlags(&c.join[l], cudaEventDisableTiming);
      if (e != cudaSuccess) { delete s; return cuda_fail("cudaEventCreate", e); }
    }
  }
  if (lanes > 1) {
    e = cudaEventCreateWithFlags(&c.fork, cudaEventDisableTiming);
    if (e != cudaSuccess) { delete s; return cuda_fail("cudaEventCreate", e); }
  }
  // Thread-local capture: CUDA calls of other threads are not affected by it.
  e = cudaStreamBeginCapture(c.lane[0], cudaStreamCaptureModeThreadLocal);
  if (e != cudaSuccess) { delete s; return cuda_fail("cudaStreamBeginCapture", e); }
  c.capturing = true;
  if (lanes > 1) {   // fork: every other lane joins the capture behind the first one's start
    e = cudaEventRecord(c.fork, c.lane[0]);
    for (int l = 1; l < lanes && e == cudaSuccess; ++l) e = cudaStreamWaitEvent(c.lane[l], c.fork, 0);
    if (e != cudaSuccess) { delete s; return cuda_fail("capture fork", e); }
  }
  for (int i = 0; i < n; ++i) {
    const pn_status st = pn_graph_run(graphs[i], inputs[i], n_inputs[i], outputs[i], n_outputs[i], c.lane[i % lanes]);
    if (st != PN_OK) {
      const std::string why = std::string("item ") + std::to_string(i) + ": " + pn_last_error();
      delete s;
      return fail(st, why);
    }
    s->n_kernels += (int)graphs[i]->launches.size();
  }
  for (int l = 1; l < lanes; ++l) {   // join
    e = cudaEventRecord(c.join[l], c.lane[l]);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(c.lane[0], c.join[l], 0);
    if (e != cudaSuccess) { delete s; return cuda_fail("capture join", e); }
  }
  c.capturing = false;
  e = cudaStreamEndCapture(c.lane[0], &s->graph);
  if (e != cudaSuccess || !s->graph) { delete s; return cuda_fail("cudaStreamEndCapture", e); }
  e = cudaGraphInstantiate(&s->exec, s->graph, 0);
  if (e != cudaSuccess) { cudaGraphDestroy(s->graph); delete s; return cuda_fail("cudaGraphInstantiate", e); }
  *out = s;
  return PN_OK;
}

pn_status pn_sequence_run(pn_sequence_t* s, void* stream) {
  if (!s || !s->exec) return fail(PN_ERR_INVALID_ARG, "null sequence");
  DeviceScope scope(s->device);
  if (scope.err != cudaSuccess) return cuda_fail("cudaSetDevice", scope.err);
  const cudaError_t e = cudaGraphLaunch(s->exec, (cudaStream_t)stream);
  if (e != cudaSuccess) return cuda_fail("cudaGraphLaunch", e);
  return PN_OK;
}

pn_status pn_sequence_query(const pn_sequence_t* s, int what, void* out, size_t out_bytes) {
  if (!s || !out || out_bytes < sizeof(int64_t)) return fail(PN_ERR_INVALID_ARG, "null argument or buffer too small");
  int64_t v;
  switch (what) {
    case PN_SQ_N_ITEMS: v = s->n_items; break;
    case PN_SQ_N_KERNELS: v = s->n_kernels; break;
    default: return fail(PN_ERR_INVALID_ARG, "unknown query");
  }
  *static_cast<int64_t*>(out) = v;
  return PN_OK;
}

pn_status pn_sequence_destroy(pn_sequence_t* s) {
  if (!s) return PN_OK;
  if (s->exec) cudaGraphExecDestroy(s->exec);
  if (s->graph) cudaGraphDestroy(s->graph);
  delete s;
  return PN_OK;
}

#pragma GCC visibility pop
}  // extern "C"
