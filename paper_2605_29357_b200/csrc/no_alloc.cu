// no_alloc.cu -- pn_graph_run_static: the unfused (one kernel per node) evaluation for
// callers that must not allocate device memory.  The intermediates between the per-node
// kernels, which pn_graph_run keeps in a workspace obtained with cudaMalloc when the handle
// is created, live here in one fixed array that is part of the library's device image.
#include <cuda_runtime.h>

#include <mutex>
#include <string>

#include "../../include/pn.h"
#include "handle.h"

namespace pn {
cudaError_t launch_plan(const LaunchPlan& lp, cudaStream_t stream);   // kernels.cu
}

using namespace pn;

// The scratch itself, at file scope.  Every GPU that loads the library holds these bytes until
// the process exits, whether or not the entry point is ever called.
static __device__ __align__(256) unsigned char g_static_scratch[PN_STATIC_SCRATCH_BYTES];

namespace {

// In host code the name above is only a stand-in for the symbol: its address as a device
// pointer has to be asked for, once per device, with that device current.
constexpr int kMaxDevices = 64;
void* g_scratch_ptr[kMaxDevices] = {};
std::mutex g_setup_mutex;

pn_status scratch_for_device(int device, void** out) {
  if (device < 0 || device >= kMaxDevices) return fail(PN_ERR_DEVICE, "device ordinal out of range");
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_ptr[device]) {
    cudaError_t e = cudaSetDevice(device);
    if (e != cudaSuccess) return fail(PN_ERR_CUDA, std::string("cudaSetDevice: ") + cudaGetErrorString(e));
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (e != cudaSuccess || !ptr) return fail(PN_ERR_CUDA, std::string("cudaGetSymbolAddress: ") + cudaGetErrorString(e));
    g_scratch_ptr[device] = ptr;
  }
  *out = g_scratch_ptr[device];
  return PN_OK;
}

int64_t bytes_of(const Tensor& t) { return t.numel() * dtype_bytes(t.dtype); }

}  // namespace

extern "C" {
#pragma GCC visibility push(default)

pn_status pn_graph_run_static(pn_graph_t* h, const void* const* inputs, int n_inputs, void* const* outputs,
                              int n_outputs, void* stream) {
  if (!h || (!inputs && n_inputs > 0) || !outputs) return fail(PN_ERR_INVALID_ARG, "null argument");
  if (h->plan_only) return fail(PN_ERR_DEVICE, "handle was created with PN_FLAG_PLAN_ONLY");
  if (!(h->flags & PN_FLAG_UNFUSED) || !(h->flags & PN_FLAG_STATIC_SCRATCH))
    return fail(PN_ERR_INVALID_ARG, "pn_graph_run_static needs a handle created with PN_FLAG_UNFUSED | PN_FLAG_STATIC_SCRATCH");
  const Graph& g = h->g;
  if (n_inputs != (int)g.inputs.size() || n_outputs != (int)g.outputs.size())
    return fail(PN_ERR_COUNT, "expected " + std::to_string(g.inputs.size()) + " inputs and " +
                                  std::to_string(g.outputs.size()) + " outputs");
  if (h->workspace_bytes > (size_t)PN_STATIC_SCRATCH_BYTES)
    return fail(PN_ERR_TOO_LARGE, "the graph's intermediates need " + std::to_string(h->workspace_bytes) +
                                      " bytes; the static scratch holds " + std::to_string((long long)PN_STATIC_SCRATCH_BYTES));
  for (const Tensor& t : g.tensors) if (t.numel() == 0) return PN_OK;   // nothing to compute
  const bool scalar = (h->flags & PN_FLAG_FORCE_SCALAR) != 0;
  for (int i = 0; i < n_inputs; ++i) {
    if (!inputs[i]) return fail(PN_ERR_INVALID_ARG, "input " + std::to_string(i) + " is null");
    const uintptr_t m = scalar ? (uintptr_t)(dtype_bytes(g.tensors[g.inputs[i]].dtype) - 1) : 15;
    if ((uintptr_t)inputs[i] & m) return fail(PN_ERR_ALIGNMENT, "input " + std::to_string(i) + " is not aligned");
  }
  for (int o = 0; o < n_outputs; ++o) {
    if (!outputs[o]) return fail(PN_ERR_INVALID_ARG, "output " + std::to_string(o) + " is null");
    const uintptr_t m = scalar ? (uintptr_t)(dtype_bytes(g.tensors[g.outputs[o]].dtype) - 1) : 15;
    if ((uintptr_t)outputs[o] & m) return fail(PN_ERR_ALIGNMENT, "output " + std::to_string(o) + " is not aligned");
    const char* b0 = (const char*)outputs[o];
    const char* b1 = b0 + bytes_of(g.tensors[g.outputs[o]]);
    for (int i = 0; i < n_inputs; ++i) {
      const char* a0 = (const char*)inputs[i];
      if (a0 < b1 && b0 < a0 + bytes_of(g.tensors[g.inputs[i]]))
        return fail(PN_ERR_INVALID_ARG, "input " + std::to_string(i) + " overlaps output " + std::to_string(o));
    }
  }
  void* scratch = nullptr;
  pn_status st = scratch_for_device(h->device, &scratch);
  if (st != PN_OK) return st;
  // Every intermediate is fully written by the kernel that produces it before any kernel
  // reads it (the launches are stream-ordered), so nothing left by an earlier call is ever
  // read and nothing needs clearing.
  for (PlannedLaunch& pl : h->launches) {
    for (int q = 0; q < pl.plan.p.n_io; ++q) {
      const IoSource& s = pl.src[q];
      pl.plan.p.io[q].base = s.kind == 0 ? const_cast<void*>(inputs[s.index])
                           : s.kind == 1 ? outputs[s.index]
                                         : (void*)((char*)scratch + s.index);
    }
    if (pl.spec.fn) {
      std::string err;
      if (!spec_launch(pl.spec, pl.plan, stream, err)) return fail(PN_ERR_CUDA, err);
    } else {
      const cudaError_t e = launch_plan(pl.plan, (cudaStream_t)stream);
      if (e != cudaSuccess) return fail(PN_ERR_CUDA, std::string("launch: ") + cudaGetErrorString(e));
    }
  }
  return PN_OK;
}

#pragma GCC visibility pop
}  // extern "C"
