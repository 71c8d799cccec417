// no_alloc.cu -- pn_graph_run_static: the unfused (one kernel per node) evaluation for
// callers that must not allocate device memory.  The intermediates between the per-node
// kernels, which pn_graph_run keeps in a workspace obtained with cudaMalloc when the handle
// is created, live here in one fixed array that is part of the library's device image.
#include <cuda_runtime.h>

#include <mutex>
#include <string>

#include "../../include/pn.h"
#include "handle.h"

using namespace pn;

// The scratch itself, at file scope.  A GPU starts holding these bytes when this file's device
// code is first loaded onto it (the set-up below, at the create of a static-scratch handle) and
// holds them until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[PN_STATIC_SCRATCH_BYTES];

namespace {

// In host code the name above is only a stand-in for the symbol: its address as a device
// pointer has to be asked for, once per device, with that device current.
constexpr int kMaxDevices = 64;
void* g_scratch_ptr[kMaxDevices] = {};
std::mutex g_setup_mutex;

}  // namespace

namespace pn {

// Set-up, called by pn_graph_create for PN_FLAG_STATIC_SCRATCH handles: the lookup may make the
// runtime load this file's device code onto the device, which is when the array's memory is
// reserved there -- so it happens at create time, where a failure can be reported, and never in
// a run.  The caller's current device is left as it was.
int static_scratch_address(int device, void** out) {
  if (device < 0 || device >= kMaxDevices) return fail(PN_ERR_DEVICE, "device ordinal out of range");
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_ptr[device]) {
    DeviceScope scope(device);
    if (scope.err != cudaSuccess) return fail(PN_ERR_CUDA, std::string("cudaSetDevice: ") + cudaGetErrorString(scope.err));
    void* ptr = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (e != cudaSuccess || !ptr) return fail(PN_ERR_CUDA, std::string("cudaGetSymbolAddress: ") + cudaGetErrorString(e));
    g_scratch_ptr[device] = ptr;
  }
  *out = g_scratch_ptr[device];
  return PN_OK;
}

}  // namespace pn

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
  // the same pointer rules as pn_graph_run: alignment, no output over an input or another output
  const pn_status st = check_run_arguments(h, inputs, n_inputs, outputs, n_outputs);
  if (st != PN_OK) return st;
  if (!h->static_scratch) return fail(PN_ERR_CUDA, "the static scratch was not set up when the handle was created");
  // Every intermediate is fully written by the kernel that produces it before any kernel
  // reads it (the launches are stream-ordered), so nothing left by an earlier call is ever
  // read and nothing needs clearing.
  return enqueue_launches(h, inputs, outputs, h->static_scratch, stream, 0, 0);
}

#pragma GCC visibility pop
}  // extern "C"
