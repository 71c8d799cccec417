// handle.h -- what a pn_graph_t is, for the files that implement the C ABI.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "graph.h"
#include "spec.h"

namespace pn {

// where the pointer behind one io entry of one launch comes from
struct IoSource { int kind; int64_t index; };   // kind 0 user input, 1 user output, 2 workspace offset

struct PlannedLaunch {
  LaunchPlan plan;
  std::vector<IoSource> src;
  SpecKernel spec;   // fn == nullptr: run the plan on the interpreter
};

// Record the calling thread's failure text (read back by pn_last_error) and pass the status on.
int fail(int status, const std::string& msg);

// Makes a device current for a scope and puts the caller's current device back afterwards, so
// that no entry point changes what the calling thread had selected.
struct DeviceScope {
  int prev = -1;
  bool switched = false;
  cudaError_t err = cudaSuccess;
  explicit DeviceScope(int device) {   // device < 0: nothing to do (a handle without a device)
    if (device < 0) return;
    err = cudaGetDevice(&prev);
    if (err == cudaSuccess && prev != device) { err = cudaSetDevice(device); switched = err == cudaSuccess; }
  }
  ~DeviceScope() { if (switched) cudaSetDevice(prev); }
  DeviceScope(const DeviceScope&) = delete;
  DeviceScope& operator=(const DeviceScope&) = delete;
};

}  // namespace pn

struct pn_graph;

namespace pn {

// The argument checks shared by every run entry point: counts, null pointers, alignment, and that
// no output overlaps an input or another output.  Returns a pn_status.
int check_run_arguments(const pn_graph* h, const void* const* inputs, int n_inputs, void* const* outputs, int n_outputs);

// Enqueue the launches of a handle on `stream` with its pointers taken from `inputs`, `outputs`
// and `workspace`; item_end > 0 restricts a single fused launch to the work items
// [item_begin, item_end).  The handle's own plan is only read.
int enqueue_launches(const pn_graph* h, const void* const* inputs, void* const* outputs, void* workspace,
                     void* stream, int64_t item_begin, int64_t item_end);

// pn_graph_run_static's set-up: the device address of the fixed scratch array on `device`
// (looked up once per device, with that device current).  Returns a pn_status.
int static_scratch_address(int device, void** out);

}  // namespace pn

struct pn_graph {
  pn::Graph g;
  unsigned flags = 0;
  int device = 0;
  int n_nodes = 0;                          // operator nodes of the descriptor (before any rewriting)
  bool plan_only = false;
  std::vector<pn::PlannedLaunch> launches;
  void* workspace = nullptr;
  size_t workspace_bytes = 0;
  void* split_ws = nullptr;                 // partials and arrival counters of split-row launches
  int64_t compulsory_bytes = 0;
  std::vector<void*> stage_in, stage_out;   // device staging of pn_graph_run_host
  void* copy_in = nullptr;                  // streams and events of the pipelined pn_graph_run_host
  void* copy_out = nullptr;                 // (cudaStream_t / cudaEvent_t, created on first use)
  std::vector<void*> pipe_events;
  uint32_t* status = nullptr;               // device word of the checked accessors (PN_FLAG_BOUNDS)
  void* static_scratch = nullptr;           // PN_FLAG_STATIC_SCRATCH: the fixed array's address on this device
};

// pn_graph_bind's result: the launches of a handle with one set of pointers filled in.
struct pn_bound {
  const pn_graph* g = nullptr;
  std::vector<pn::LaunchPlan> plans;        // copies of the handle's plans carrying the pointers
};
