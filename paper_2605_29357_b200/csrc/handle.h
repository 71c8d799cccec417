// handle.h -- what a pn_graph_t is, for the files that implement the C ABI.
#pragma once
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

}  // namespace pn

struct pn_graph {
  pn::Graph g;
  unsigned flags = 0;
  int device = 0;
  bool plan_only = false;
  std::vector<pn::PlannedLaunch> launches;
  void* workspace = nullptr;
  size_t workspace_bytes = 0;
  int64_t compulsory_bytes = 0;
  std::vector<void*> stage_in, stage_out;   // device staging of pn_graph_run_host
  void* copy_in = nullptr;                  // streams and events of the pipelined pn_graph_run_host
  void* copy_out = nullptr;                 // (cudaStream_t / cudaEvent_t, created on first use)
  std::vector<void*> pipe_events;
  uint32_t* status = nullptr;               // device word of the checked accessors (PN_FLAG_BOUNDS)
};
