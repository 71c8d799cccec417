// spec.h -- per-graph specialised kernels (see spec.cpp).
#pragma once
#include <string>

#include "plan.h"

namespace pn {

struct SpecKernel {
  void* fn = nullptr;     // CUfunction of the loaded kernel; owned by a process-wide cache
  int occupancy = 0;      // resident CTAs per SM at the plan's block size and shared memory
};

// True when NVRTC and the driver API could be opened (compile_only: NVRTC alone is enough);
// otherwise *why says what is missing.
bool spec_available(std::string* why, bool compile_only = false);

// Translate the plan's bytecode into a kernel, compile it for sm_100a, load it on the
// current device and re-size the plan's grid from the kernel's occupancy.
bool spec_compile(LaunchPlan& lp, int device, int sm_count, SpecKernel& out, std::string& err);

// A handle that goes away gives its kernel back: the cache may then unload it.
void spec_release(void* fn);

// Loaded modules in the cache, and how many of them a live handle uses.
void spec_cache_stats(int64_t* modules, int64_t* in_use);

// Enqueue the specialised kernel of a plan on a stream.
bool spec_launch(const SpecKernel& k, const LaunchPlan& lp, void* stream, std::string& err);

// Compile the plan's generated kernel with NVRTC and discard the result (needs no GPU).
bool spec_check(const LaunchPlan& lp, std::string& err);

// The generated part of the source, for inspection.
std::string spec_source(const LaunchPlan& lp);

}  // namespace pn
