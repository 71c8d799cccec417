// api.cpp -- the exported C ABI (see include/pn.h): handle life cycle, pointer checks,
// launches, the unfused one-kernel-per-node path, and the host-memory convenience call.
#include <cuda_runtime.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <new>
#include <string>
#include <vector>

#include "../../include/pn.h"
#include "graph.h"
#include "handle.h"
#include "spec.h"
#include "lower_common.h"

namespace pn {
cudaError_t launch_plan(const LaunchPlan& lp, cudaStream_t stream);   // kernels.cu
}

using namespace pn;

namespace {
thread_local std::string g_last_error;
}  // namespace

namespace pn {
int fail(int status, const std::string& msg) { g_last_error = msg; return status; }
}  // namespace pn

namespace {

int64_t tensor_bytes(const Tensor& t) { return t.numel() * dtype_bytes(t.dtype); }

bool any_empty(const Graph& g) {
  for (const Tensor& t : g.tensors) if (t.numel() == 0) return true;
  return false;
}

// The graph executed by one launch: the nodes `members` of g, in a topological order.  Its
// inputs are the tensors the members read that no member produces; its outputs are the tensors a
// member produces that a node outside the group reads or that are outputs of g.
void group_subgraph(const Graph& g, const std::vector<int>& members, Graph& sub, std::vector<int>& orig_of_sub) {
  sub = Graph();
  orig_of_sub.clear();
  std::vector<char> inside(g.nodes.size(), 0), made_here(g.tensors.size(), 0), read_outside(g.tensors.size(), 0);
  for (int ni : members) inside[ni] = 1;
  for (int ni : members) for (int k = 0; k < g.nodes[ni].n_out; ++k) made_here[g.nodes[ni].out[k]] = 1;
  for (size_t ni = 0; ni < g.nodes.size(); ++ni)
    if (!inside[ni])
      for (int k = 0; k < g.nodes[ni].n_in; ++k)
        if (g.nodes[ni].in[k] < g.tensors.size()) read_outside[g.nodes[ni].in[k]] = 1;
  auto add = [&](int orig) {
    for (size_t i = 0; i < orig_of_sub.size(); ++i) if (orig_of_sub[i] == orig) return (int)i;
    Tensor t = g.tensors[orig];
    // (a part of a cat result is always stored: that store is what the cat is)
    t.role = made_here[orig] ? (uint8_t)(((g.tensors[orig].role & 2) || read_outside[orig] || g.tensors[orig].embed_parent >= 0) ? 2 : 0) : (uint8_t)1;
    t.producer = -1;
    sub.tensors.push_back(t);
    orig_of_sub.push_back(orig);
    return (int)sub.tensors.size() - 1;
  };
  for (int ni : members) {
    const Node& n = g.nodes[ni];
    Node m = n;
    for (int k = 0; k < n.n_in; ++k) {
      if (n.in[k] == kImm0 || n.in[k] == kImm1) continue;
      m.in[k] = (uint32_t)add((int)n.in[k]);
    }
    for (int k = 0; k < n.n_out; ++k) {
      m.out[k] = (uint32_t)add((int)n.out[k]);
      sub.tensors[m.out[k]].producer = (int)sub.nodes.size();
    }
    sub.nodes.push_back(m);
  }
  for (size_t i = 0; i < sub.tensors.size(); ++i) {
    if (sub.tensors[i].role & 1) sub.inputs.push_back((int)i);
    if (sub.tensors[i].role & 2) sub.outputs.push_back((int)i);
  }
}

// A graph that does not fit one kernel (a bytecode, register, scalar-slot, I/O or stage budget, or
// a combination the fused lowering does not take, such as a second softmax) is cut into the
// cheapest sequence of fused launches: consecutive runs of nodes, each lowered on its own, the
// tensors that cross a cut materialised once in the workspace.  Cheapest by a two-term estimate of
// the time: the bytes every launch moves (its inputs read once, its outputs written once) at
// 6 bytes per nanosecond, plus 3 microseconds per launch -- so cuts go through per-row results and
// other small tensors, and a launch is not added to save a few kilobytes; found by dynamic
// programming over the cut positions.  Returns false when some node cannot be lowered even alone.
bool partition_graph(const Graph& g, unsigned flags, const DeviceModel& dev, std::vector<std::vector<int>>& groups) {
  const int n = (int)g.nodes.size();
  if (n < 2 || n > 512) return false;
  // The runs are taken from the nodes ordered by reduction depth (how many reductions lie between a
  // node and the graph's inputs; ties in descriptor order), which is again a topological order: a
  // kernel takes a few consecutive depths, so its runs should not be interrupted by nodes of other
  // depths that merely happen to be listed in between.
  std::vector<int> t_level(g.tensors.size(), 0), n_level(n, 0), order(n);
  for (int i = 0; i < n; ++i) {
    const Node& nd = g.nodes[i];
    int lv = 0;
    for (int k = 0; k < nd.n_in; ++k) if (nd.in[k] < g.tensors.size()) lv = std::max(lv, t_level[nd.in[k]]);
    for (int k = 0; k < nd.n_in; ++k)   // (a cat result is as deep as its deepest part)
      if (nd.in[k] < g.tensors.size() && g.tensors[nd.in[k]].assembled)
        for (const Tensor& P : g.tensors) if (P.embed_parent == (int)nd.in[k] && P.producer >= 0 && P.producer < i) lv = std::max(lv, n_level[P.producer]);
    n_level[i] = lv;
    const bool reduces = is_reduction(nd.op) || is_composite(nd.op) || is_dim_reduction(nd.op);
    for (int k = 0; k < nd.n_out; ++k) t_level[nd.out[k]] = lv + (reduces ? 1 : 0);
    order[i] = i;
  }
  // ... and among the nodes that are ready at the same depth, one that works on the shape of the node
  // listed before it comes first, so that a chain over one shape is not interleaved with a chain
  // over another (two operands of a cat, say, each with its own producers).
  {
    std::vector<int> pending(n, 0);
    std::vector<std::vector<int>> users(n);
    for (int i = 0; i < n; ++i)
      for (int k = 0; k < g.nodes[i].n_in; ++k) {
        const uint32_t t = g.nodes[i].in[k];
        if (t >= g.tensors.size()) continue;
        std::vector<int> producers;
        if (g.tensors[t].producer >= 0) producers.push_back(g.tensors[t].producer);
        if (g.tensors[t].assembled) for (const Tensor& P : g.tensors) if (P.embed_parent == (int)t && P.producer >= 0) producers.push_back(P.producer);
        for (int pr : producers) if (pr != i) { users[pr].push_back(i); pending[i]++; }
      }
    using lowering::Shape4;
    auto shape_of = [&](int i) { return lowering::align4(g.tensors[g.nodes[i].out[0]]); };
    std::vector<char> done(n, 0);
    int last = -1;
    for (int pos = 0; pos < n; ++pos) {
      int pick = -1;
      for (int i = 0; i < n; ++i) {
        if (done[i] || pending[i] > 0) continue;
        if (pick < 0) { pick = i; continue; }
        if (n_level[i] != n_level[pick]) { if (n_level[i] < n_level[pick]) pick = i; continue; }
        if (last >= 0) {
          const Shape4 sl = shape_of(last), si = shape_of(i), sp = shape_of(pick);
          const bool mi = memcmp(&sl, &si, sizeof(sl)) == 0, mp = memcmp(&sl, &sp, sizeof(sl)) == 0;
          if (mi && !mp) pick = i;
        }
      }
      if (pick < 0) return false;   // (cannot happen: the descriptor is in topological order)
      order[pos] = pick; done[pick] = 1; last = pick;
      for (int u : users[pick]) pending[u]--;
    }
  }
  const int64_t kInf = INT64_MAX / 4;
  std::vector<int64_t> best(n + 1, kInf);
  std::vector<int> from(n + 1, -1);
  best[0] = 0;
  for (int i = 0; i < n; ++i) {
    if (best[i] >= kInf) continue;
    std::vector<int> members;
    int misses = 0;
    for (int j = i; j < n; ++j) {
      members.push_back(order[j]);
      {   // a launch cannot both store a part of a cat result and read that result
        bool clash = false;
        for (int a : members)
          for (int k = 0; k < g.nodes[a].n_in && !clash; ++k) {
            const uint32_t t = g.nodes[a].in[k];
            if (t >= g.tensors.size() || !g.tensors[t].assembled) continue;
            for (int b : members) if (g.tensors[g.nodes[b].out[0]].embed_parent == (int)t) clash = true;
          }
        if (clash) { if (++misses > 24) break; continue; }
      }
      Graph sub;
      std::vector<int> orig;
      group_subgraph(g, members, sub, orig);
      LaunchPlan lp;
      std::string err;
      // A run over a budget stays over it when it grows.  A run that fails for another reason may
      // become lowerable again with a few more nodes (a tensor of a broadcast shape cannot be cut
      // at -- a launch stores only full-shape and per-row tensors -- but can stay inside a launch).
      const int st = lower_graph(sub, flags, dev, lp, err);
      if (st != PN_OK && getenv("PN_DEBUG_PARTITION")) fprintf(stderr, "partition: run [%d, %d] status %d: %s\n", i, j, st, err.c_str());
      if (st == PN_ERR_TOO_LARGE) break;
      if (st != PN_OK) { if (++misses > 24) break; continue; }
      misses = 0;
      int64_t bytes = 0;
      for (int t : sub.inputs) bytes += tensor_bytes(sub.tensors[t]);
      for (int t : sub.outputs) bytes += tensor_bytes(sub.tensors[t]);
      const int64_t cand = best[i] + bytes / 6 + 3000;   // estimated nanoseconds
      if (cand < best[j + 1]) { best[j + 1] = cand; from[j + 1] = i; }
    }
  }
  if (best[n] >= kInf) return false;
  groups.clear();
  for (int j = n; j > 0; j = from[j]) {
    std::vector<int> m;
    for (int k = from[j]; k < j; ++k) m.push_back(order[k]);
    groups.insert(groups.begin(), m);
  }
  if (getenv("PN_DEBUG_PARTITION"))
    for (size_t k = 0; k < groups.size(); ++k) {
      std::string line = "partition: launch " + std::to_string(k) + " = nodes";
      for (int m : groups[k]) line += " " + std::to_string(m);
      fprintf(stderr, "%s\n", line.c_str());
    }
  return groups.size() > 1;
}

pn_status check_counts(const pn_graph* h, const void* const* inputs, int n_inputs, void* const* outputs, int n_outputs) {
  if (!h || (!inputs && n_inputs > 0) || !outputs) return fail(PN_ERR_INVALID_ARG, "null argument");
  if (h->plan_only) return fail(PN_ERR_DEVICE, "handle was created with PN_FLAG_PLAN_ONLY");
  if (n_inputs != (int)h->g.inputs.size() || n_outputs != (int)h->g.outputs.size())
    return fail(PN_ERR_COUNT, "expected " + std::to_string(h->g.inputs.size()) + " inputs and " +
                                  std::to_string(h->g.outputs.size()) + " outputs");
  return PN_OK;
}

void fill_pointers(const pn_graph* h, const PlannedLaunch& pl, const void* const* inputs, void* const* outputs, void* workspace, LaunchPlan& lp) {
  for (int q = 0; q < lp.p.n_io; ++q) {
    const IoSource& s = pl.src[q];
    char* base = s.kind == 0 ? (char*)const_cast<void*>(inputs[s.index])
               : s.kind == 1 ? (char*)outputs[s.index]
                             : (char*)workspace + s.index;
    lp.p.io[q].base = base + lp.io_offset[q] * dtype_bytes(lp.p.io[q].dtype);
  }
  (void)h;
}

pn_status launch_filled(const PlannedLaunch& pl, const LaunchPlan& lp, void* stream) {
  if (pl.spec.fn) {
    std::string err;
    if (!spec_launch(pl.spec, lp, stream, err)) return fail(PN_ERR_CUDA, err);
  } else {
    const cudaError_t e = launch_plan(lp, (cudaStream_t)stream);
    if (e != cudaSuccess) return fail(PN_ERR_CUDA, std::string("launch: ") + cudaGetErrorString(e));
  }
  return PN_OK;
}

}  // namespace

namespace pn {

int check_run_arguments(const pn_graph* h, const void* const* inputs, int n_inputs, void* const* outputs, int n_outputs) {
  const pn_status st = check_counts(h, inputs, n_inputs, outputs, n_outputs);
  if (st != PN_OK) return st;
  const Graph& g = h->g;
  const bool scalar = (h->flags & PN_FLAG_FORCE_SCALAR) != 0;
  for (int i = 0; i < n_inputs; ++i) {
    if (!inputs[i]) return fail(PN_ERR_INVALID_ARG, "input " + std::to_string(i) + " is null");
    const uintptr_t m = scalar ? (uintptr_t)(dtype_bytes(g.tensors[g.inputs[i]].dtype) - 1) : 15;
    if ((uintptr_t)inputs[i] & m) return fail(PN_ERR_ALIGNMENT, "input " + std::to_string(i) + " is not aligned");
  }
  for (int i = 0; i < n_outputs; ++i) {
    if (!outputs[i]) return fail(PN_ERR_INVALID_ARG, "output " + std::to_string(i) + " is null");
    const uintptr_t m = scalar ? (uintptr_t)(dtype_bytes(g.tensors[g.outputs[i]].dtype) - 1) : 15;
    if ((uintptr_t)outputs[i] & m) return fail(PN_ERR_ALIGNMENT, "output " + std::to_string(i) + " is not aligned");
  }
  // inputs go through the read-only data path: none may overlap an output; outputs are
  // written independently: none may overlap another
  for (int o = 0; o < n_outputs; ++o) {
    const char* b0 = (const char*)outputs[o];
    const char* b1 = b0 + tensor_bytes(g.tensors[g.outputs[o]]);
    for (int i = 0; i < n_inputs; ++i) {
      const char* a0 = (const char*)inputs[i];
      const char* a1 = a0 + tensor_bytes(g.tensors[g.inputs[i]]);
      if (a0 < b1 && b0 < a1) return fail(PN_ERR_INVALID_ARG, "input " + std::to_string(i) + " overlaps output " + std::to_string(o));
    }
    for (int i = 0; i < o; ++i) {
      const char* a0 = (const char*)outputs[i];
      const char* a1 = a0 + tensor_bytes(g.tensors[g.outputs[i]]);
      if (a0 < b1 && b0 < a1) return fail(PN_ERR_INVALID_ARG, "outputs " + std::to_string(i) + " and " + std::to_string(o) + " overlap");
    }
  }
  return PN_OK;
}

int enqueue_launches(const pn_graph* h, const void* const* inputs, void* const* outputs, void* workspace,
                     void* stream, int64_t item_begin, int64_t item_end) {
  DeviceScope dev(h->device);
  if (dev.err != cudaSuccess) return fail(PN_ERR_CUDA, std::string("cudaSetDevice: ") + cudaGetErrorString(dev.err));
  for (const PlannedLaunch& pl : h->launches) {
    LaunchPlan lp = pl.plan;   // the pointers go into a copy: the handle itself is only read
    fill_pointers(h, pl, inputs, outputs, workspace, lp);
    if (item_end > 0) { lp.p.item_begin = item_begin; lp.p.item_end = item_end; }
    const pn_status st = launch_filled(pl, lp, stream);
    if (st != PN_OK) return st;
  }
  return PN_OK;
}

}  // namespace pn

extern "C" {
#pragma GCC visibility push(default)

pn_status pn_graph_create(const void* desc, size_t desc_bytes, int device, unsigned flags, pn_graph_t** out) {
  if (out) *out = nullptr;
  if (!desc || !out) return fail(PN_ERR_INVALID_ARG, "null argument");
  pn_graph* h = new (std::nothrow) pn_graph();
  if (!h) return fail(PN_ERR_INVALID_ARG, "out of host memory");
  std::string err;
  int st = parse_descriptor(desc, desc_bytes, h->g, err);
  if (st != PN_OK) { delete h; return fail(st, err); }
  h->n_nodes = (int)h->g.nodes.size();
  st = expand_concatenations(h->g, err);   // a cat of several operands becomes stores into blocks of its result
  if (st != PN_OK) { delete h; return fail(st, err); }
  prune_dead_nodes(h->g);                  // what reaches no output is not part of f_G
  if ((flags & PN_FLAG_BOUNDS) && (flags & PN_FLAG_STATIC_SCRATCH)) { delete h; return fail(PN_ERR_INVALID_ARG, "PN_FLAG_BOUNDS allocates a status word: it cannot be combined with PN_FLAG_STATIC_SCRATCH"); }
  h->flags = flags;
  h->device = device;
  h->plan_only = (flags & PN_FLAG_PLAN_ONLY) != 0;

  // The kernels specialised per graph need NVRTC (and, to be loaded, the driver library).  A create
  // that cannot have them fails rather than fall back silently to the interpreter, which is an
  // order of magnitude slower: the caller has to ask for the interpreter by name.
  DeviceModel dev;
  std::string why;
  dev.specialise = !(flags & PN_FLAG_INTERPRET) && spec_available(&why, h->plan_only);
  if (!dev.specialise && !(flags & (PN_FLAG_INTERPRET | PN_FLAG_ALLOW_INTERPRET))) {
    delete h;
    return fail(PN_ERR_DEVICE, "kernels cannot be specialised for this graph: " + why +
                                   " (PN_FLAG_ALLOW_INTERPRET accepts the much slower built-in interpreter kernels instead)");
  }
  if (!h->plan_only) {
    int count = 0;
    cudaError_t e = cudaGetDeviceCount(&count);
    if (e != cudaSuccess || device < 0 || device >= count) { delete h; return fail(PN_ERR_DEVICE, "no such CUDA device"); }
    cudaDeviceProp prop;
    e = cudaGetDeviceProperties(&prop, device);
    if (e != cudaSuccess) { delete h; return fail(PN_ERR_CUDA, cudaGetErrorString(e)); }
    if (prop.major != 10) { delete h; return fail(PN_ERR_DEVICE, "the kernels are built for sm_100a only"); }
    dev.sm_count = prop.multiProcessorCount;
    dev.max_smem_per_block = (int)prop.sharedMemPerBlockOptin;
    dev.have_device = true;
  }
  // everything below that touches the device does so with it current; the caller's own current
  // device is put back when this function returns
  DeviceScope scope(h->plan_only ? -1 : device);
  if (!h->plan_only && scope.err != cudaSuccess) { delete h; return fail(PN_ERR_CUDA, std::string("cudaSetDevice: ") + cudaGetErrorString(scope.err)); }

  const Graph& g = h->g;
  for (int t : g.inputs) h->compulsory_bytes += tensor_bytes(g.tensors[t]);
  for (int t : g.outputs) h->compulsory_bytes += tensor_bytes(g.tensors[t]);
  if (any_empty(g)) { *out = h; return PN_OK; }   // nothing to compute: runs are no-ops

  // ---- which nodes run in which launch -----------------------------------------------------------
  std::vector<std::vector<int>> groups;
  if (flags & PN_FLAG_UNFUSED) {
    for (size_t ni = 0; ni < g.nodes.size(); ++ni) groups.push_back({(int)ni});   // one launch per node
  } else {
    groups.emplace_back();
    for (size_t ni = 0; ni < g.nodes.size(); ++ni) groups[0].push_back((int)ni);
    // does the whole graph fit one kernel?  If a budget or an unsupported combination says no, cut it
    // into the cheapest sequence of fused launches (PN_FLAG_ONE_KERNEL asks for the refusal instead)
    LaunchPlan probe;
    std::string why_not;
    bool any_assembled = false;
    for (const Tensor& T : g.tensors) any_assembled = any_assembled || T.assembled;
    int whole;
    if (any_assembled) {   // (the cat results themselves take no part in a launch: only their parts do)
      Graph sub;
      std::vector<int> orig;
      group_subgraph(g, groups[0], sub, orig);
      whole = lower_graph(sub, flags, dev, probe, why_not);
    } else whole = lower_graph(g, flags, dev, probe, why_not);
    // a cat result is complete only when the launches that store its parts are done: a node that
    // reads it cannot share a launch with them
    for (const Node& nd : g.nodes)
      for (int k = 0; k < nd.n_in; ++k)
        if (nd.in[k] < g.tensors.size() && g.tensors[nd.in[k]].assembled && whole == PN_OK) { whole = PN_ERR_UNSUPPORTED_OP; why_not = "a cat result is read inside the graph"; }
    if (whole == PN_ERR_SHAPE && any_assembled) whole = PN_ERR_UNSUPPORTED_OP;   // parts of different shapes: one launch each
    if ((whole == PN_ERR_TOO_LARGE || whole == PN_ERR_UNSUPPORTED_OP) && !(flags & PN_FLAG_ONE_KERNEL)) {
      std::vector<std::vector<int>> cut;
      if (partition_graph(g, flags, dev, cut)) groups.swap(cut);
    }
  }
  // tensors that cross from one launch to a later one live in a workspace, in their declared dtype
  std::vector<int> group_of_node(g.nodes.size(), 0);
  for (size_t gi = 0; gi < groups.size(); ++gi) for (int ni : groups[gi]) group_of_node[ni] = (int)gi;
  std::vector<int64_t> ws_off(g.tensors.size(), -1);
  size_t ws = 0;
  for (size_t t = 0; t < g.tensors.size(); ++t) {
    const Tensor& T = g.tensors[t];
    if (T.role != 0 || T.embed_parent >= 0) continue;          // the caller's buffers; parts live in their parent
    bool stored = T.assembled;                                  // a cat result is always materialised
    if (!stored && T.producer >= 0 && groups.size() > 1)
      for (size_t ni = 0; ni < g.nodes.size() && !stored; ++ni)
        for (int k = 0; k < g.nodes[ni].n_in; ++k)
          if (g.nodes[ni].in[k] == t && group_of_node[ni] != group_of_node[T.producer]) stored = true;
    if (!stored) continue;
    ws_off[t] = (int64_t)ws;
    ws += ((size_t)tensor_bytes(T) + 255) / 256 * 256;
  }
  for (size_t gi = 0; gi < groups.size(); ++gi) {
    PlannedLaunch pl;
    std::vector<int> orig;
    bool plain_whole = groups.size() == 1;
    for (const Tensor& T : g.tensors) plain_whole = plain_whole && !T.assembled;
    if (plain_whole) {
      st = lower_graph(g, flags, dev, pl.plan, err);
      for (size_t t = 0; t < g.tensors.size(); ++t) orig.push_back((int)t);
    } else {
      Graph sub;
      group_subgraph(g, groups[gi], sub, orig);
      st = lower_graph(sub, flags, dev, pl.plan, err);
      if (st != PN_OK) err = (groups[gi].size() == 1 ? "node " + std::to_string(groups[gi][0]) + " (unfused): " : "launch " + std::to_string(gi) + ": ") + err;
    }
    if (st != PN_OK) { delete h; return fail(st, err); }
    for (int q = 0; q < pl.plan.p.n_io; ++q) {
      int t = orig[pl.plan.io_tensor[q]];
      pl.plan.p.io[q].numel = g.tensors[t].numel() - (pl.plan.io_is_output[q] ? 0 : pl.plan.io_offset[q]);   // (an input sliced along the last dimension starts later)
      if (pl.plan.io_is_output[q] && g.tensors[t].embed_parent >= 0) {   // a part of a cat result: stored inside it
        t = g.tensors[t].embed_parent;
        pl.plan.p.io[q].numel = g.tensors[t].numel() - pl.plan.io_offset[q];
      }
      IoSource s{2, ws_off[t]};
      // a tensor that is both read and written by the graph's caller (an input passed through) is
      // looked up on the side this launch uses it on
      if (!pl.plan.io_is_output[q]) for (size_t i = 0; i < g.inputs.size(); ++i) if (g.inputs[i] == t) s = IoSource{0, (int64_t)i};
      if (pl.plan.io_is_output[q] || s.kind == 2) for (size_t i = 0; i < g.outputs.size(); ++i) if (g.outputs[i] == t) s = IoSource{1, (int64_t)i};
      if (s.kind == 2 && s.index < 0) { delete h; return fail(PN_ERR_INVALID_ARG, "internal: a tensor between two launches has no storage"); }
      pl.src.push_back(s);
    }
    h->launches.push_back(pl);
  }
  h->workspace_bytes = ws;
  if (!h->plan_only && ws > 0 && !(flags & PN_FLAG_STATIC_SCRATCH)) {
    cudaError_t e = cudaMalloc(&h->workspace, ws);
    if (e != cudaSuccess) { delete h; return fail(PN_ERR_CUDA, std::string("workspace: ") + cudaGetErrorString(e)); }
  }
  // a handle that will run from the fixed scratch array: its address on this device is looked up
  // now, at set-up, so that the runs themselves only read it
  if (!h->plan_only && (flags & PN_FLAG_STATIC_SCRATCH)) {
    st = static_scratch_address(device, &h->static_scratch);
    if (st != PN_OK) { delete h; return st; }
  }
  if (flags & PN_FLAG_PLAIN_LAUNCH) for (PlannedLaunch& pl : h->launches) pl.plan.plain_launch = 1;
  // checked accessors: one status word on the device, shared by the launches of the handle
  if (flags & PN_FLAG_BOUNDS) {
    for (PlannedLaunch& pl : h->launches) pl.plan.bounds = 1;
    if (!h->plan_only) {
      cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&h->status), sizeof(uint32_t));
      if (e == cudaSuccess) e = cudaMemset(h->status, 0, sizeof(uint32_t));
      if (e != cudaSuccess) { pn_graph_destroy(h); return fail(PN_ERR_CUDA, std::string("status word: ") + cudaGetErrorString(e)); }
      for (PlannedLaunch& pl : h->launches) pl.plan.p.status = h->status;
    }
  }
  // a kernel of its own for every launch, unless the interpreter was asked for
  if (!h->plan_only && dev.specialise) {
    cudaFree(0);   // makes the device's primary context current for the driver calls
    for (PlannedLaunch& pl : h->launches)
      if (!spec_compile(pl.plan, device, dev.sm_count, pl.spec, err)) {
        pn_graph_destroy(h);
        return fail(PN_ERR_CUDA, err);
      }
  }
  // split-row launches: partials and arrival counters in device memory of the handle, the counters
  // zero at rest
  {
    auto uses_tickets = [](const LaunchPlan& lp) { return lp.family == FAM_SPLIT || (lp.family == FAM_COLUMN && lp.p.splits > 1); };
    auto sizes = [](const LaunchPlan& lp, size_t& part_bytes, size_t& ticket_bytes) {
      const KernelParams& P = lp.p;
      if (lp.family == FAM_SPLIT) {   // a partial (three floats) per reduction, slice and row; a counter per row
        part_bytes = (size_t)P.rows * P.splits * P.stage[0].n_red * 3 * sizeof(float);
        ticket_bytes = (size_t)P.rows * sizeof(uint32_t);
      } else {                        // column family: the accumulators of a column tile per slice; a counter per item
        const size_t items = (size_t)P.rows * P.chunks;
        part_bytes = items * P.splits * P.stage[0].n_red * ((size_t)P.col_tx * lp.vl * lp.ng) * sizeof(float);
        ticket_bytes = items * sizeof(uint32_t);
      }
      part_bytes = (part_bytes + 255) / 256 * 256;
      ticket_bytes = (ticket_bytes + 255) / 256 * 256;
    };
    size_t need = 0;
    for (PlannedLaunch& pl : h->launches)
      if (uses_tickets(pl.plan)) { size_t a = 0, b = 0; sizes(pl.plan, a, b); need += a + b; }
    if (need > 0 && !h->plan_only) {
      cudaError_t e = cudaMalloc(&h->split_ws, need);
      if (e == cudaSuccess) e = cudaMemset(h->split_ws, 0, need);
      if (e != cudaSuccess) { pn_graph_destroy(h); return fail(PN_ERR_CUDA, std::string("split-row workspace: ") + cudaGetErrorString(e)); }
      size_t off = 0;
      for (PlannedLaunch& pl : h->launches)
        if (uses_tickets(pl.plan)) {
          size_t a = 0, b = 0;
          sizes(pl.plan, a, b);
          pl.plan.p.split_part = reinterpret_cast<float*>((char*)h->split_ws + off); off += a;
          pl.plan.p.split_ticket = reinterpret_cast<uint32_t*>((char*)h->split_ws + off); off += b;
        }
    }
    h->workspace_bytes += need;
  }
  *out = h;
  return PN_OK;
}

pn_status pn_graph_run(pn_graph_t* h, const void* const* inputs, int n_inputs, void* const* outputs,
                       int n_outputs, void* stream) {
  pn_status st = check_counts(h, inputs, n_inputs, outputs, n_outputs);
  if (st != PN_OK) return st;
  if (h->flags & PN_FLAG_STATIC_SCRATCH)
    return fail(PN_ERR_INVALID_ARG, "this handle owns no workspace: run it with pn_graph_run_static");
  if (any_empty(h->g)) return PN_OK;   // nothing to compute
  st = check_run_arguments(h, inputs, n_inputs, outputs, n_outputs);
  if (st != PN_OK) return st;
  return enqueue_launches(h, inputs, outputs, h->workspace, stream, 0, 0);
}

pn_status pn_graph_bind(pn_graph_t* h, const void* const* inputs, int n_inputs, void* const* outputs, int n_outputs,
                        pn_bound_t** out) {
  if (out) *out = nullptr;
  if (!out) return fail(PN_ERR_INVALID_ARG, "null argument");
  pn_status st = check_counts(h, inputs, n_inputs, outputs, n_outputs);
  if (st != PN_OK) return st;
  if (h->flags & PN_FLAG_STATIC_SCRATCH) return fail(PN_ERR_INVALID_ARG, "static-scratch handles are run with pn_graph_run_static");
  if (!any_empty(h->g)) {
    st = check_run_arguments(h, inputs, n_inputs, outputs, n_outputs);
    if (st != PN_OK) return st;
  }
  pn_bound* b = new (std::nothrow) pn_bound();
  if (!b) return fail(PN_ERR_INVALID_ARG, "out of host memory");
  b->g = h;
  if (!any_empty(h->g))
    for (const PlannedLaunch& pl : h->launches) {
      b->plans.push_back(pl.plan);
      fill_pointers(h, pl, inputs, outputs, h->workspace, b->plans.back());
    }
  *out = b;
  return PN_OK;
}

pn_status pn_bound_run(pn_bound_t* b, void* stream) {
  if (!b || !b->g) return fail(PN_ERR_INVALID_ARG, "null argument");
  const pn_graph* h = b->g;
  DeviceScope dev(h->device);
  if (dev.err != cudaSuccess) return fail(PN_ERR_CUDA, std::string("cudaSetDevice: ") + cudaGetErrorString(dev.err));
  for (size_t i = 0; i < b->plans.size(); ++i) {
    const pn_status st = launch_filled(h->launches[i], b->plans[i], stream);
    if (st != PN_OK) return st;
  }
  return PN_OK;
}

pn_status pn_bound_run_many(pn_bound_t* const* bound, int n, void* stream) {
  if (n < 0 || (n > 0 && !bound)) return fail(PN_ERR_INVALID_ARG, "null argument");
  for (int i = 0; i < n; ++i)
    if (!bound[i] || !bound[i]->g) return fail(PN_ERR_INVALID_ARG, "bound object " + std::to_string(i) + " is null");
  int current = -2;   // the device made current so far (-2: none yet); the caller's is put back at the end
  int callers = 0;
  cudaError_t e = n > 0 ? cudaGetDevice(&callers) : cudaSuccess;
  if (e != cudaSuccess) return fail(PN_ERR_CUDA, std::string("cudaGetDevice: ") + cudaGetErrorString(e));
  pn_status st = PN_OK;
  for (int i = 0; i < n && st == PN_OK; ++i) {
    const pn_graph* h = bound[i]->g;
    if (h->device != current && !(current == -2 && h->device == callers)) {
      e = cudaSetDevice(h->device);
      if (e != cudaSuccess) { st = fail(PN_ERR_CUDA, std::string("cudaSetDevice: ") + cudaGetErrorString(e)); break; }
    }
    current = h->device;
    for (size_t k = 0; k < bound[i]->plans.size() && st == PN_OK; ++k) st = launch_filled(h->launches[k], bound[i]->plans[k], stream);
  }
  if (current >= 0 && current != callers) cudaSetDevice(callers);
  return st;
}

pn_status pn_bound_destroy(pn_bound_t* b) {
  delete b;
  return PN_OK;
}

pn_status pn_graph_run_host(pn_graph_t* h, const void* const* inputs, int n_inputs, void* const* outputs,
                            int n_outputs, void* stream) {
  pn_status st = check_counts(h, inputs, n_inputs, outputs, n_outputs);
  if (st != PN_OK) return st;
  if (h->flags & PN_FLAG_STATIC_SCRATCH)   // before anything is allocated for it
    return fail(PN_ERR_INVALID_ARG, "this handle owns no workspace and may not allocate: run it with pn_graph_run_static on device buffers");
  const Graph& g = h->g;
  if (any_empty(g)) return PN_OK;
  DeviceScope dev(h->device);
  if (dev.err != cudaSuccess) return fail(PN_ERR_CUDA, std::string("cudaSetDevice: ") + cudaGetErrorString(dev.err));
  cudaStream_t s = (cudaStream_t)stream;
  cudaError_t e;
  if (h->stage_in.empty() && h->stage_out.empty()) {
    for (int pass = 0; pass < 2; ++pass)
      for (int t : pass == 0 ? g.inputs : g.outputs) {
        void* p = nullptr;
        e = cudaMalloc(&p, std::max<size_t>((size_t)tensor_bytes(g.tensors[t]), 16));
        if (e != cudaSuccess) return fail(PN_ERR_CUDA, std::string("staging: ") + cudaGetErrorString(e));
        (pass == 0 ? h->stage_in : h->stage_out).push_back(p);
      }
  }
  for (int i = 0; i < n_inputs; ++i) if (!inputs[i]) return fail(PN_ERR_INVALID_ARG, "input " + std::to_string(i) + " is null");
  for (int i = 0; i < n_outputs; ++i) if (!outputs[i]) return fail(PN_ERR_INVALID_ARG, "output " + std::to_string(i) + " is null");

  // ---- can the work be cut into pieces along its outermost dimension? ----------------------
  // A fused launch walks its work items in order of the outermost leading dimension, and every
  // dense tensor that has that dimension holds one contiguous slab per index of it.  Then the copy
  // in of piece k + 1, the kernel on piece k and the copy out of piece k - 1 run at the same time
  // (the two copy directions use the link in both directions at once).
  struct Cut { int64_t outer = 0, items_per_outer = 0; std::vector<int64_t> stride; } cut;   // stride in elements per outer index; 0 = whole tensor
  int64_t in_bytes = 0;
  for (int t : g.inputs) in_bytes += tensor_bytes(g.tensors[t]);
  if (h->launches.size() == 1 && in_bytes >= (8ll << 20)) {
    const LaunchPlan& lp = h->launches[0].plan;
    const KernelParams& P = lp.p;
    bool ok = P.cluster >= 1 && P.family != FAM_SPLIT && P.splits <= 1;   // (kernels with arrival counters run whole)
    for (int q = 0; q < P.n_io; ++q) ok = ok && !P.io[q].mapped;
    cut.stride.assign(P.n_io, 0);
    if (ok && P.family == FAM_COLUMN) {
      cut.outer = P.rows; cut.items_per_outer = P.chunks;
      for (int q = 0; q < P.n_io; ++q) cut.stride[q] = P.io[q].lead_stride[2];
    } else if (ok && P.split_chunks && P.rows == 1) {
      const int64_t chunk_cols = 32ll * lp.vl * lp.ng;
      cut.outer = P.chunks; cut.items_per_outer = 1;
      for (int q = 0; q < P.n_io; ++q) cut.stride[q] = P.io[q].col_stride ? chunk_cols : 0;
    } else if (ok) {
      int d0 = -1;
      for (int i = 0; i < 3 && d0 < 0; ++i) if (P.lead_dim[i] > 1) d0 = i;
      if (d0 >= 0) {
        cut.outer = P.lead_dim[d0];
        cut.items_per_outer = P.rows / cut.outer * (P.split_chunks ? P.chunks : 1);
        for (int q = 0; q < P.n_io; ++q) cut.stride[q] = P.io[q].lead_stride[d0];
      }
    }
    for (int q = 0; q < P.n_io && cut.outer > 0; ++q)
      if (h->launches[0].src[q].kind == 1 && cut.stride[q] == 0) cut.outer = 0;   // an output without the outer dimension
  }
  const int pieces = (int)std::min<int64_t>(std::min<int64_t>(cut.outer, 16), std::max<int64_t>(1, in_bytes / (24ll << 20)));
  if (pieces < 2) {   // plain: copy in, run, copy out
    for (int i = 0; i < n_inputs; ++i) {
      e = cudaMemcpyAsync(h->stage_in[i], inputs[i], (size_t)tensor_bytes(g.tensors[g.inputs[i]]), cudaMemcpyHostToDevice, s);
      if (e != cudaSuccess) return fail(PN_ERR_CUDA, std::string("copy in: ") + cudaGetErrorString(e));
    }
    st = pn_graph_run(h, (const void* const*)h->stage_in.data(), n_inputs, h->stage_out.data(), n_outputs, stream);
    if (st != PN_OK) return st;
    for (int i = 0; i < n_outputs; ++i) {
      e = cudaMemcpyAsync(outputs[i], h->stage_out[i], (size_t)tensor_bytes(g.tensors[g.outputs[i]]), cudaMemcpyDeviceToHost, s);
      if (e != cudaSuccess) return fail(PN_ERR_CUDA, std::string("copy out: ") + cudaGetErrorString(e));
    }
    e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return fail(PN_ERR_CUDA, std::string("sync: ") + cudaGetErrorString(e));
    return PN_OK;
  }

  // ---- pipelined: copy-in stream, the caller's stream for the kernels, copy-out stream -----------
  if (!h->copy_in) {
    cudaStream_t a = nullptr, b = nullptr;
    e = cudaStreamCreateWithFlags(&a, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&b, cudaStreamNonBlocking);
    if (e != cudaSuccess) { if (a) cudaStreamDestroy(a); return fail(PN_ERR_CUDA, std::string("copy streams: ") + cudaGetErrorString(e)); }
    h->copy_in = a; h->copy_out = b;
  }
  while ((int)h->pipe_events.size() < 2 * pieces + 1) {
    cudaEvent_t ev = nullptr;
    e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
    if (e != cudaSuccess) return fail(PN_ERR_CUDA, std::string("events: ") + cudaGetErrorString(e));
    h->pipe_events.push_back(ev);
  }
  cudaStream_t s_in = (cudaStream_t)h->copy_in, s_out = (cudaStream_t)h->copy_out;
  const PlannedLaunch& pl = h->launches[0];
  auto ev = [&](int i) { return (cudaEvent_t)h->pipe_events[i]; };
  auto check = [&](cudaError_t err, const char* what) { return err == cudaSuccess ? PN_OK : fail(PN_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(err)); };
  // what the caller queued on its stream comes first
  if ((st = check(cudaEventRecord(ev(2 * pieces), s), "event")) != PN_OK) return st;
  if ((st = check(cudaStreamWaitEvent(s_in, ev(2 * pieces), 0), "wait")) != PN_OK) return st;
  // tensors without the outer dimension: whole, before the first piece
  for (int q = 0; q < pl.plan.p.n_io; ++q) {
    const IoSource& src = pl.src[q];
    if (src.kind != 0 || cut.stride[q] != 0) continue;
    e = cudaMemcpyAsync(h->stage_in[src.index], inputs[src.index], (size_t)tensor_bytes(g.tensors[g.inputs[src.index]]), cudaMemcpyHostToDevice, s_in);
    if ((st = check(e, "copy in")) != PN_OK) return st;
  }
  pn_status result = PN_OK;
  for (int k = 0; k < pieces && result == PN_OK; ++k) {
    const int64_t a = cut.outer * k / pieces, b = cut.outer * (k + 1) / pieces;
    for (int q = 0; q < pl.plan.p.n_io && result == PN_OK; ++q) {
      const IoSource& src = pl.src[q];
      if (src.kind != 0 || cut.stride[q] == 0) continue;
      const Tensor& T = g.tensors[g.inputs[src.index]];
      const int64_t es = dtype_bytes(T.dtype), lo = a * cut.stride[q], hi = std::min<int64_t>(b * cut.stride[q], T.numel());
      if (hi > lo) result = check(cudaMemcpyAsync((char*)h->stage_in[src.index] + lo * es, (const char*)inputs[src.index] + lo * es, (size_t)((hi - lo) * es), cudaMemcpyHostToDevice, s_in), "copy in");
    }
    if (result == PN_OK) result = check(cudaEventRecord(ev(2 * k), s_in), "event");
    if (result == PN_OK) result = check(cudaStreamWaitEvent(s, ev(2 * k), 0), "wait");
    if (result != PN_OK) break;
    result = enqueue_launches(h, (const void* const*)h->stage_in.data(), h->stage_out.data(), h->workspace, stream,
                              a * cut.items_per_outer, b * cut.items_per_outer);
    if (result == PN_OK) result = check(cudaEventRecord(ev(2 * k + 1), s), "event");
    if (result == PN_OK) result = check(cudaStreamWaitEvent(s_out, ev(2 * k + 1), 0), "wait");
    for (int q = 0; q < pl.plan.p.n_io && result == PN_OK; ++q) {
      const IoSource& src = pl.src[q];
      if (src.kind != 1) continue;
      const Tensor& T = g.tensors[g.outputs[src.index]];
      const int64_t es = dtype_bytes(T.dtype), lo = a * cut.stride[q], hi = std::min<int64_t>(b * cut.stride[q], T.numel());
      if (hi > lo) result = check(cudaMemcpyAsync((char*)outputs[src.index] + lo * es, (const char*)h->stage_out[src.index] + lo * es, (size_t)((hi - lo) * es), cudaMemcpyDeviceToHost, s_out), "copy out");
    }
  }
  // wait for everything that was queued, also after a failure
  cudaStreamSynchronize(s_in);
  e = cudaStreamSynchronize(s);
  const cudaError_t e2 = cudaStreamSynchronize(s_out);
  if (result != PN_OK) return result;
  if (e != cudaSuccess || e2 != cudaSuccess) return fail(PN_ERR_CUDA, std::string("sync: ") + cudaGetErrorString(e != cudaSuccess ? e : e2));
  return PN_OK;
}

pn_status pn_graph_destroy(pn_graph_t* h) {
  if (!h) return PN_OK;
  if (!h->plan_only) {
    DeviceScope scope(h->device);
    for (PlannedLaunch& pl : h->launches) spec_release(pl.spec.fn);   // the kernel cache may unload what nobody uses
    if (h->workspace) cudaFree(h->workspace);
    if (h->split_ws) cudaFree(h->split_ws);
    if (h->status) cudaFree(h->status);
    if (h->copy_in) cudaStreamDestroy((cudaStream_t)h->copy_in);
    if (h->copy_out) cudaStreamDestroy((cudaStream_t)h->copy_out);
    for (void* ev : h->pipe_events) cudaEventDestroy((cudaEvent_t)ev);
    for (void* p : h->stage_in) cudaFree(p);
    for (void* p : h->stage_out) cudaFree(p);
  }
  delete h;
  return PN_OK;
}

pn_status pn_graph_query(const pn_graph_t* h, int what, void* out, size_t out_bytes) {
  if (!h || !out) return fail(PN_ERR_INVALID_ARG, "null argument");
  const Graph& g = h->g;
  std::vector<int64_t> v;
  auto meta = [&](const std::vector<int>& ids) {
    for (int t : ids) {
      const Tensor& T = g.tensors[t];
      v.push_back(T.dtype); v.push_back(T.rank);
      for (int d = 0; d < 4; ++d) v.push_back(d < T.rank ? T.dims[d] : 0);
    }
  };
  switch (what) {
    case PN_Q_N_INPUTS: v.push_back((int64_t)g.inputs.size()); break;
    case PN_Q_N_OUTPUTS: v.push_back((int64_t)g.outputs.size()); break;
    case PN_Q_INPUT_META: meta(g.inputs); break;
    case PN_Q_OUTPUT_META: meta(g.outputs); break;
    case PN_Q_COMPULSORY_BYTES: v.push_back(h->compulsory_bytes); break;
    case PN_Q_N_KERNELS: v.push_back((int64_t)h->launches.size()); break;
    case PN_Q_N_NODES: v.push_back((int64_t)h->n_nodes); break;
    case PN_Q_WORKSPACE_BYTES: v.push_back((int64_t)h->workspace_bytes); break;
    case PN_Q_KERNEL_INFO:
      for (const PlannedLaunch& pl : h->launches) {
        const LaunchPlan& p = pl.plan;
        const int64_t row[14] = {p.family, p.grid, p.block, p.p.cluster, p.smem_bytes, p.vl, p.ng, p.p.chunks,
                                 p.code_words, p.p.n_stages, p.p.rows, p.p.row_len, p.specialised, p.p.splits};
        v.insert(v.end(), row, row + 14);
      }
      break;
    case PN_Q_BOUNDS_STATUS: {
      if (!(h->flags & PN_FLAG_BOUNDS) || !h->status) return fail(PN_ERR_INVALID_ARG, "the handle was not created with PN_FLAG_BOUNDS on a device");
      uint32_t w = 0;
      const cudaError_t e = cudaMemcpy(&w, h->status, sizeof(w), cudaMemcpyDeviceToHost);   // waits for the device
      if (e != cudaSuccess) return fail(PN_ERR_CUDA, std::string("status word: ") + cudaGetErrorString(e));
      v.push_back((int64_t)w);
      break;
    }
    case PN_Q_KERNEL_CACHE: {
      int64_t modules = 0, in_use = 0;
      spec_cache_stats(&modules, &in_use);
      v.push_back(modules); v.push_back(in_use);
      break;
    }
    default: return fail(PN_ERR_INVALID_ARG, "unknown query");
  }
  if (out_bytes < v.size() * sizeof(int64_t)) return fail(PN_ERR_INVALID_ARG, "query buffer too small");
  if (!v.empty()) memcpy(out, v.data(), v.size() * sizeof(int64_t));
  return PN_OK;
}

pn_status pn_graph_codegen(const pn_graph_t* h, int kernel, int compile, char* out, size_t out_bytes, size_t* needed) {
  if (!h) return fail(PN_ERR_INVALID_ARG, "null argument");
  if (kernel < 0 || kernel >= (int)h->launches.size()) return fail(PN_ERR_INVALID_ARG, "no such kernel");
  const LaunchPlan& lp = h->launches[kernel].plan;
  const std::string src = spec_source(lp);
  if (needed) *needed = src.size();
  if (out && out_bytes > 0) {
    const size_t n = std::min(src.size(), out_bytes - 1);
    memcpy(out, src.data(), n);
    out[n] = '\0';
  }
  if (compile) {
    std::string err;
    if (!spec_check(lp, err)) return fail(PN_ERR_CUDA, err);
  }
  return PN_OK;
}

const char* pn_status_string(pn_status s) {
  switch (s) {
    case PN_OK: return "ok";
    case PN_ERR_INVALID_ARG: return "invalid argument";
    case PN_ERR_BAD_DESCRIPTOR: return "malformed descriptor";
    case PN_ERR_UNSUPPORTED_OP: return "unsupported operator or combination";
    case PN_ERR_SHAPE: return "shape error";
    case PN_ERR_TOO_LARGE: return "graph exceeds a kernel budget";
    case PN_ERR_ALIGNMENT: return "pointer alignment";
    case PN_ERR_COUNT: return "wrong number of inputs or outputs";
    case PN_ERR_DEVICE: return "device error";
    case PN_ERR_CUDA: return "CUDA error";
    default: return "unknown status";
  }
}

const char* pn_last_error(void) { return g_last_error.c_str(); }

#pragma GCC visibility pop
}  // extern "C"
