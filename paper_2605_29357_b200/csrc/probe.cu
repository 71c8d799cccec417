// probe.cu -- pn_stream_probe: a hand-written streaming kernel that moves bytes through HBM in a
// chosen read : write mix and does nothing else.  Its rate is the ceiling a fused kernel of the
// same mix is judged against (a softmax is 1 : 1, a residual + LayerNorm 2 : 1, a long-row
// reduction read-only), next to the plain device copy.
//
// Three ways of reading: 128-bit loads through the read-only path, the same loads without
// allocating in L1, and 1-D bulk copies (cp.async.bulk) into a ring of shared-memory stages that
// complete on mbarriers and are issued by one elected thread of a producer warp.  Bulk copies
// read this GPU's own memory only and are never multicast.  Every mbarrier wait is a try_wait
// loop with a retry limit: a wait that runs out sets a bit in the status word, the kernel
// waits (again bounded) for its own copies in flight and returns.
#include <cstring>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>
#include <string>

#include "../../include/pn.h"
#include "handle.h"

using namespace pn;

namespace {

constexpr unsigned kWaitLimit = 1u << 22;   // polls of one mbarrier wait before it gives up

__device__ __forceinline__ uint4 ld_nc(const uint4* p) { return __ldg(p); }
__device__ __forceinline__ uint4 ld_nc_noalloc(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ void st_plain(uint4* p, uint4 v) { *p = v; }
__device__ __forceinline__ void st_stream(uint4* p, uint4 v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void st_plain(uint2* p, uint2 v) { *p = v; }
__device__ __forceinline__ void st_stream(uint2* p, uint2 v) {
  asm volatile("st.global.cs.v2.u32 [%0], {%1, %2};" ::"l"(p), "r"(v.x), "r"(v.y) : "memory");
}
__device__ __forceinline__ uint4 mix4(uint4 a, uint4 b) { return make_uint4(a.x ^ b.x, a.y ^ b.y, a.z ^ b.z, a.w ^ b.w); }

// What a unit (16 bytes of every read array) turns into: 16 bytes for c, 8 bytes for d.
template <int NW16, int NW8, bool CS>
__device__ __forceinline__ void emit(uint4 x, uint4* c, uint2* d, size_t idx, uint4& sink) {
  if constexpr (NW16 > 0) { if constexpr (CS) st_stream(c + idx, x); else st_plain(c + idx, x); }
  if constexpr (NW8 > 0) { const uint2 h = make_uint2(x.x ^ x.z, x.y ^ x.w); if constexpr (CS) st_stream(d + idx, h); else st_plain(d + idx, h); }
  if constexpr (NW16 == 0 && NW8 == 0) sink = mix4(sink, x);
}

// Loads straight into registers.  LAYOUT 0: grid-stride over units; 1: every block owns one
// contiguous range of the arrays; 2: the arrays are cut into runs of `run` units, the blocks take
// the runs in turn and walk each from its start to its end.  U units per thread are in flight
// together.
template <int NR, int NW16, int NW8, int U, bool NOALLOC, bool CS, int LAYOUT>
__global__ void probe_direct(const uint4* __restrict__ a, const uint4* __restrict__ b, uint4* __restrict__ c,
                             uint2* __restrict__ d, size_t units, size_t run, unsigned* status) {
  // launched like the generated graph kernels: set up while the kernel before it in the stream still
  // runs, and waiting here until that one is complete
  asm volatile("griddepcontrol.wait;" ::: "memory");
  uint4 sink = make_uint4(0, 0, 0, 0);
  size_t begin, end, step;
  if (LAYOUT == 0) { begin = (size_t)blockIdx.x * blockDim.x + threadIdx.x; end = units; step = (size_t)gridDim.x * blockDim.x; }
  else if (LAYOUT == 1) {
    const size_t per = (units + gridDim.x - 1) / gridDim.x;
    begin = per * blockIdx.x + threadIdx.x; end = min(units, per * (blockIdx.x + 1)); step = blockDim.x;
  } else { begin = 0; end = 0; step = blockDim.x; }
  const size_t n_runs = LAYOUT == 2 ? (units + run - 1) / run : 1;
  for (size_t r = LAYOUT == 2 ? blockIdx.x : 0; r < n_runs; r += LAYOUT == 2 ? gridDim.x : n_runs) {
  if (LAYOUT == 2) { begin = r * run + threadIdx.x; end = min(units, (r + 1) * run); }
  for (size_t i = begin; i < end; i += step * U) {
    uint4 va[U], vb[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const size_t idx = i + u * step;
      va[u] = make_uint4(u, 1, 2, 3); vb[u] = make_uint4(0, 0, 0, 0);
      if (idx < end) {
        if constexpr (NR >= 1) va[u] = NOALLOC ? ld_nc_noalloc(a + idx) : ld_nc(a + idx);
        if constexpr (NR >= 2) vb[u] = NOALLOC ? ld_nc_noalloc(b + idx) : ld_nc(b + idx);
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const size_t idx = i + u * step;
      if (idx < end) emit<NW16, NW8, CS>(mix4(va[u], vb[u]), c, d, idx, sink);
    }
  }
  }
  // a read-only probe must keep its loads alive: the store below never happens in practice
  if (NW16 == 0 && NW8 == 0 && (sink.x ^ sink.y ^ sink.z ^ sink.w) == 0x9E3779B9u && sink.x == 0x7F4A7C15u) atomicOr(status, 0x80000000u);
}

// Read-only, the access pattern of a reduction over a leading dimension: the array is rows of C units;
// a block owns a strip of TX units by RS consecutive rows and its blockDim.x / TX walkers go down the
// rows, U rows of each in flight together.  Blocks are numbered so that neighbours own neighbouring
// strips of the same rows.
template <int U>
__global__ void probe_strips(const uint4* __restrict__ a, size_t units, int C, int TX, int RS, unsigned* status) {
  const size_t rows = units / C;
  const int ctiles = C / TX, TY = blockDim.x / TX;
  const int ct = blockIdx.x % ctiles;
  const size_t rb = blockIdx.x / ctiles;
  const int tx = threadIdx.x % TX, ty = threadIdx.x / TX;
  const size_t r_end = min(rows, (rb + 1) * (size_t)RS);
  uint4 sink = make_uint4(0, 0, 0, 0);
  for (size_t r0 = rb * (size_t)RS + ty; r0 < r_end; r0 += (size_t)TY * U) {
    uint4 v[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const size_t r = r0 + (size_t)u * TY;
      v[u] = make_uint4(0, 0, 0, 0);
      if (r < r_end) v[u] = ld_nc(a + r * C + (size_t)ct * TX + tx);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) sink = mix4(sink, v[u]);
  }
  if ((sink.x ^ sink.y ^ sink.z ^ sink.w) == 0x9E3779B9u && sink.x == 0x7F4A7C15u) atomicOr(status, 0x80000000u);
}

// ---- bulk copies into a shared-memory ring -----------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// true when the phase with the given parity has completed; gives up after kWaitLimit polls
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, unsigned parity) {
  const uint32_t addr = smem_u32(bar);
  for (unsigned n = 0; n < kWaitLimit; ++n) {
    uint32_t done;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(done) : "r"(addr), "r"(parity) : "memory");
    if (done) return true;
  }
  return false;
}
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, unsigned bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// One producer warp (its lane 0 issues the copies) and blockDim.x - 32 consumer threads.  A stage
// holds TILE units of every read array.  Every block owns one contiguous range of the arrays.
template <int NR, int NW16, int NW8, bool CS>
__global__ void probe_bulk(const uint4* __restrict__ a, const uint4* __restrict__ b, uint4* __restrict__ c,
                           uint2* __restrict__ d, size_t units, int stages, int tile_units, unsigned* status) {
  extern __shared__ __align__(128) unsigned char smem[];
  uint64_t* full = reinterpret_cast<uint64_t*>(smem);
  uint64_t* empty = full + stages;
  uint4* ring = reinterpret_cast<uint4*>(smem + 1024);
  const int consumers = blockDim.x - 32, cwarps = consumers / 32;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) { mbar_init(full + s, 1); mbar_init(empty + s, cwarps); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const size_t per = ((units + gridDim.x - 1) / gridDim.x + tile_units - 1) / tile_units * tile_units;
  const size_t begin = min(units, per * blockIdx.x), end = min(units, per * (blockIdx.x + 1));
  const int n_tiles = (int)((end - begin + tile_units - 1) / tile_units);
  if (warp == cwarps) {   // the producer warp
    if (lane == 0) {
      bool ok = true;
      int issued = 0;
      for (int t = 0; t < n_tiles && ok; ++t) {
        const int s = t % stages;
        if (t >= stages) ok = mbar_wait(empty + s, ((t / stages) - 1) & 1);
        if (!ok) break;
        const size_t u0 = begin + (size_t)t * tile_units;
        const unsigned n = (unsigned)min((size_t)tile_units, end - u0);
        mbar_expect_tx(full + s, n * 16u * NR);
        bulk_load(ring + (size_t)(s * NR) * tile_units, a + u0, n * 16u, full + s);
        if constexpr (NR >= 2) bulk_load(ring + (size_t)(s * NR + 1) * tile_units, b + u0, n * 16u, full + s);
        issued = t + 1;
      }
      if (!ok) {   // a wait ran out: record it, then let the copies in flight land before the block may exit
        atomicOr(status, 1u);
        for (int t = max(0, issued - stages); t < issued; ++t) mbar_wait(full + t % stages, (t / stages) & 1);
      }
    }
  } else {
    uint4 sink = make_uint4(0, 0, 0, 0);
    bool ok = true;
    for (int t = 0; t < n_tiles && ok; ++t) {
      const int s = t % stages;
      ok = mbar_wait(full + s, (t / stages) & 1);
      if (!ok) { atomicOr(status, 2u); break; }
      const size_t u0 = begin + (size_t)t * tile_units;
      const int n = (int)min((size_t)tile_units, end - u0);
      const uint4* ra = ring + (size_t)(s * NR) * tile_units;
      for (int i = threadIdx.x; i < n; i += consumers) {
        uint4 x = ra[i];
        if constexpr (NR >= 2) x = mix4(x, ra[tile_units + i]);
        emit<NW16, NW8, CS>(x, c, d, u0 + i, sink);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty + s);
    }
    if (NW16 == 0 && NW8 == 0 && (sink.x ^ sink.y ^ sink.z ^ sink.w) == 0x9E3779B9u && sink.x == 0x7F4A7C15u) atomicOr(status, 0x80000000u);
  }
}

template <int NR, int NW16, int NW8>
cudaError_t launch_mix(int loader, int store, int layout, int block, int unroll, int grid, int stages, int tile_units,
                       const uint4* a, const uint4* b, uint4* c, uint2* d, size_t units, unsigned* status, cudaStream_t s) {
  if (loader == PN_PROBE_BULK) {
    if (NR == 0) return cudaErrorInvalidValue;
    const size_t smem = 1024 + (size_t)stages * tile_units * 16 * NR;
    auto k = store ? probe_bulk<NR, NW16, NW8, true> : probe_bulk<NR, NW16, NW8, false>;
    cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    k<<<grid, block + 32, smem, s>>>(a, b, c, d, units, stages, tile_units, status);
    return cudaGetLastError();
  }
  cudaLaunchConfig_t lc;
  memset(&lc, 0, sizeof(lc));
  lc.gridDim = dim3((unsigned)grid, 1, 1); lc.blockDim = dim3((unsigned)block, 1, 1); lc.dynamicSmemBytes = 0; lc.stream = s;
  cudaLaunchAttribute overlap;
  overlap.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  overlap.val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = &overlap; lc.numAttrs = 1;
  cudaError_t le = cudaSuccess;
#define PN_PROBE_GO(U, NA, CS, LY) le = cudaLaunchKernelEx(&lc, probe_direct<NR, NW16, NW8, U, NA, CS, LY>, a, b, c, d, units, (size_t)tile_units, status)
#define PN_PROBE_U(NA, CS, LY)                                                            \
  switch (unroll) {                                                                       \
    case 1: PN_PROBE_GO(1, NA, CS, LY); break;                                            \
    case 2: PN_PROBE_GO(2, NA, CS, LY); break;                                            \
    case 4: PN_PROBE_GO(4, NA, CS, LY); break;                                            \
    case 8: PN_PROBE_GO(8, NA, CS, LY); break;                                            \
    default: return cudaErrorInvalidValue;                                                \
  }
  const bool na = loader == PN_PROBE_LDG_NOALLOC;
  if (layout == 0) { if (na) { if (store) { PN_PROBE_U(true, true, 0) } else { PN_PROBE_U(true, false, 0) } } else { if (store) { PN_PROBE_U(false, true, 0) } else { PN_PROBE_U(false, false, 0) } } }
  else if (layout == 2) { if (store) { PN_PROBE_U(false, true, 2) } else { PN_PROBE_U(false, false, 2) } }
  else { if (na) { if (store) { PN_PROBE_U(true, true, 1) } else { PN_PROBE_U(true, false, 1) } } else { if (store) { PN_PROBE_U(false, true, 1) } else { PN_PROBE_U(false, false, 1) } } }
#undef PN_PROBE_U
#undef PN_PROBE_GO
  return le != cudaSuccess ? le : cudaGetLastError();
}

}  // namespace

extern "C" {
#pragma GCC visibility push(default)

pn_status pn_stream_probe(int mix, const pn_probe_config* cfg, const void* a, const void* b, void* c, void* d,
                          size_t units, void* status_word, void* stream) {
  if (!cfg || !status_word) return fail(PN_ERR_INVALID_ARG, "null argument");
  const int nr = mix == PN_MIX_WRITE ? 0 : (mix == PN_MIX_READ || mix == PN_MIX_1_1) ? 1 : 2;
  const bool w16 = mix != PN_MIX_READ, w8 = mix == PN_MIX_4_3;
  if (mix < PN_MIX_READ || mix > PN_MIX_4_3) return fail(PN_ERR_INVALID_ARG, "unknown mix");
  if ((nr >= 1 && !a) || (nr >= 2 && !b) || (w16 && !c) || (w8 && !d)) return fail(PN_ERR_INVALID_ARG, "a buffer of this mix is null");
  for (const void* p : {a, b, (const void*)c, (const void*)d, (const void*)status_word})
    if ((uintptr_t)p & 15) return fail(PN_ERR_ALIGNMENT, "probe buffers must be aligned to 16 bytes");
  if (cfg->block < 32 || cfg->block > 992 || cfg->block % 32 || (cfg->grid < 1 && cfg->layout != 3)) return fail(PN_ERR_INVALID_ARG, "block must be a multiple of 32 up to 992, grid positive");
  if (cfg->loader < PN_PROBE_LDG || cfg->loader > PN_PROBE_BULK) return fail(PN_ERR_INVALID_ARG, "unknown loader");
  if (cfg->loader == PN_PROBE_BULK) {
    if (nr == 0) return fail(PN_ERR_INVALID_ARG, "a write-only probe has nothing to load");
    if (cfg->stages < 2 || cfg->stages > 16 || cfg->tile_units < 32 || cfg->tile_units > 4096)
      return fail(PN_ERR_INVALID_ARG, "bulk loader: 2..16 stages of 32..4096 units");
    if (1024 + (size_t)cfg->stages * cfg->tile_units * 16 * nr > 227 * 1024) return fail(PN_ERR_TOO_LARGE, "the ring does not fit in shared memory");
  } else {
    if (cfg->unroll != 1 && cfg->unroll != 2 && cfg->unroll != 4 && cfg->unroll != 8) return fail(PN_ERR_INVALID_ARG, "unroll must be 1, 2, 4 or 8");
    if (cfg->layout < 0 || cfg->layout > 3 || (cfg->layout == 2 && cfg->tile_units < 1)) return fail(PN_ERR_INVALID_ARG, "layout must be 0 .. 3 (2 with tile_units > 0 as the run length)");
  }
  if (units == 0) return PN_OK;
  if (cfg->layout == 3) {   // strips: read-only
    if (mix != PN_MIX_READ || cfg->loader != PN_PROBE_LDG) return fail(PN_ERR_INVALID_ARG, "the strip layout is a read-only probe with plain loads");
    const int C = cfg->tile_units, TX = cfg->strip_units, RS = cfg->rows_per_block;
    if (C < 1 || TX < 1 || RS < 1 || C % TX || cfg->block % TX || units % (size_t)C) return fail(PN_ERR_INVALID_ARG, "strips: tile_units (row length) must divide the array and be a multiple of strip_units, which must divide block");
    const size_t rows = units / C;
    const size_t blocks = (rows + RS - 1) / RS * (C / TX);
    if (blocks > (1u << 30)) return fail(PN_ERR_TOO_LARGE, "too many strips");
    unsigned* st = (unsigned*)status_word;
    cudaStream_t s = (cudaStream_t)stream;
    switch (cfg->unroll) {
      case 1: probe_strips<1><<<(unsigned)blocks, cfg->block, 0, s>>>((const uint4*)a, units, C, TX, RS, st); break;
      case 2: probe_strips<2><<<(unsigned)blocks, cfg->block, 0, s>>>((const uint4*)a, units, C, TX, RS, st); break;
      case 4: probe_strips<4><<<(unsigned)blocks, cfg->block, 0, s>>>((const uint4*)a, units, C, TX, RS, st); break;
      default: probe_strips<8><<<(unsigned)blocks, cfg->block, 0, s>>>((const uint4*)a, units, C, TX, RS, st); break;
    }
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(PN_ERR_CUDA, std::string("probe launch: ") + cudaGetErrorString(e));
    return PN_OK;
  }
  const uint4* pa = (const uint4*)a; const uint4* pb = (const uint4*)b; uint4* pc = (uint4*)c; uint2* pd = (uint2*)d;
  cudaError_t e;
#define PN_MIX_GO(NR, W16, W8) launch_mix<NR, W16, W8>(cfg->loader, cfg->streaming_stores, cfg->layout, cfg->block, cfg->unroll, cfg->grid, cfg->stages, cfg->tile_units, pa, pb, pc, pd, units, (unsigned*)status_word, (cudaStream_t)stream)
  switch (mix) {
    case PN_MIX_READ: e = PN_MIX_GO(1, 0, 0); break;
    case PN_MIX_WRITE: e = PN_MIX_GO(0, 1, 0); break;
    case PN_MIX_1_1: e = PN_MIX_GO(1, 1, 0); break;
    case PN_MIX_2_1: e = PN_MIX_GO(2, 1, 0); break;
    default: e = PN_MIX_GO(2, 1, 1); break;
  }
#undef PN_MIX_GO
  if (e != cudaSuccess) return fail(PN_ERR_CUDA, std::string("probe launch: ") + cudaGetErrorString(e));
  return PN_OK;
}

#pragma GCC visibility pop
}  // extern "C"
