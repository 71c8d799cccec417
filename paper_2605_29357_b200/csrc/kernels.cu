// kernels.cu -- the kernels compiled into the library: the bytecode interpreter, one
// instance per tile shape (VL, NG, K).  The device code is in device_lib.cuh, which also
// serves, as text, the kernels specialised per graph at create time.
//
// This file is compiled once per instance (with -DPN_VL= -DPN_NG= -DPN_K=, so that the instances
// build side by side) and once without them for the dispatch functions.
#include <cuda_runtime.h>

#include "plan.h"

#define PN_CAT_(a, b, c, d) a##_##b##_##c##_##d
#define PN_CAT(a, b, c, d) PN_CAT_(a, b, c, d)
// The instances compiled into the library: (VL, NG, K).  The lowering asks only for these.
#define PN_INSTANCES(X) X(1, 8, 4) X(4, 2, 4) X(4, 4, 2) X(8, 1, 4) X(8, 2, 2)

#ifdef PN_VL
#define PN_BOUNDS_RUNTIME 1   // the interpreter kernels check when the launch carries a status word
#include "device_lib.cuh"

namespace pn {

template <int VL, int NG, int K>
__global__ void __launch_bounds__(VL * NG > 8 ? 256 : 512)
fused_kernel(const __grid_constant__ KernelParams p) {
  extern __shared__ __align__(16) unsigned char smem[];
  if (p.family == FAM_COLUMN) column_body<Interp<VL, NG, K>>(p, smem);
  else fused_body<Interp<VL, NG, K>>(p, smem);
}

cudaError_t PN_CAT(launch_instance, PN_VL, PN_NG, PN_K)(const LaunchPlan& lp, cudaStream_t stream) {
  auto kern = fused_kernel<PN_VL, PN_NG, PN_K>;
  cudaError_t e = cudaSuccess;
  if (lp.smem_bytes > 48 * 1024) {
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, lp.smem_bytes);
    if (e != cudaSuccess) return e;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(lp.grid, 1, 1);
  cfg.blockDim = dim3(lp.block, 1, 1);
  cfg.dynamicSmemBytes = lp.smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  if (lp.p.cluster > 1) {
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = lp.p.cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
  }
  return cudaLaunchKernelEx(&cfg, kern, lp.p);
}

// Resident CTAs per SM of the instance (0 on failure).
int PN_CAT(occupancy_instance, PN_VL, PN_NG, PN_K)(int block, int smem_bytes) {
  int n = 0;
  return cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, fused_kernel<PN_VL, PN_NG, PN_K>, block, smem_bytes) == cudaSuccess ? n : 0;
}

}  // namespace pn

#else   // the dispatch functions

namespace pn {

#define PN_X(A, B, C)                                                                        \
  cudaError_t PN_CAT(launch_instance, A, B, C)(const LaunchPlan& lp, cudaStream_t stream);  \
  int PN_CAT(occupancy_instance, A, B, C)(int block, int smem_bytes);
PN_INSTANCES(PN_X)
#undef PN_X

cudaError_t launch_plan(const LaunchPlan& lp, cudaStream_t stream) {
#define PN_X(A, B, C) if (lp.vl == A && lp.ng == B && lp.k == C) return PN_CAT(launch_instance, A, B, C)(lp, stream);
  PN_INSTANCES(PN_X)
#undef PN_X
  return cudaErrorInvalidValue;
}

// Resident CTAs per SM of an instance, for sizing grids (0 on failure).
int instance_occupancy(int vl_, int ng_, int k_, int block, int smem_bytes) {
#define PN_X(A, B, C) if (vl_ == A && ng_ == B && k_ == C) return PN_CAT(occupancy_instance, A, B, C)(block, smem_bytes);
  PN_INSTANCES(PN_X)
#undef PN_X
  return 0;
}

}  // namespace pn
#endif
