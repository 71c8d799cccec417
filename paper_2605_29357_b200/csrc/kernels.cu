// kernels.cu -- the fused kernels (sm_100a).
//
// One kernel template serves every family.  A *team* of threads (a warp, a thread block,
// or the thread blocks of a cluster) owns one row of the iteration space at a time; each
// thread holds a register tile of NG groups of VL consecutive elements and interprets the
// tile bytecode on it: loads widen to fp32 in registers, the pointwise DAG runs in
// registers, reductions fold the tile into a 3-float partial that is combined thread ->
// warp (shuffles) -> block (shared memory) -> cluster (distributed shared memory), per-row
// scalar programs run on the combined values, and the epilogue narrows and stores.  Every
// graph input is read once and every output written once.
//
// No spin-waits anywhere: cross-thread hand-offs are __syncwarp / __syncthreads /
// cluster barriers only.  Nothing traps.
#include <cooperative_groups.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <math_constants.h>

#include "plan.h"

namespace cg = cooperative_groups;

namespace pn {

// ---------------------------------------------------------------------------------------
// small helpers
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ float bits_f(uint32_t u) { return __uint_as_float(u); }
__device__ __forceinline__ uint32_t f_bits(float f) { return __float_as_uint(f); }

__device__ __forceinline__ int dtype_size(int dt) {
  switch (dt) {
    case kF32: case kI32: return 4;
    case kF16: case kBF16: return 2;
    case kI64: return 8;
    default: return 1;
  }
}

// Load BYTES contiguous bytes (address aligned to min(BYTES,16)) into 32-bit words.
template <int BYTES>
__device__ __forceinline__ void load_words(const char* p, uint32_t* w) {
  if constexpr (BYTES >= 16) {
#pragma unroll
    for (int i = 0; i < BYTES / 16; ++i) {
      uint4 v = __ldg(reinterpret_cast<const uint4*>(p) + i);
      w[4 * i] = v.x; w[4 * i + 1] = v.y; w[4 * i + 2] = v.z; w[4 * i + 3] = v.w;
    }
  } else if constexpr (BYTES == 8) {
    uint2 v = __ldg(reinterpret_cast<const uint2*>(p));
    w[0] = v.x; w[1] = v.y;
  } else if constexpr (BYTES == 4) {
    w[0] = __ldg(reinterpret_cast<const uint32_t*>(p));
  } else if constexpr (BYTES == 2) {
    w[0] = __ldg(reinterpret_cast<const uint16_t*>(p));
  } else {
    w[0] = __ldg(reinterpret_cast<const uint8_t*>(p));
  }
}

template <int BYTES>
__device__ __forceinline__ void store_words(char* p, const uint32_t* w) {
  if constexpr (BYTES >= 16) {
#pragma unroll
    for (int i = 0; i < BYTES / 16; ++i)
      reinterpret_cast<uint4*>(p)[i] = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
  } else if constexpr (BYTES == 8) {
    *reinterpret_cast<uint2*>(p) = make_uint2(w[0], w[1]);
  } else if constexpr (BYTES == 4) {
    *reinterpret_cast<uint32_t*>(p) = w[0];
  } else if constexpr (BYTES == 2) {
    *reinterpret_cast<uint16_t*>(p) = static_cast<uint16_t>(w[0]);
  } else {
    *reinterpret_cast<uint8_t*>(p) = static_cast<uint8_t>(w[0]);
  }
}

__device__ __forceinline__ float widen_scalar(const char* p, int dt) {
  switch (dt) {
    case kF32: return __ldg(reinterpret_cast<const float*>(p));
    case kF16: return __half2float(__ushort_as_half(__ldg(reinterpret_cast<const uint16_t*>(p))));
    case kBF16: return bits_f(static_cast<uint32_t>(__ldg(reinterpret_cast<const uint16_t*>(p))) << 16);
    case kI8: return static_cast<float>(static_cast<int8_t>(__ldg(reinterpret_cast<const uint8_t*>(p))));
    case kBool: return __ldg(reinterpret_cast<const uint8_t*>(p)) ? 1.f : 0.f;
    case kI32: return static_cast<float>(__ldg(reinterpret_cast<const int32_t*>(p)));
    default: return static_cast<float>(__ldg(reinterpret_cast<const long long*>(p)));
  }
}

// Storage bits of one group of VL elements -> VL floats, in place.
template <int VL>
__device__ __forceinline__ void widen_group(float* g, int dt) {
  uint32_t w[VL];
#pragma unroll
  for (int i = 0; i < VL; ++i) w[i] = f_bits(g[i]);
  switch (dt) {
    case kF32: case kI64: break;  // i64 operands are converted at load time
    case kBF16:
#pragma unroll
      for (int i = 0; i < VL; ++i) g[i] = bits_f((i & 1) ? (w[i >> 1] & 0xFFFF0000u) : (w[i >> 1] << 16));
      break;
    case kF16:
#pragma unroll
      for (int i = 0; i < VL; ++i)
        g[i] = __half2float(__ushort_as_half(static_cast<uint16_t>(w[i >> 1] >> ((i & 1) * 16))));
      break;
    case kI8:
#pragma unroll
      for (int i = 0; i < VL; ++i)
        g[i] = static_cast<float>(static_cast<int8_t>((w[i >> 2] >> ((i & 3) * 8)) & 0xFF));
      break;
    case kBool:
#pragma unroll
      for (int i = 0; i < VL; ++i) g[i] = ((w[i >> 2] >> ((i & 3) * 8)) & 0xFF) ? 1.f : 0.f;
      break;
    case kI32:
#pragma unroll
      for (int i = 0; i < VL; ++i) g[i] = static_cast<float>(static_cast<int32_t>(w[i]));
      break;
  }
}

template <int VL>
__device__ __forceinline__ void load_group_raw(const char* base, long long elem, int dt, float* g) {
  uint32_t w[VL];
#pragma unroll
  for (int i = 0; i < VL; ++i) w[i] = 0;
  switch (dt) {
    case kF32: case kI32: load_words<VL * 4>(base + elem * 4, w); break;
    case kF16: case kBF16: load_words<VL * 2>(base + elem * 2, w); break;
    case kI8: case kBool: load_words<VL>(base + elem, w); break;
    default:  // i64: converted here, WIDEN is then a no-op
#pragma unroll
      for (int i = 0; i < VL; ++i)
        w[i] = f_bits(static_cast<float>(__ldg(reinterpret_cast<const long long*>(base) + elem + i)));
      break;
  }
#pragma unroll
  for (int i = 0; i < VL; ++i) g[i] = bits_f(w[i]);
}

template <int VL>
__device__ __forceinline__ void store_group(char* base, long long elem, int dt, const float* g) {
  uint32_t w[VL];
  switch (dt) {
    case kF32:
#pragma unroll
      for (int i = 0; i < VL; ++i) w[i] = f_bits(g[i]);
      store_words<VL * 4>(base + elem * 4, w);
      break;
    case kI32:
#pragma unroll
      for (int i = 0; i < VL; ++i) w[i] = static_cast<uint32_t>(__float2int_rz(g[i]));
      store_words<VL * 4>(base + elem * 4, w);
      break;
    case kBF16:
      if constexpr (VL == 1) {
        w[0] = __bfloat16_as_ushort(__float2bfloat16_rn(g[0]));
      } else {
#pragma unroll
        for (int i = 0; i < VL / 2; ++i) {
          __nv_bfloat162 h = __floats2bfloat162_rn(g[2 * i], g[2 * i + 1]);
          w[i] = *reinterpret_cast<uint32_t*>(&h);
        }
      }
      store_words<VL * 2>(base + elem * 2, w);
      break;
    case kF16:
      if constexpr (VL == 1) {
        w[0] = __half_as_ushort(__float2half_rn(g[0]));
      } else {
#pragma unroll
        for (int i = 0; i < VL / 2; ++i) {
          __half2 h = __floats2half2_rn(g[2 * i], g[2 * i + 1]);
          w[i] = *reinterpret_cast<uint32_t*>(&h);
        }
      }
      store_words<VL * 2>(base + elem * 2, w);
      break;
    case kI8: case kBool: {
#pragma unroll
      for (int i = 0; i < (VL + 3) / 4; ++i) w[i] = 0;
#pragma unroll
      for (int i = 0; i < VL; ++i) {
        uint32_t b = dt == kBool ? (g[i] != 0.f ? 1u : 0u)
                                 : (static_cast<uint32_t>(__float2int_rz(g[i])) & 0xFFu);
        w[i >> 2] |= b << ((i & 3) * 8);
      }
      store_words<VL>(base + elem, w);
      break;
    }
    default:  // i64
#pragma unroll
      for (int i = 0; i < VL; ++i)
        reinterpret_cast<long long*>(base)[elem + i] = static_cast<long long>(__float2int_rz(g[i]));
      break;
  }
}

// ---------------------------------------------------------------------------------------
// scalar math (fp32).  The fp32 outputs are held to rtol 1e-5, so the special-function
// unit's approximations are used only where a correction keeps the error near 1e-7.
// ---------------------------------------------------------------------------------------
// e^x = 2^(x*log2 e).  The product is split into its rounded value t and the rounding
// residual r (recovered exactly by an fma, plus the low part of log2 e); 2^t comes from
// ex2.approx (relative error about 2^-22) and the residual is applied as a first-order
// factor.  Overflow gives +inf, large negative arguments 0, NaN stays NaN.
__device__ __forceinline__ float f_exp(float x) {
  const float L2E_HI = 1.4426950216293335f, L2E_LO = 1.9259629911266175e-8f, LN2 = 0.6931471805599453f;
  const float t = x * L2E_HI;
  float r = fmaf(x, L2E_HI, -t);
  r = fmaf(x, L2E_LO, r);
  const float e = exp2f(t);   // ex2.approx
  return (fabsf(x) < 100.f) ? fmaf(e, r * LN2, e) : e;   // skip the correction at inf / overflow
}
__device__ __forceinline__ float f_sigmoid(float x) { return __fdividef(1.f, 1.f + f_exp(-x)); }
// 0.5 x (1 + tanh u) = x / (1 + e^(-2u)),  u = sqrt(2/pi) (x + 0.044715 x^3)
__device__ __forceinline__ float f_gelu_tanh(float x) {
  const float k0 = 0.7978845608028654f, k1 = 0.044715f;
  const float u = k0 * fmaf(k1 * x * x, x, x);
  return x * f_sigmoid(2.f * u);
}
__device__ __forceinline__ float f_gelu_erf(float x) { return 0.5f * x * (1.f + erff(x * 0.7071067811865476f)); }
__device__ __forceinline__ float f_max_nan(float a, float b) { return (a != a || b != b) ? CUDART_NAN_F : fmaxf(a, b); }
__device__ __forceinline__ float f_min_nan(float a, float b) { return (a != a || b != b) ? CUDART_NAN_F : fminf(a, b); }

// ---------------------------------------------------------------------------------------
// reduction partials
// ---------------------------------------------------------------------------------------
struct Part { float a, b, c; };

__device__ __forceinline__ Part red_identity(int kind) {
  switch (kind) {
    case RED_MAX: return {-CUDART_INF_F, 0.f, 0.f};
    case RED_MIN: return {CUDART_INF_F, 0.f, 0.f};
    case RED_ARGMAX: return {-CUDART_INF_F, bits_f(0x7FFFFFFFu), 0.f};
    case RED_ARGMIN: return {CUDART_INF_F, bits_f(0x7FFFFFFFu), 0.f};
    case RED_LSE: case RED_SOFTMAX: return {-CUDART_INF_F, 0.f, 0.f};
    default: return {0.f, 0.f, 0.f};
  }
}

// true when (v2, i2) should replace (v1, i1): larger value, NaN above everything, and on
// equal values (or both NaN) the lower column
__device__ __forceinline__ bool arg_better(float v2, int i2, float v1, int i1, bool want_max) {
  const bool n1 = v1 != v1, n2 = v2 != v2;
  if (n1 || n2) return n2 && (!n1 || i2 < i1);
  if (v2 == v1) return i2 < i1;
  return want_max ? v2 > v1 : v2 < v1;
}

__device__ __forceinline__ Part red_combine(int kind, Part x, Part y) {
  switch (kind) {
    case RED_SUM: x.a += y.a; break;
    case RED_MAX: x.a = f_max_nan(x.a, y.a); break;
    case RED_MIN: x.a = f_min_nan(x.a, y.a); break;
    case RED_ARGMAX: case RED_ARGMIN:
      if (arg_better(y.a, (int)f_bits(y.b), x.a, (int)f_bits(x.b), kind == RED_ARGMAX)) x = y;
      break;
    case RED_LSE: case RED_SOFTMAX: {
      const float m = fmaxf(x.a, y.a);
      if (m == -CUDART_INF_F) { x.b = 0.f; }
      else { x.b = x.b * f_exp(x.a - m) + y.b * f_exp(y.a - m); }
      x.a = m;
      break;
    }
    default: {  // RED_MEANVAR: pairwise update of (count, mean, M2)
      const float n = x.a + y.a;
      if (n > 0.f) {
        const float d = y.b - x.b, r = y.a / n;
        x.c = x.c + y.c + d * d * x.a * r;
        x.b = fmaf(d, r, x.b);
      }
      x.a = n;
      break;
    }
  }
  return x;
}

__device__ __forceinline__ Part warp_combine(int kind, Part v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    Part w;
    w.a = __shfl_xor_sync(0xFFFFFFFFu, v.a, o);
    w.b = __shfl_xor_sync(0xFFFFFFFFu, v.b, o);
    w.c = __shfl_xor_sync(0xFFFFFFFFu, v.c, o);
    // fixed operand order (lower lane first): both partners compute the same value
    v = (threadIdx.x & o) ? red_combine(kind, w, v) : red_combine(kind, v, w);
  }
  return v;
}

// ---------------------------------------------------------------------------------------
// the tile machine
// ---------------------------------------------------------------------------------------
struct TileCtx {
  const long long* rowoff;  // shared: element offset of this row for every io entry
  float* part;              // shared: this thread's partials, part[(r*3+q)*part_stride]
  float* slots;             // shared: per-row scalar slots of this team
  float* stash;             // shared: parked tile values (already offset by threadIdx.x)
  int part_stride;          // threads per CTA
  int col0;                 // column of (group 0, element 0)
  int gstride;              // columns between consecutive groups
  int col_end;              // one past the last valid column of this slice
  int chunk, chunks;        // position within the slice (chunk 0 starts a reduction)
  bool leader;              // this thread performs per-row scalar stores
};

// Run the statements with `r` bound to tile register k (kAccReg names the accumulator).
// A macro, so that every case is straight-line code on statically indexed registers.
#define PN_CASE_REG(n, ...) \
  case n: if constexpr (K > n) { float(&r)[V] = reg[n]; __VA_ARGS__ } break;
#define PN_WITH_REG(k, ...)                                 \
  switch (k) {                                              \
    PN_CASE_REG(0, __VA_ARGS__) PN_CASE_REG(1, __VA_ARGS__) \
    PN_CASE_REG(2, __VA_ARGS__) PN_CASE_REG(3, __VA_ARGS__) \
    default: { float(&r)[V] = acc; __VA_ARGS__ } break;     \
  }
#define PN_UNROLL _Pragma("unroll")

// SCALAR = true: the per-row scalar program (VL = NG = 1); loads are slot reads, stores go to
// the row's element of a per-row output and are done by the leader only.
template <int VL, int NG, int K, bool SCALAR>
__device__ __forceinline__ void run_program(const KernelParams& p, int pc, const int pc_end,
                                            const TileCtx& cx, float (&acc)[VL * NG],
                                            float (&reg)[K][VL * NG], float& ts) {
  constexpr int V = VL * NG;
  while (pc < pc_end) {
    const uint32_t word = p.code[pc++];
    const int op = word & 0xFF, a = (word >> 8) & 0xFF, b = (word >> 16) & 0xFF, c = word >> 24;

#define PN_UNARY(expr)                        \
  {                                           \
    PN_UNROLL for (int e = 0; e < V; ++e) {   \
      const float x = acc[e];                 \
      acc[e] = (expr);                        \
    }                                         \
  } break;

#define PN_BINARY(expr)                                                    \
  {                                                                        \
    if (b == OPK_REG) {                                                    \
      PN_WITH_REG(a, PN_UNROLL for (int e = 0; e < V; ++e) {               \
        const float x = acc[e]; const float y = r[e];                      \
        acc[e] = (expr);                                                   \
      })                                                                   \
    } else {                                                               \
      const float y = (b == OPK_IMM) ? bits_f(p.code[pc++]) : cx.slots[a]; \
      PN_UNROLL for (int e = 0; e < V; ++e) {                              \
        const float x = acc[e];                                            \
        acc[e] = (expr);                                                   \
      }                                                                    \
    }                                                                      \
  } break;

    switch (op) {
      // ---------------------------------------------------------------- memory
      case OP_LDRAW: {
        if constexpr (!SCALAR) {
          const char* base = static_cast<const char*>(p.io[a].base);
          const long long off = cx.rowoff[a];
          const int dt = p.io[a].dtype;
          PN_WITH_REG(b, PN_UNROLL for (int j = 0; j < NG; ++j) {
            const int col = cx.col0 + j * cx.gstride;
            if (col < cx.col_end) {
              load_group_raw<VL>(base, off + col, dt, &r[j * VL]);
            } else {
              PN_UNROLL for (int i = 0; i < VL; ++i) r[j * VL + i] = 0.f;
            }
          })
        }
        break;
      }
      case OP_WIDEN: {
        if constexpr (!SCALAR) {
          const int dt = p.io[a].dtype;
          if (dt != kF32 && dt != kI64) {
            PN_WITH_REG(b, PN_UNROLL for (int j = 0; j < NG; ++j) widen_group<VL>(&r[j * VL], dt);)
          }
        }
        break;
      }
      case OP_LDBC: {
        const int dt = p.io[a].dtype;
        const float v = widen_scalar(static_cast<const char*>(p.io[a].base) + cx.rowoff[a] * dtype_size(dt), dt);
        PN_WITH_REG(b, PN_UNROLL for (int e = 0; e < V; ++e) r[e] = v;)
        break;
      }
      case OP_LD:
        PN_WITH_REG(a, PN_UNROLL for (int e = 0; e < V; ++e) acc[e] = r[e];)
        break;
      case OP_ST:
        PN_WITH_REG(a, PN_UNROLL for (int e = 0; e < V; ++e) r[e] = acc[e];)
        break;
      case OP_STOUT: {
        char* base = static_cast<char*>(p.io[a].base);
        const long long off = cx.rowoff[a];
        const int dt = p.io[a].dtype;
        if constexpr (SCALAR) {
          if (cx.leader) store_group<1>(base, off, dt, &acc[0]);
        } else {
          PN_UNROLL for (int j = 0; j < NG; ++j) {
            const int col = cx.col0 + j * cx.gstride;
            if (col < cx.col_end) store_group<VL>(base, off + col, dt, &acc[j * VL]);
          }
        }
        break;
      }
      case OP_STOUT_I: {
        if constexpr (SCALAR) {
          if (cx.leader) {
            const int v = static_cast<int>(f_bits(acc[0]));
            char* base = static_cast<char*>(p.io[a].base);
            const long long off = cx.rowoff[a];
            if (p.io[a].dtype == kI64) reinterpret_cast<long long*>(base)[off] = v;
            else reinterpret_cast<int*>(base)[off] = v;
          }
        }
        break;
      }
      // ---------------------------------------------------------------- unary
      case OP_NEG: PN_UNARY(-x)
      case OP_ABS: PN_UNARY(fabsf(x))
      case OP_EXP: PN_UNARY(f_exp(x))
      case OP_LOG: PN_UNARY(logf(x))
      case OP_SQRT: PN_UNARY(sqrtf(x))
      case OP_RSQRT: PN_UNARY(1.f / sqrtf(x))
      case OP_RECIP: PN_UNARY(1.f / x)
      case OP_TANH: PN_UNARY(tanhf(x))
      case OP_SIGMOID: PN_UNARY(f_sigmoid(x))
      case OP_SILU: PN_UNARY(x * f_sigmoid(x))
      case OP_GELU_TANH: PN_UNARY(f_gelu_tanh(x))
      case OP_GELU_ERF: PN_UNARY(f_gelu_erf(x))
      case OP_RELU: PN_UNARY((x != x) ? x : fmaxf(x, 0.f))
      case OP_SQUARE: PN_UNARY(x * x)
      case OP_ERF: PN_UNARY(erff(x))
      case OP_RND_BF16: PN_UNARY(__bfloat162float(__float2bfloat16_rn(x)))
      case OP_RND_F16: PN_UNARY(__half2float(__float2half_rn(x)))
      case OP_TRUNC: PN_UNARY(truncf(x))
      case OP_NEZ: PN_UNARY(x != 0.f ? 1.f : 0.f)
      case OP_I2F: PN_UNARY(static_cast<float>(static_cast<int>(f_bits(x))))
      // ---------------------------------------------------------------- binary
      case OP_ADD: PN_BINARY(x + y)
      case OP_SUB: PN_BINARY(x - y)
      case OP_RSUB: PN_BINARY(y - x)
      case OP_MUL: PN_BINARY(x * y)
      case OP_DIV: PN_BINARY(x / y)
      case OP_RDIV: PN_BINARY(y / x)
      case OP_MAX: PN_BINARY(f_max_nan(x, y))
      case OP_MIN: PN_BINARY(f_min_nan(x, y))
      case OP_GT: PN_BINARY(x > y ? 1.f : 0.f)
      case OP_GE: PN_BINARY(x >= y ? 1.f : 0.f)
      case OP_LT: PN_BINARY(x < y ? 1.f : 0.f)
      case OP_LE: PN_BINARY(x <= y ? 1.f : 0.f)
      case OP_EQ: PN_BINARY(x == y ? 1.f : 0.f)
      case OP_NE: PN_BINARY(x != y ? 1.f : 0.f)
      case OP_LSEFIN: PN_BINARY((fabsf(x) == CUDART_INF_F) ? x : x + logf(y))
      // ---------------------------------------------------------------- ternary
      case OP_WHERE: case OP_FMA: {
        const int kx = c & 15, ky = c >> 4;
        float xs = 0.f, ys = 0.f;
        if (kx == OPK_IMM) xs = bits_f(p.code[pc++]); else if (kx == OPK_SLOT) xs = cx.slots[a];
        if (ky == OPK_IMM) ys = bits_f(p.code[pc++]); else if (ky == OPK_SLOT) ys = cx.slots[b];
        float yt[V];
        if (ky == OPK_REG) {
          PN_WITH_REG(b, PN_UNROLL for (int e = 0; e < V; ++e) yt[e] = r[e];)
        } else {
          PN_UNROLL for (int e = 0; e < V; ++e) yt[e] = ys;
        }
        if (kx == OPK_REG) {
          PN_WITH_REG(a, PN_UNROLL for (int e = 0; e < V; ++e)
            acc[e] = (op == OP_WHERE) ? (acc[e] != 0.f ? r[e] : yt[e]) : fmaf(acc[e], r[e], yt[e]);)
        } else {
          PN_UNROLL for (int e = 0; e < V; ++e)
            acc[e] = (op == OP_WHERE) ? (acc[e] != 0.f ? xs : yt[e]) : fmaf(acc[e], xs, yt[e]);
        }
        break;
      }
      // ---------------------------------------------------------------- reductions
      case OP_RED: {
        if constexpr (!SCALAR) {
          const int kind = a;
          Part t = red_identity(kind);
          // fold the valid elements of the tile, in element order
          if (kind == RED_SUM) {
            PN_UNROLL for (int j = 0; j < NG; ++j)
              if (cx.col0 + j * cx.gstride < cx.col_end) {
                PN_UNROLL for (int i = 0; i < VL; ++i) t.a += acc[j * VL + i];
              }
          } else if (kind == RED_MAX || kind == RED_MIN) {
            PN_UNROLL for (int j = 0; j < NG; ++j)
              if (cx.col0 + j * cx.gstride < cx.col_end) {
                PN_UNROLL for (int i = 0; i < VL; ++i)
                  t.a = kind == RED_MAX ? f_max_nan(t.a, acc[j * VL + i]) : f_min_nan(t.a, acc[j * VL + i]);
              }
          } else if (kind == RED_ARGMAX || kind == RED_ARGMIN) {
            int bi = 0x7FFFFFFF;
            float bv = t.a;
            PN_UNROLL for (int j = 0; j < NG; ++j) {
              const int col = cx.col0 + j * cx.gstride;
              if (col < cx.col_end) {
                PN_UNROLL for (int i = 0; i < VL; ++i) {
                  const float v = acc[j * VL + i];
                  if (arg_better(v, col + i, bv, bi, kind == RED_ARGMAX)) { bv = v; bi = col + i; }
                }
              }
            }
            t.a = bv; t.b = bits_f(static_cast<uint32_t>(bi));
          } else if (kind == RED_LSE || kind == RED_SOFTMAX) {
            float m = -CUDART_INF_F;
            PN_UNROLL for (int j = 0; j < NG; ++j)
              if (cx.col0 + j * cx.gstride < cx.col_end) {
                PN_UNROLL for (int i = 0; i < VL; ++i) m = fmaxf(m, acc[j * VL + i]);
              }
            const float ms = (m == -CUDART_INF_F) ? 0.f : m;   // keeps exp(x - ms) free of inf - inf
            float s = 0.f;
            PN_UNROLL for (int j = 0; j < NG; ++j) {
              const bool ok = cx.col0 + j * cx.gstride < cx.col_end;
              PN_UNROLL for (int i = 0; i < VL; ++i) {
                const float ev = ok ? f_exp(acc[j * VL + i] - ms) : 0.f;
                s += ev;
                if (kind == RED_SOFTMAX) acc[j * VL + i] = ev;
              }
            }
            t.a = m; t.b = s;
            if (kind == RED_SOFTMAX) ts = ms;
          } else {  // RED_MEANVAR
            float n = 0.f, sum = 0.f;
            PN_UNROLL for (int j = 0; j < NG; ++j)
              if (cx.col0 + j * cx.gstride < cx.col_end) {
                n += static_cast<float>(VL);
                PN_UNROLL for (int i = 0; i < VL; ++i) sum += acc[j * VL + i];
              }
            const float mean = n > 0.f ? sum / n : 0.f;
            float m2 = 0.f;
            PN_UNROLL for (int j = 0; j < NG; ++j)
              if (cx.col0 + j * cx.gstride < cx.col_end) {
                PN_UNROLL for (int i = 0; i < VL; ++i) { const float d = acc[j * VL + i] - mean; m2 = fmaf(d, d, m2); }
              }
            t.a = n; t.b = mean; t.c = m2;
          }
          float* ps = cx.part + b * 3 * cx.part_stride;
          if (cx.chunk > 0) {
            const Part prev{ps[0], ps[cx.part_stride], ps[2 * cx.part_stride]};
            t = red_combine(kind, prev, t);
          }
          ps[0] = t.a; ps[cx.part_stride] = t.b; ps[2 * cx.part_stride] = t.c;
        }
        break;
      }
      case OP_SCALE_TS: {
        const float f = f_exp(ts - cx.slots[a]) * cx.slots[b];
        PN_UNROLL for (int e = 0; e < V; ++e) acc[e] *= f;
        break;
      }
      // ---------------------------------------------------------------- stash
      case OP_SPILL: case OP_FILL: {
        if constexpr (!SCALAR) {
          float* sp = cx.stash + ((size_t)(b * cx.chunks + cx.chunk) * V) * cx.part_stride;
          PN_WITH_REG(a, PN_UNROLL for (int e = 0; e < V; ++e) {
            if (op == OP_SPILL) sp[e * cx.part_stride] = r[e]; else r[e] = sp[e * cx.part_stride];
          })
        }
        break;
      }
      case OP_SPILL_TS: case OP_FILL_TS: {
        if constexpr (!SCALAR) {
          float* sp = cx.stash + ((size_t)(b * cx.chunks + cx.chunk) * V) * cx.part_stride;
          if (op == OP_SPILL_TS) *sp = ts; else ts = *sp;
        }
        break;
      }
      // ---------------------------------------------------------------- scalar programs
      case OP_SLD:
        PN_UNROLL for (int e = 0; e < V; ++e) acc[e] = cx.slots[a];
        break;
      case OP_SST:
        if constexpr (SCALAR) {
          __syncwarp();
          if ((threadIdx.x & 31) == 0) cx.slots[a] = acc[0];
          __syncwarp();
        }
        break;
      default: break;
    }
#undef PN_UNARY
#undef PN_BINARY
  }
}

// ---------------------------------------------------------------------------------------
// the kernel
// ---------------------------------------------------------------------------------------
template <int VL, int NG, int K>
__global__ void __launch_bounds__(VL * NG > 8 ? 256 : 512)
fused_kernel(const __grid_constant__ KernelParams p, const int family) {
  constexpr int V = VL * NG;
  extern __shared__ __align__(16) unsigned char smem[];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  const bool warp_team = family <= FAM_WARP;
  const int team_threads = warp_team ? 32 : (int)blockDim.x;
  const int team_tid = warp_team ? lane : tid;
  const int team_in_cta = warp_team ? warp : 0;
  const int crank = (p.cluster > 1) ? (int)cg::this_cluster().block_rank() : 0;

  long long* rowoff = reinterpret_cast<long long*>(smem + p.sm_rowoff) + team_in_cta * kMaxIo;
  float* part = reinterpret_cast<float*>(smem + p.sm_part);
  float* wpart = reinterpret_cast<float*>(smem + p.sm_wpart);
  float* slots = reinterpret_cast<float*>(smem + p.sm_slots) + team_in_cta * kMaxSlots;
  float* ctapart = reinterpret_cast<float*>(smem + p.sm_ctapart);
  float* stash = reinterpret_cast<float*>(smem + p.sm_stash);

  TileCtx cx;
  cx.rowoff = rowoff;
  cx.part = part + tid;
  cx.part_stride = blockDim.x;
  cx.slots = slots;
  cx.stash = stash + tid;
  cx.gstride = team_threads * VL;
  cx.chunks = p.chunks;
  cx.chunk = 0;
  cx.leader = (team_tid == 0) && (crank == 0);

  const long long n_items = p.split_chunks ? p.rows * p.chunks : p.rows;
  long long team_global, n_teams;
  if (warp_team) { team_global = (long long)blockIdx.x * nwarps + warp; n_teams = (long long)gridDim.x * nwarps; }
  else { team_global = blockIdx.x / p.cluster; n_teams = gridDim.x / p.cluster; }

  const int slice_lo = crank * p.slice_len;
  const int slice_hi = min(p.row_len, slice_lo + p.slice_len);
  cx.col_end = slice_hi;
  const int chunk_cols = team_threads * V;
  unsigned parity = 0;

  float acc[V];
  float reg[K][V];
  float ts = 0.f;
#pragma unroll
  for (int e = 0; e < V; ++e) acc[e] = 0.f;
#pragma unroll
  for (int k = 0; k < K; ++k) {
#pragma unroll
    for (int e = 0; e < V; ++e) reg[k][e] = 0.f;
  }

  for (long long item = team_global; item < n_items; item += n_teams) {
    long long row = item;
    int c_first = 0, c_count = p.chunks;
    if (p.split_chunks) { row = item / p.chunks; c_first = (int)(item - row * p.chunks); c_count = 1; }

    // element offset of this row in every input / output
    if (team_tid < p.n_io) {
      const IoDesc& io = p.io[team_tid];
      long long r = row;
      const long long i2 = r % p.lead_dim[2]; r /= p.lead_dim[2];
      const long long i1 = r % p.lead_dim[1]; r /= p.lead_dim[1];
      rowoff[team_tid] = r * io.lead_stride[0] + i1 * io.lead_stride[1] + i2 * io.lead_stride[2];
    }
    if (warp_team) __syncwarp(); else __syncthreads();

    for (int s = 0; s < p.n_stages; ++s) {
      const StageDesc& st = p.stage[s];
      for (int c = c_first; c < c_first + c_count; ++c) {
        cx.chunk = p.split_chunks ? 0 : c;
        cx.col0 = slice_lo + c * chunk_cols + team_tid * VL;
        run_program<VL, NG, K, false>(p, st.elem_begin, st.elem_end, cx, acc, reg, ts);
      }
      if (st.n_red == 0 && st.scal_begin == st.scal_end) continue;

      // ---- combine the partials of this stage over the team, then the scalar program ---
      if (warp_team) {
        for (int r = 0; r < st.n_red; ++r) {
          const int kind = st.red[r].kind;
          Part v{cx.part[(r * 3) * cx.part_stride], cx.part[(r * 3 + 1) * cx.part_stride],
                 cx.part[(r * 3 + 2) * cx.part_stride]};
          v = warp_combine(kind, v);
          if (lane == 0) { float* d = slots + st.red[r].slot; d[0] = v.a; d[1] = v.b; d[2] = v.c; }
        }
        __syncwarp();
        {
          float sacc[1] = {0.f}, sreg[4][1] = {{0.f}, {0.f}, {0.f}, {0.f}}, sts = 0.f;
          run_program<1, 1, 4, true>(p, st.scal_begin, st.scal_end, cx, sacc, sreg, sts);
        }
        __syncwarp();
      } else {
        for (int r = 0; r < st.n_red; ++r) {
          const int kind = st.red[r].kind;
          Part v{cx.part[(r * 3) * cx.part_stride], cx.part[(r * 3 + 1) * cx.part_stride],
                 cx.part[(r * 3 + 2) * cx.part_stride]};
          v = warp_combine(kind, v);
          if (lane == 0) { float* w = wpart + (warp * kMaxRed + r) * 3; w[0] = v.a; w[1] = v.b; w[2] = v.c; }
        }
        __syncthreads();
        if (warp == 0) {
          for (int r = 0; r < st.n_red; ++r) {
            const int kind = st.red[r].kind;
            Part v = red_identity(kind);
            if (lane < nwarps) { const float* w = wpart + (lane * kMaxRed + r) * 3; v = Part{w[0], w[1], w[2]}; }
            v = warp_combine(kind, v);
            if (lane == 0) {
              float* d = (p.cluster > 1) ? ctapart + (parity * kMaxRed + r) * 3 : slots + st.red[r].slot;
              d[0] = v.a; d[1] = v.b; d[2] = v.c;
            }
          }
        }
        if (p.cluster > 1) {
          cg::cluster_group cl = cg::this_cluster();
          cl.sync();   // every CTA's partial is now in its own shared memory
          if (warp == 0) {
            for (int r = 0; r < st.n_red; ++r) {
              const int kind = st.red[r].kind;
              Part v = red_identity(kind);
              if (lane < p.cluster) {
                const float* w = cl.map_shared_rank(ctapart, lane) + (parity * kMaxRed + r) * 3;
                v = Part{w[0], w[1], w[2]};
              }
              v = warp_combine(kind, v);
              if (lane == 0) { float* d = slots + st.red[r].slot; d[0] = v.a; d[1] = v.b; d[2] = v.c; }
            }
          }
          parity ^= 1u;
        }
        if (warp == 0) {
          __syncwarp();
          float sacc[1] = {0.f}, sreg[4][1] = {{0.f}, {0.f}, {0.f}, {0.f}}, sts = 0.f;
          run_program<1, 1, 4, true>(p, st.scal_begin, st.scal_end, cx, sacc, sreg, sts);
        }
        __syncthreads();
      }
    }
    // the next item rewrites rowoff / slots: everyone must be done reading them
    if (warp_team) __syncwarp(); else __syncthreads();
  }
  // a CTA's shared memory may still be read by its cluster peers until they pass this point
  if (p.cluster > 1) cg::this_cluster().sync();
}

// ---------------------------------------------------------------------------------------
// host-side launch
// ---------------------------------------------------------------------------------------
template <int VL, int NG, int K>
static cudaError_t launch_instance(const LaunchPlan& lp, cudaStream_t stream) {
  auto kern = fused_kernel<VL, NG, K>;
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
  return cudaLaunchKernelEx(&cfg, kern, lp.p, (int)lp.family);
}

// The instances compiled into the library: (VL, NG, K).  The lowering asks only for these.
#define PN_INSTANCES(X) X(1, 8, 4) X(4, 2, 4) X(4, 4, 2) X(8, 1, 4) X(8, 2, 2)

cudaError_t launch_plan(const LaunchPlan& lp, cudaStream_t stream) {
#define PN_X(A, B, C) if (lp.vl == A && lp.ng == B && lp.k == C) return launch_instance<A, B, C>(lp, stream);
  PN_INSTANCES(PN_X)
#undef PN_X
  return cudaErrorInvalidValue;
}

// Resident CTAs per SM of an instance, for sizing grids (0 on failure).
int instance_occupancy(int vl_, int ng_, int k_, int block, int smem_bytes) {
  int n = 0;
  cudaError_t e = cudaErrorInvalidValue;
#define PN_X(A, B, C) \
  if (vl_ == A && ng_ == B && k_ == C) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, fused_kernel<A, B, C>, block, smem_bytes);
  PN_INSTANCES(PN_X)
#undef PN_X
  return e == cudaSuccess ? n : 0;
}

}  // namespace pn
