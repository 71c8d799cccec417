// device_lib.cuh -- device side of the fused kernels (sm_100a), self-contained: it includes
// no header, so that the same text serves the kernels compiled into the library (the bytecode
// interpreter) and the kernels specialised per graph at create time (NVRTC).  plan.h must
// precede it.
//
// A *team* of threads (a warp, a thread block, or the thread blocks of a cluster) owns one
// row of the iteration space at a time; each thread holds a register tile of NG groups of VL
// consecutive elements.  Loads widen to fp32 in registers, the pointwise DAG runs in
// registers, reductions fold the tile into a 3-float partial that is combined thread -> warp
// (shuffles) -> block (shared memory) -> cluster (distributed shared memory), per-row scalar
// programs run on the combined values, and the epilogue narrows and stores.  Every graph
// input is read once and every output written once.
//
// A program (class Prog) supplies the tile code and the scalar code of each stage: either by
// interpreting the bytecode (Interp) or as straight-line code generated from the same
// bytecode.  Both are built from the op_* functions below: one definition of every operation.
//
// No spin-waits anywhere: cross-thread hand-offs are __syncwarp / __syncthreads / cluster
// barriers only.  Nothing traps.
#pragma once

namespace pn {

#define PN_DEV __device__ __forceinline__
#define PN_UNROLL _Pragma("unroll")
#define PN_INF __int_as_float(0x7f800000)
#define PN_NAN __int_as_float(0x7fffffff)

PN_DEV float bits_f(uint32_t u) { return __uint_as_float(u); }
PN_DEV uint32_t f_bits(float f) { return __float_as_uint(f); }

PN_DEV int dtype_size(int dt) {
  switch (dt) {
    case kF32: case kI32: return 4;
    case kF16: case kBF16: return 2;
    case kI64: return 8;
    default: return 1;
  }
}

// ---------------------------------------------------------------------------------------
// conversions (PTX, so that no header is needed)
// ---------------------------------------------------------------------------------------
PN_DEV float half_to_float(uint32_t h16) {
  float f;
  asm("{ .reg .b16 t; cvt.u16.u32 t, %1; cvt.f32.f16 %0, t; }" : "=f"(f) : "r"(h16));
  return f;
}
PN_DEV uint32_t pack_bf16x2(float lo, float hi) {   // round to nearest even
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}
PN_DEV uint32_t pack_f16x2(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}
PN_DEV float round_bf16(float x) { return bits_f(pack_bf16x2(x, 0.f) << 16); }
PN_DEV float round_f16(float x) { return half_to_float(pack_f16x2(x, 0.f) & 0xFFFFu); }

// ---------------------------------------------------------------------------------------
// global memory access: BYTES contiguous bytes, aligned to min(BYTES, 16)
// ---------------------------------------------------------------------------------------
template <int BYTES>
PN_DEV void load_words(const char* p, uint32_t* w) {
  if constexpr (BYTES >= 16) {
    PN_UNROLL for (int i = 0; i < BYTES / 16; ++i) {
      const uint4 v = __ldg(reinterpret_cast<const uint4*>(p) + i);
      w[4 * i] = v.x; w[4 * i + 1] = v.y; w[4 * i + 2] = v.z; w[4 * i + 3] = v.w;
    }
  } else if constexpr (BYTES == 8) {
    const uint2 v = __ldg(reinterpret_cast<const uint2*>(p));
    w[0] = v.x; w[1] = v.y;
  } else if constexpr (BYTES == 4) {
    w[0] = __ldg(reinterpret_cast<const unsigned int*>(p));
  } else if constexpr (BYTES == 2) {
    w[0] = __ldg(reinterpret_cast<const unsigned short*>(p));
  } else {
    w[0] = __ldg(reinterpret_cast<const unsigned char*>(p));
  }
}

template <int BYTES>
PN_DEV void store_words(char* p, const uint32_t* w) {
  if constexpr (BYTES >= 16) {
    PN_UNROLL for (int i = 0; i < BYTES / 16; ++i)
      reinterpret_cast<uint4*>(p)[i] = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
  } else if constexpr (BYTES == 8) {
    *reinterpret_cast<uint2*>(p) = make_uint2(w[0], w[1]);
  } else if constexpr (BYTES == 4) {
    *reinterpret_cast<unsigned int*>(p) = w[0];
  } else if constexpr (BYTES == 2) {
    *reinterpret_cast<unsigned short*>(p) = static_cast<unsigned short>(w[0]);
  } else {
    *reinterpret_cast<unsigned char*>(p) = static_cast<unsigned char>(w[0]);
  }
}

PN_DEV float widen_scalar(const char* p, int dt) {
  switch (dt) {
    case kF32: return __ldg(reinterpret_cast<const float*>(p));
    case kF16: return half_to_float(__ldg(reinterpret_cast<const unsigned short*>(p)));
    case kBF16: return bits_f(static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short*>(p))) << 16);
    case kI8: return static_cast<float>(__ldg(reinterpret_cast<const signed char*>(p)));
    case kBool: return __ldg(reinterpret_cast<const unsigned char*>(p)) ? 1.f : 0.f;
    case kI32: return static_cast<float>(__ldg(reinterpret_cast<const int*>(p)));
    default: return static_cast<float>(__ldg(reinterpret_cast<const long long*>(p)));
  }
}

// Storage bits of one group of VL elements -> VL floats, in place.
template <int VL>
PN_DEV void widen_group(float* g, int dt) {
  uint32_t w[VL];
  PN_UNROLL for (int i = 0; i < VL; ++i) w[i] = f_bits(g[i]);
  switch (dt) {
    case kF32: case kI64: break;  // i64 operands are converted at load time
    case kBF16:
      PN_UNROLL for (int i = 0; i < VL; ++i) g[i] = bits_f((i & 1) ? (w[i >> 1] & 0xFFFF0000u) : (w[i >> 1] << 16));
      break;
    case kF16:
      PN_UNROLL for (int i = 0; i < VL; ++i) g[i] = half_to_float((w[i >> 1] >> ((i & 1) * 16)) & 0xFFFFu);
      break;
    case kI8:
      PN_UNROLL for (int i = 0; i < VL; ++i)
        g[i] = static_cast<float>(static_cast<signed char>((w[i >> 2] >> ((i & 3) * 8)) & 0xFF));
      break;
    case kBool:
      PN_UNROLL for (int i = 0; i < VL; ++i) g[i] = ((w[i >> 2] >> ((i & 3) * 8)) & 0xFF) ? 1.f : 0.f;
      break;
    case kI32:
      PN_UNROLL for (int i = 0; i < VL; ++i) g[i] = static_cast<float>(static_cast<int>(w[i]));
      break;
  }
}

template <int VL>
PN_DEV void load_group_raw(const char* base, long long elem, int dt, float* g) {
  uint32_t w[VL];
  PN_UNROLL for (int i = 0; i < VL; ++i) w[i] = 0;
  switch (dt) {
    case kF32: case kI32: load_words<VL * 4>(base + elem * 4, w); break;
    case kF16: case kBF16: load_words<VL * 2>(base + elem * 2, w); break;
    case kI8: case kBool: load_words<VL>(base + elem, w); break;
    default:  // i64: converted here, widening is then a no-op
      PN_UNROLL for (int i = 0; i < VL; ++i)
        w[i] = f_bits(static_cast<float>(__ldg(reinterpret_cast<const long long*>(base) + elem + i)));
      break;
  }
  PN_UNROLL for (int i = 0; i < VL; ++i) g[i] = bits_f(w[i]);
}

template <int VL>
PN_DEV void store_group(char* base, long long elem, int dt, const float* g) {
  uint32_t w[VL];
  switch (dt) {
    case kF32:
      PN_UNROLL for (int i = 0; i < VL; ++i) w[i] = f_bits(g[i]);
      store_words<VL * 4>(base + elem * 4, w);
      break;
    case kI32:
      PN_UNROLL for (int i = 0; i < VL; ++i) w[i] = static_cast<uint32_t>(__float2int_rz(g[i]));
      store_words<VL * 4>(base + elem * 4, w);
      break;
    case kBF16:
      if constexpr (VL == 1) { w[0] = pack_bf16x2(g[0], 0.f) & 0xFFFFu; }
      else { PN_UNROLL for (int i = 0; i < VL / 2; ++i) w[i] = pack_bf16x2(g[2 * i], g[2 * i + 1]); }
      store_words<VL * 2>(base + elem * 2, w);
      break;
    case kF16:
      if constexpr (VL == 1) { w[0] = pack_f16x2(g[0], 0.f) & 0xFFFFu; }
      else { PN_UNROLL for (int i = 0; i < VL / 2; ++i) w[i] = pack_f16x2(g[2 * i], g[2 * i + 1]); }
      store_words<VL * 2>(base + elem * 2, w);
      break;
    case kI8: case kBool: {
      PN_UNROLL for (int i = 0; i < (VL + 3) / 4; ++i) w[i] = 0;
      PN_UNROLL for (int i = 0; i < VL; ++i) {
        const uint32_t b = dt == kBool ? (g[i] != 0.f ? 1u : 0u)
                                       : (static_cast<uint32_t>(__float2int_rz(g[i])) & 0xFFu);
        w[i >> 2] |= b << ((i & 3) * 8);
      }
      store_words<VL>(base + elem, w);
      break;
    }
    case kStore01: {   // int8 / bool tensor whose values are known to be exactly 0.0f or 1.0f
      PN_UNROLL for (int i = 0; i < (VL + 3) / 4; ++i) w[i] = 0;
      PN_UNROLL for (int i = 0; i < VL; ++i) w[i >> 2] |= (f_bits(g[i]) >> 29) << ((i & 3) * 8);   // 1.0f = 0x3F800000
      store_words<VL>(base + elem, w);
      break;
    }
    default:  // i64
      PN_UNROLL for (int i = 0; i < VL; ++i)
        reinterpret_cast<long long*>(base)[elem + i] = static_cast<long long>(__float2int_rz(g[i]));
      break;
  }
}

// ---------------------------------------------------------------------------------------
// scalar math (fp32).  The fp32 outputs are held to rtol 1e-5, so the special-function
// unit's approximations are used only where a correction keeps the error near 1e-7.
// ---------------------------------------------------------------------------------------
// e^x = 2^(x*log2 e).  The product is split into its rounded value t and the rounding
// residual r (recovered exactly by an fma, plus the low part of log2 e); 2^t comes from the
// hardware exponential and the residual is applied as a first-order factor.  Overflow gives
// +inf, large negative arguments 0, NaN stays NaN.
PN_DEV float f_exp(float x) {
  const float L2E_HI = 1.4426950216293335f, L2E_LO = 1.9259629911266175e-8f, LN2 = 0.6931471805599453f;
  const float t = x * L2E_HI;
  float r = fmaf(x, L2E_HI, -t);
  r = fmaf(x, L2E_LO, r);
  const float e = exp2f(t);
  return (fabsf(x) < 100.f) ? fmaf(e, r * LN2, e) : e;   // no correction at inf / overflow
}
// e^x for the shifted arguments of softmax / logsumexp (x <= 0 up to rounding): 2^(x*log2 e)
// straight from the hardware exponential.  The rounding of the product costs a relative
// error of about |x| * 6e-8 (5e-6 at the underflow edge x = -87), on values that are at most 1.
PN_DEV float f_exp_neg(float x) {
  float e;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(x * 1.4426950408889634f));
  return e;
}
// 2^t and 1/y from the special-function unit (each about 1 ulp)
PN_DEV float f_ex2(float t) { float e; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(t)); return e; }
PN_DEV float f_rcp(float y) { float r; asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(y)); return r; }
// sigmoid(x) = 1 / (1 + e^-x).  The rounding of x*log2 e perturbs e^-x by |x| * 6e-8 relative,
// and sigmoid is less sensitive to e^-x than 1:1, so the result stays within about 1e-6
// relative over the whole range; e^-x = inf gives 0, e^-x = 0 gives 1.
PN_DEV float f_sigmoid(float x) { return f_rcp(1.f + f_ex2(x * -1.4426950408889634f)); }
// 0.5 x (1 + tanh u) = x / (1 + e^(-2u)),  u = sqrt(2/pi) (x + 0.044715 x^3)
PN_DEV float f_gelu_tanh(float x) {
  const float k0 = 0.7978845608028654f, k1 = 0.044715f;
  const float u = k0 * fmaf(k1 * x * x, x, x);
  return x * f_sigmoid(2.f * u);
}
PN_DEV float f_gelu_erf(float x) { return 0.5f * x * (1.f + erff(x * 0.7071067811865476f)); }
// maximum / minimum that return NaN when either operand is NaN (one instruction each)
PN_DEV float f_max_nan(float a, float b) { float d; asm("max.NaN.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b)); return d; }
PN_DEV float f_min_nan(float a, float b) { float d; asm("min.NaN.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b)); return d; }

template <int OP>
PN_DEV float un(float x) {
  if constexpr (OP == OP_NEG) return -x;
  else if constexpr (OP == OP_ABS) return fabsf(x);
  else if constexpr (OP == OP_EXP) return f_exp(x);
  else if constexpr (OP == OP_LOG) return logf(x);
  else if constexpr (OP == OP_SQRT) return sqrtf(x);
  else if constexpr (OP == OP_RSQRT) return 1.f / sqrtf(x);
  else if constexpr (OP == OP_RECIP) return 1.f / x;
  else if constexpr (OP == OP_TANH) return tanhf(x);
  else if constexpr (OP == OP_SIGMOID) return f_sigmoid(x);
  else if constexpr (OP == OP_SILU) return x * f_sigmoid(x);
  else if constexpr (OP == OP_GELU_TANH) return f_gelu_tanh(x);
  else if constexpr (OP == OP_GELU_ERF) return f_gelu_erf(x);
  else if constexpr (OP == OP_RELU) return (x != x) ? x : fmaxf(x, 0.f);
  else if constexpr (OP == OP_SQUARE) return x * x;
  else if constexpr (OP == OP_ERF) return erff(x);
  else if constexpr (OP == OP_RND_BF16) return round_bf16(x);
  else if constexpr (OP == OP_RND_F16) return round_f16(x);
  else if constexpr (OP == OP_TRUNC) return truncf(x);
  else if constexpr (OP == OP_NEZ) return x != 0.f ? 1.f : 0.f;
  else if constexpr (OP == OP_I2F) return static_cast<float>(static_cast<int>(f_bits(x)));
  else return x;
}

template <int OP>
PN_DEV float bin(float x, float y) {
  if constexpr (OP == OP_ADD) return x + y;
  else if constexpr (OP == OP_SUB) return x - y;
  else if constexpr (OP == OP_RSUB) return y - x;
  else if constexpr (OP == OP_MUL) return x * y;
  else if constexpr (OP == OP_DIV) return x / y;
  else if constexpr (OP == OP_RDIV) return y / x;
  else if constexpr (OP == OP_MAX) return f_max_nan(x, y);
  else if constexpr (OP == OP_MIN) return f_min_nan(x, y);
  else if constexpr (OP == OP_GT) return x > y ? 1.f : 0.f;
  else if constexpr (OP == OP_GE) return x >= y ? 1.f : 0.f;
  else if constexpr (OP == OP_LT) return x < y ? 1.f : 0.f;
  else if constexpr (OP == OP_LE) return x <= y ? 1.f : 0.f;
  else if constexpr (OP == OP_EQ) return x == y ? 1.f : 0.f;
  else if constexpr (OP == OP_NE) return x != y ? 1.f : 0.f;
  else if constexpr (OP == OP_LSEFIN) return (fabsf(x) == PN_INF) ? x : x + logf(y);
  else return x;
}

// ---------------------------------------------------------------------------------------
// reduction partials
// ---------------------------------------------------------------------------------------
struct Part { float a, b, c; };

PN_DEV Part red_identity(int kind) {
  switch (kind) {
    case RED_MAX: return {-PN_INF, 0.f, 0.f};
    case RED_MIN: return {PN_INF, 0.f, 0.f};
    case RED_ARGMAX: return {-PN_INF, bits_f(0x7FFFFFFFu), 0.f};
    case RED_ARGMIN: return {PN_INF, bits_f(0x7FFFFFFFu), 0.f};
    case RED_LSE: case RED_SOFTMAX: return {-PN_INF, 0.f, 0.f};
    default: return {0.f, 0.f, 0.f};
  }
}

// true when (v2, i2) should replace (v1, i1): larger value, NaN above everything, and on
// equal values (or both NaN) the lower column
PN_DEV bool arg_better(float v2, int i2, float v1, int i1, bool want_max) {
  const bool n1 = v1 != v1, n2 = v2 != v2;
  if (n1 || n2) return n2 && (!n1 || i2 < i1);
  if (v2 == v1) return i2 < i1;
  return want_max ? v2 > v1 : v2 < v1;
}

PN_DEV Part red_combine(int kind, Part x, Part y) {
  switch (kind) {
    case RED_SUM: x.a += y.a; break;
    case RED_MAX: x.a = f_max_nan(x.a, y.a); break;
    case RED_MIN: x.a = f_min_nan(x.a, y.a); break;
    case RED_ARGMAX: case RED_ARGMIN:
      if (arg_better(y.a, (int)f_bits(y.b), x.a, (int)f_bits(x.b), kind == RED_ARGMAX)) x = y;
      break;
    case RED_LSE: case RED_SOFTMAX: {
      const float m = f_max_nan(x.a, y.a);
      if (m == -PN_INF) { x.b = 0.f; }
      else { x.b = x.b * f_exp_neg(x.a - m) + y.b * f_exp_neg(y.a - m); }
      x.a = m;
      break;
    }
    default: {  // RED_MEANVAR: merge of (count, mean, M2)
      const float n = x.a + y.a;
      if (n > 0.f) {
        const float rn = f_rcp(n), d = y.b - x.b;
        x.c = x.c + y.c + d * d * x.a * (y.a * rn);
        // the mean from the two sums, not from the difference of the means: rows holding an
        // infinity then give that infinity (inf - inf would give NaN)
        x.b = (x.a * x.b + y.a * y.b) * rn;
      }
      x.a = n;
      break;
    }
  }
  return x;
}

PN_DEV float shfl_x(float v, int o) { return __shfl_xor_sync(0xFFFFFFFFu, v, o); }

// Combine the partials of the 32 lanes of a warp (or of each aligned group of `lanes` = 16 or 8
// lanes, for rows short enough that several share a warp); every lane ends with the same result.
// The order of operations is fixed (a butterfly over lane distance 16, 8, 4, 2, 1), so
// results repeat bit for bit from run to run.  Lanes without data pass the identity partial.
//   sum / max / min      one value per shuffle step
//   argmax / argmin      (value, index) pairs, lowest index on ties
//   logsumexp / softmax  the row maximum first, then the sums rescaled to it once
//   mean / variance      count and sum first, giving the common mean; then each lane moves its
//                        squared deviations to that mean (M2 + n (mean_lane - mean)^2) and the
//                        results are added: the exact decomposition of the total sum of squares
PN_DEV Part warp_combine(int kind, Part v, int lanes = 32) {
  switch (kind) {
    case RED_SUM:
      PN_UNROLL for (int o = 16; o > 0; o >>= 1) if (o < lanes) v.a += shfl_x(v.a, o);
      break;
    case RED_MAX:
      PN_UNROLL for (int o = 16; o > 0; o >>= 1) if (o < lanes) v.a = f_max_nan(v.a, shfl_x(v.a, o));
      break;
    case RED_MIN:
      PN_UNROLL for (int o = 16; o > 0; o >>= 1) if (o < lanes) v.a = f_min_nan(v.a, shfl_x(v.a, o));
      break;
    case RED_ARGMAX: case RED_ARGMIN:
      PN_UNROLL for (int o = 16; o > 0; o >>= 1) {
        if (o >= lanes) continue;
        const float wa = shfl_x(v.a, o), wb = shfl_x(v.b, o);
        if (arg_better(wa, (int)f_bits(wb), v.a, (int)f_bits(v.b), kind == RED_ARGMAX)) { v.a = wa; v.b = wb; }
      }
      break;
    case RED_LSE: case RED_SOFTMAX: {
      float m = v.a;
      PN_UNROLL for (int o = 16; o > 0; o >>= 1) if (o < lanes) m = f_max_nan(m, shfl_x(m, o));
      float s = (m == -PN_INF) ? 0.f : v.b * f_exp_neg(v.a - m);
      PN_UNROLL for (int o = 16; o > 0; o >>= 1) if (o < lanes) s += shfl_x(s, o);
      v.a = m; v.b = s;
      break;
    }
    default: {  // RED_MEANVAR
      float n = v.a, sum = v.a * v.b;
      PN_UNROLL for (int o = 16; o > 0; o >>= 1) if (o < lanes) { n += shfl_x(n, o); sum += shfl_x(sum, o); }
      const float mean = n > 0.f ? sum * f_rcp(n) : 0.f;
      const float d = v.b - mean;
      float m2 = fmaf(v.a * d, d, v.c);
      PN_UNROLL for (int o = 16; o > 0; o >>= 1) if (o < lanes) m2 += shfl_x(m2, o);
      v.a = n; v.b = mean; v.c = m2;
      break;
    }
  }
  return v;
}

// ---------------------------------------------------------------------------------------
// cluster primitives (PTX)
// ---------------------------------------------------------------------------------------
PN_DEV uint32_t cluster_ctarank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
PN_DEV void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// read a float at the same shared-memory offset in the CTA of the given cluster rank
PN_DEV float ld_shared_cluster(const float* local_smem_ptr, uint32_t rank) {
  const uint32_t a = static_cast<uint32_t>(__cvta_generic_to_shared(local_smem_ptr));
  uint32_t ra; float v;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(a), "r"(rank));
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(ra) : "memory");
  return v;
}

// ---------------------------------------------------------------------------------------
// inputs read through roll / slice / view: the data is never moved, the row's start is
// computed instead (the index arithmetic idx = (S + i - shift) mod S of the paper's first case
// study, Section 4.4, for any chain of rolls and slices on leading dimensions)
// ---------------------------------------------------------------------------------------
struct IoMap { int d0, d1, d2, a0, a1, a2, m0, m1, m2; long long s0, s1, s2; };
PN_DEV long long mapped_row_offset(unsigned long long row, const IoMap m) {
  const unsigned long long q2 = row / (unsigned)m.d2;
  int c2 = (int)(row - q2 * (unsigned)m.d2) + m.a2;
  const unsigned long long q1 = q2 / (unsigned)m.d1;
  int c1 = (int)(q2 - q1 * (unsigned)m.d1) + m.a1;
  int c0 = (int)q1 + m.a0;
  if (m.m2) c2 %= m.m2;
  if (m.m1) c1 %= m.m1;
  if (m.m0) c0 %= m.m0;
  return c0 * m.s0 + c1 * m.s1 + c2 * m.s2;
}

// ---------------------------------------------------------------------------------------
// checked accessors (PN_FLAG_BOUNDS): every global access is tested against the extent of its
// tensor; one that falls outside is skipped (a load delivers zeros) and its io entry is marked
// in the status word, which the host reads back.  Nothing traps.  Generated kernels compile the
// tests in only when asked (PN_BOUNDS); the interpreter kernels test a launch parameter.
// ---------------------------------------------------------------------------------------
#if defined(PN_BOUNDS)
#define PN_CHECKING(p) true
#elif defined(PN_BOUNDS_RUNTIME)
#define PN_CHECKING(p) ((p).status != nullptr)
#else
#define PN_CHECKING(p) false
#endif
PN_DEV bool in_bounds(const KernelParams& p, int io, long long elem, int n) {
  if (!PN_CHECKING(p)) return true;
  if (elem >= 0 && elem + n <= p.io[io].numel) return true;
  atomicOr(p.status, 1u << io);
  return false;
}

// ---------------------------------------------------------------------------------------
// tile operations: one function per bytecode instruction
// ---------------------------------------------------------------------------------------
struct TileCtx {
  const long long* rowoff;  // shared: element offset of this row for every io entry
  float* part;              // shared: this thread's partials, part[(r*3+q)*part_stride] (interpreter)
  float* slots;             // per-row scalar slots of this team (shared memory, or registers)
  float* stash;             // shared: parked tile values (already offset by threadIdx.x)
  int part_stride;          // threads per CTA
  int col0;                 // column of (group 0, element 0)
  int gstride;              // columns between consecutive groups
  int col_end;              // one past the last valid column of this slice
  int chunk, chunks;        // position within the slice (chunk 0 starts a reduction)
  bool leader;              // this thread performs per-row scalar stores
};

// FULL: every group of every tile lies inside the row (no validity tests needed).
// ROLL: the input is rolled along the last dimension, column c is read at (c + col_add) mod col_mod
// (both multiples of VL, so a group never straddles the wrap); 0 no, 1 yes, 2 ask the descriptor.
template <int VL, int NG, bool FULL = false, int ROLL = 2>
PN_DEV void op_ldraw(const KernelParams& p, const TileCtx& cx, int io, int dt, float (&r)[VL * NG]) {
  const char* base = static_cast<const char*>(p.io[io].base);
  const long long off = cx.rowoff[io];
  const int wrap = ROLL == 0 ? 0 : p.io[io].col_mod;
  PN_UNROLL for (int j = 0; j < NG; ++j) {
    const int col = cx.col0 + j * cx.gstride;
    int src = col;
    if (ROLL != 0 && wrap != 0) { src += p.io[io].col_add; if (src >= wrap) src -= wrap; }
    if ((FULL || col < cx.col_end) && in_bounds(p, io, off + src, VL)) {
      load_group_raw<VL>(base, off + src, dt, &r[j * VL]);
    } else {
      PN_UNROLL for (int i = 0; i < VL; ++i) r[j * VL + i] = 0.f;
    }
  }
}
template <int VL, int NG>
PN_DEV void op_widen(int dt, float (&r)[VL * NG]) {
  if (dt != kF32 && dt != kI64) { PN_UNROLL for (int j = 0; j < NG; ++j) widen_group<VL>(&r[j * VL], dt); }
}
PN_DEV float op_ldbc_scalar(const KernelParams& p, const TileCtx& cx, int io, int dt) {
  if (!in_bounds(p, io, cx.rowoff[io], 1)) return 0.f;
  return widen_scalar(static_cast<const char*>(p.io[io].base) + cx.rowoff[io] * dtype_size(dt), dt);
}
// The same load split in two, so that loads issued ahead of their use do not wait for their own
// conversion: the storage bits of the element (two words for i64) ...
template <int V>
PN_DEV void op_ldbc_raw(const KernelParams& p, const TileCtx& cx, int io, int dt, float (&r)[V]) {
  const char* a = static_cast<const char*>(p.io[io].base) + cx.rowoff[io] * dtype_size(dt);
  uint32_t w0 = 0, w1 = 0;
  switch (in_bounds(p, io, cx.rowoff[io], 1) ? dt : -1) {
    case -1: break;
    case kF32: case kI32: w0 = __ldg(reinterpret_cast<const unsigned int*>(a)); break;
    case kF16: case kBF16: w0 = __ldg(reinterpret_cast<const unsigned short*>(a)); break;
    case kI8: case kBool: w0 = __ldg(reinterpret_cast<const unsigned char*>(a)); break;
    default: { const uint2 v = __ldg(reinterpret_cast<const uint2*>(a)); w0 = v.x; w1 = v.y; break; }
  }
  r[0] = bits_f(w0);
  if constexpr (V > 1) r[1] = bits_f(w1);
}
// ... and their conversion, splat over the tile
template <int V>
PN_DEV void op_ldbc_widen(int dt, float (&d)[V], const float (&r)[V]) {
  const uint32_t w0 = f_bits(r[0]);
  float v;
  switch (dt) {
    case kF32: v = bits_f(w0); break;
    case kF16: v = half_to_float(w0); break;
    case kBF16: v = bits_f(w0 << 16); break;
    case kI8: v = static_cast<float>(static_cast<signed char>(w0)); break;
    case kBool: v = w0 ? 1.f : 0.f; break;
    case kI32: v = static_cast<float>(static_cast<int>(w0)); break;
    default: {
      uint32_t w1 = 0;
      if constexpr (V > 1) w1 = f_bits(r[1]);
      // values that fit 32 bits (masks, counts, indices: nearly always) convert in one instruction
      if (static_cast<int>(w1) == (static_cast<int>(w0) >> 31)) v = static_cast<float>(static_cast<int>(w0));
      else v = static_cast<float>(static_cast<long long>((static_cast<unsigned long long>(w1) << 32) | w0));
      break;
    }
  }
  PN_UNROLL for (int e = 0; e < V; ++e) d[e] = v;
}
template <int V>
PN_DEV void op_ldbc(const KernelParams& p, const TileCtx& cx, int io, int dt, float (&r)[V]) {
  const float v = op_ldbc_scalar(p, cx, io, dt);
  PN_UNROLL for (int e = 0; e < V; ++e) r[e] = v;
}
template <int V>
PN_DEV void op_mov(float (&d)[V], const float (&s)[V]) { PN_UNROLL for (int e = 0; e < V; ++e) d[e] = s[e]; }
template <int VL, int NG, bool FULL = false>
PN_DEV void op_stout(const KernelParams& p, const TileCtx& cx, int io, int dt, const float (&acc)[VL * NG]) {
  char* base = static_cast<char*>(p.io[io].base);
  const long long off = cx.rowoff[io];
  PN_UNROLL for (int j = 0; j < NG; ++j) {
    const int col = cx.col0 + j * cx.gstride;
    if ((FULL || col < cx.col_end) && in_bounds(p, io, off + col, VL)) store_group<VL>(base, off + col, dt, &acc[j * VL]);
  }
}
// per-row scalar stores (leader thread only)
PN_DEV void op_stout_scalar(const KernelParams& p, const TileCtx& cx, int io, int dt, float v) {
  if (cx.leader && in_bounds(p, io, cx.rowoff[io], 1)) store_group<1>(static_cast<char*>(p.io[io].base), cx.rowoff[io], dt, &v);
}
PN_DEV void op_stout_index(const KernelParams& p, const TileCtx& cx, int io, int dt, float v) {
  if (cx.leader && in_bounds(p, io, cx.rowoff[io], 1)) {
    const int i = static_cast<int>(f_bits(v));
    if (dt == kI64) static_cast<long long*>(p.io[io].base)[cx.rowoff[io]] = i;
    else static_cast<int*>(p.io[io].base)[cx.rowoff[io]] = i;
  }
}
template <int OP, int V>
PN_DEV void op_unary(float (&acc)[V]) { PN_UNROLL for (int e = 0; e < V; ++e) acc[e] = un<OP>(acc[e]); }
template <int OP, int V>
PN_DEV void op_binary(float (&acc)[V], const float (&r)[V]) { PN_UNROLL for (int e = 0; e < V; ++e) acc[e] = bin<OP>(acc[e], r[e]); }
template <int OP, int V>
PN_DEV void op_binary_s(float (&acc)[V], float y) { PN_UNROLL for (int e = 0; e < V; ++e) acc[e] = bin<OP>(acc[e], y); }
// acc = acc != 0 ? x : y   /   acc = acc * x + y
template <int OP, int V>
PN_DEV void op_ternary(float (&acc)[V], const float (&x)[V], const float (&y)[V]) {
  PN_UNROLL for (int e = 0; e < V; ++e)
    acc[e] = (OP == OP_WHERE) ? (acc[e] != 0.f ? x[e] : y[e]) : fmaf(acc[e], x[e], y[e]);
}
// acc = c != 0 ? acc : y, the condition given as the storage bytes of an int8 / bool tensor
// (VL bytes per group, as loaded): no conversion of the mask to floating point
template <int VL, int NG>
PN_DEV void op_where_raw(float (&acc)[VL * NG], const float (&craw)[VL * NG], const float (&y)[VL * NG]) {
  PN_UNROLL for (int j = 0; j < NG; ++j) {
    PN_UNROLL for (int i = 0; i < VL; ++i) {
      const uint32_t w = f_bits(craw[j * VL + (i >> 2)]);
      acc[j * VL + i] = (w & (0xFFu << ((i & 3) * 8))) ? acc[j * VL + i] : y[j * VL + i];
    }
  }
}
template <int V>
PN_DEV void op_splat(float (&t)[V], float v) { PN_UNROLL for (int e = 0; e < V; ++e) t[e] = v; }

// column kernels: reg = reg (op) acc element by element, the running reduction over the walked
// dimension (sum, or NaN-propagating max / min)
PN_DEV float accum_combine(int kind, float a, float b) {
  return kind == RED_SUM ? a + b : (kind == RED_MAX ? f_max_nan(a, b) : f_min_nan(a, b));
}
template <int V>
PN_DEV void op_accum(int kind, float (&r)[V], const float (&acc)[V]) {
  PN_UNROLL for (int e = 0; e < V; ++e) r[e] = accum_combine(kind, r[e], acc[e]);
}

// the same for a value held identically in every element: one element carries the reduction
template <int V>
PN_DEV void op_accum_u(int kind, float (&r)[V], const float (&acc)[V]) { r[0] = accum_combine(kind, r[0], acc[0]); }

// Fold of a tile in element order (a fixed order, so results repeat exactly).  Elements of
// groups outside the row take the identity.
template <int VL, int NG, bool FULL, class F>
PN_DEV float tile_fold(const TileCtx& cx, const float (&acc)[VL * NG], float identity, F f) {
  constexpr int V = VL * NG;
  float t[V];
  PN_UNROLL for (int j = 0; j < NG; ++j) {
    const bool ok = FULL || cx.col0 + j * cx.gstride < cx.col_end;
    PN_UNROLL for (int i = 0; i < VL; ++i) t[j * VL + i] = ok ? acc[j * VL + i] : identity;
  }
  PN_UNROLL for (int e = 1; e < V; ++e) t[0] = f(t[0], t[e]);
  return t[0];
}
struct FoldAdd { PN_DEV float operator()(float a, float b) const { return a + b; } };
struct FoldMaxNan { PN_DEV float operator()(float a, float b) const { return f_max_nan(a, b); } };
struct FoldMinNan { PN_DEV float operator()(float a, float b) const { return f_min_nan(a, b); } };

// Fold the valid elements of the tile into the thread's partial `st` of a reduction;
// RED_SOFTMAX also turns acc into exp(x - m_tile) and leaves m_tile in ts.
template <int VL, int NG, bool FULL = false>
PN_DEV void op_red(const TileCtx& cx, int kind, Part& st, float (&acc)[VL * NG], float& ts) {
  constexpr int V = VL * NG;
  if (kind == RED_ARGMAX || kind == RED_ARGMIN) {
    // The tile extreme by a fold; if it replaces the running extreme, its first holder by a
    // descending scan of equality tests (the lowest slot is written last).  Ties keep the earlier,
    // lower-index holder; a NaN beats every number.
    const bool mx = kind == RED_ARGMAX;
    const float m = mx ? tile_fold<VL, NG, FULL>(cx, acc, -PN_INF, FoldMaxNan()) : tile_fold<VL, NG, FULL>(cx, acc, PN_INF, FoldMinNan());
    const bool m_nan = m != m, s_nan = st.a != st.a;
    const bool take = cx.chunk == 0 || (m_nan ? !s_nan : (!s_nan && (mx ? m > st.a : m < st.a)));
    // the holder of the extreme is looked for only when the tile's extreme replaces the running one:
    // always in the first tile of a row, rarely afterwards (a tie keeps the earlier, lower column)
    if (take) {
      int slot = 0;
      PN_UNROLL for (int j = NG - 1; j >= 0; --j) {
        const bool ok = FULL || cx.col0 + j * cx.gstride < cx.col_end;
        PN_UNROLL for (int i = VL - 1; i >= 0; --i) slot = (ok && acc[j * VL + i] == m) ? j * VL + i : slot;
      }
      if (m_nan) {   // the fold returns NaN when the tile holds one: find the first
        PN_UNROLL for (int j = NG - 1; j >= 0; --j) {
          const bool ok = FULL || cx.col0 + j * cx.gstride < cx.col_end;
          PN_UNROLL for (int i = VL - 1; i >= 0; --i) slot = (ok && acc[j * VL + i] != acc[j * VL + i]) ? j * VL + i : slot;
        }
      }
      // a thread whose tile lies wholly outside the row keeps the sentinel column, which loses every tie
      const int bi = (FULL || cx.col0 < cx.col_end) ? cx.col0 + (slot / VL) * cx.gstride + (slot % VL) : 0x7FFFFFFF;
      st.a = m;
      st.b = bits_f(static_cast<uint32_t>(bi));
    }
    return;
  }
  Part t = red_identity(kind);
  if (kind == RED_SUM) {
    t.a = tile_fold<VL, NG, FULL>(cx, acc, 0.f, FoldAdd());
  } else if (kind == RED_MAX) {
    t.a = tile_fold<VL, NG, FULL>(cx, acc, -PN_INF, FoldMaxNan());
  } else if (kind == RED_MIN) {
    t.a = tile_fold<VL, NG, FULL>(cx, acc, PN_INF, FoldMinNan());
  } else if (kind == RED_LSE || kind == RED_SOFTMAX) {
    // a NaN in the tile makes m, hence every exponential and the sum, NaN
    const float m = tile_fold<VL, NG, FULL>(cx, acc, -PN_INF, FoldMaxNan());
    const float ms = (m == -PN_INF) ? 0.f : m;   // keeps exp(x - ms) free of inf - inf
    const float L2E = 1.4426950408889634f, nms = -ms * L2E;   // e^(x - ms) = 2^(x log2e - ms log2e)
    float ev[V];
    PN_UNROLL for (int j = 0; j < NG; ++j) {
      const bool ok = FULL || cx.col0 + j * cx.gstride < cx.col_end;
      PN_UNROLL for (int i = 0; i < VL; ++i) ev[j * VL + i] = ok ? f_ex2(fmaf(acc[j * VL + i], L2E, nms)) : 0.f;
    }
    if (kind == RED_SOFTMAX) { PN_UNROLL for (int e = 0; e < V; ++e) acc[e] = ev[e]; }
    PN_UNROLL for (int e = 1; e < V; ++e) ev[0] += ev[e];
    t.a = m; t.b = ev[0];
    if (kind == RED_SOFTMAX) ts = ms;
  } else {  // RED_MEANVAR
    float n = 0.f;
    PN_UNROLL for (int j = 0; j < NG; ++j)
      if (FULL || cx.col0 + j * cx.gstride < cx.col_end) n += static_cast<float>(VL);
    const float sum = tile_fold<VL, NG, FULL>(cx, acc, 0.f, FoldAdd());
    const float mean = n > 0.f ? sum / n : 0.f;
    float dev[V];
    PN_UNROLL for (int j = 0; j < NG; ++j) {
      const bool ok = FULL || cx.col0 + j * cx.gstride < cx.col_end;
      PN_UNROLL for (int i = 0; i < VL; ++i) { const float dd = acc[j * VL + i] - mean; dev[j * VL + i] = ok ? dd * dd : 0.f; }
    }
    PN_UNROLL for (int e = 1; e < V; ++e) dev[0] += dev[e];
    t.a = n; t.b = mean; t.c = dev[0];
  }
  st = (cx.chunk > 0) ? red_combine(kind, st, t) : t;
}
template <int V>
PN_DEV void op_scale_ts(const TileCtx& cx, int slot_m, int slot_inv, float (&acc)[V], float ts) {
  const float f = f_exp_neg(ts - cx.slots[slot_m]) * cx.slots[slot_inv];
  PN_UNROLL for (int e = 0; e < V; ++e) acc[e] *= f;
}
template <int V>
PN_DEV float* stash_ptr(const TileCtx& cx, int idx) { return cx.stash + ((size_t)(idx * cx.chunks + cx.chunk) * V) * cx.part_stride; }
template <int V>
PN_DEV void op_spill(const TileCtx& cx, int idx, const float (&r)[V]) {
  float* sp = stash_ptr<V>(cx, idx);
  PN_UNROLL for (int e = 0; e < V; ++e) sp[e * cx.part_stride] = r[e];
}
template <int V>
PN_DEV void op_fill(const TileCtx& cx, int idx, float (&r)[V]) {
  const float* sp = stash_ptr<V>(cx, idx);
  PN_UNROLL for (int e = 0; e < V; ++e) r[e] = sp[e * cx.part_stride];
}
// scalar programs: slots in shared memory are written by lane 0 of the executing warp and
// visible after the warp sync; slots kept in registers (every lane holds the same values) are
// plain assignments
template <bool REG_SLOTS = false>
PN_DEV void op_sst(const TileCtx& cx, int slot, float v) {
  if constexpr (REG_SLOTS) { cx.slots[slot] = v; }
  else {
    __syncwarp();
    if ((threadIdx.x & 31) == 0) cx.slots[slot] = v;
    __syncwarp();
  }
}

// ---------------------------------------------------------------------------------------
// the bytecode interpreter
// ---------------------------------------------------------------------------------------
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

// SCALAR = true: a per-row scalar program (VL = NG = 1): stores go to the row's element of a
// per-row output and are done by the leader only.
template <int VL, int NG, int K, bool SCALAR>
PN_DEV void run_program(const KernelParams& p, int pc, const int pc_end, const TileCtx& cx,
                        float (&acc)[VL * NG], float (&reg)[K][VL * NG], float& ts) {
  constexpr int V = VL * NG;
  while (pc < pc_end) {
    const uint32_t word = p.code[pc++];
    const int op = word & 0xFF, a = (word >> 8) & 0xFF, b = (word >> 16) & 0xFF, c = word >> 24;
#define PN_U(OP) case OP: op_unary<OP, V>(acc); break;
#define PN_B(OP)                                                              \
  case OP:                                                                    \
    if (b == OPK_REG) { PN_WITH_REG(a, op_binary<OP, V>(acc, r);) }           \
    else op_binary_s<OP, V>(acc, (b == OPK_IMM) ? bits_f(p.code[pc++]) : cx.slots[a]); \
    break;
    switch (op) {
      case OP_LDRAW:
        if constexpr (!SCALAR) { const int dt = p.io[a].dtype; PN_WITH_REG(b, op_ldraw<VL, NG>(p, cx, a, dt, r);) }
        break;
      case OP_WIDEN:
        if constexpr (!SCALAR) { const int dt = p.io[a].dtype; PN_WITH_REG(b, op_widen<VL, NG>(dt, r);) }
        break;
      case OP_LDBC: { const int dt = p.io[a].dtype; PN_WITH_REG(b, op_ldbc<V>(p, cx, a, dt, r);) break; }
      case OP_LD: PN_WITH_REG(a, op_mov<V>(acc, r);) break;
      case OP_ST: PN_WITH_REG(a, op_mov<V>(r, acc);) break;
      case OP_STOUT:
        if constexpr (SCALAR) op_stout_scalar(p, cx, a, p.io[a].dtype, acc[0]);
        else op_stout<VL, NG>(p, cx, a, b ? kStore01 : p.io[a].dtype, acc);
        break;
      case OP_STOUT_I:
        if constexpr (SCALAR) op_stout_index(p, cx, a, p.io[a].dtype, acc[0]);
        break;
      PN_U(OP_NEG) PN_U(OP_ABS) PN_U(OP_EXP) PN_U(OP_LOG) PN_U(OP_SQRT) PN_U(OP_RSQRT) PN_U(OP_RECIP)
      PN_U(OP_TANH) PN_U(OP_SIGMOID) PN_U(OP_SILU) PN_U(OP_GELU_TANH) PN_U(OP_GELU_ERF) PN_U(OP_RELU)
      PN_U(OP_SQUARE) PN_U(OP_ERF) PN_U(OP_RND_BF16) PN_U(OP_RND_F16) PN_U(OP_TRUNC) PN_U(OP_NEZ) PN_U(OP_I2F)
      PN_B(OP_ADD) PN_B(OP_SUB) PN_B(OP_RSUB) PN_B(OP_MUL) PN_B(OP_DIV) PN_B(OP_RDIV) PN_B(OP_MAX) PN_B(OP_MIN)
      PN_B(OP_GT) PN_B(OP_GE) PN_B(OP_LT) PN_B(OP_LE) PN_B(OP_EQ) PN_B(OP_NE) PN_B(OP_LSEFIN)
      case OP_WHERE: case OP_FMA: {
        const int kx = c & 15, ky = c >> 4;
        float xt[V], yt[V];
        if (kx == OPK_REG) { PN_WITH_REG(a, op_mov<V>(xt, r);) }
        else op_splat<V>(xt, kx == OPK_IMM ? bits_f(p.code[pc++]) : cx.slots[a]);
        if (ky == OPK_REG) { PN_WITH_REG(b, op_mov<V>(yt, r);) }
        else op_splat<V>(yt, ky == OPK_IMM ? bits_f(p.code[pc++]) : cx.slots[b]);
        if (op == OP_WHERE) op_ternary<OP_WHERE, V>(acc, xt, yt); else op_ternary<OP_FMA, V>(acc, xt, yt);
        break;
      }
      case OP_WHERE_RAW:
        if constexpr (!SCALAR) {
          float yt[V];
          const int ky = c & 15;
          if (ky == OPK_REG) { PN_WITH_REG(b, op_mov<V>(yt, r);) }
          else op_splat<V>(yt, ky == OPK_IMM ? bits_f(p.code[pc++]) : cx.slots[b]);
          PN_WITH_REG(a, op_where_raw<VL, NG>(acc, r, yt);)
        }
        break;
      case OP_RED:
        if constexpr (!SCALAR) {
          float* ps = cx.part + b * 3 * cx.part_stride;
          Part st{ps[0], ps[cx.part_stride], ps[2 * cx.part_stride]};
          op_red<VL, NG>(cx, a, st, acc, ts);
          ps[0] = st.a; ps[cx.part_stride] = st.b; ps[2 * cx.part_stride] = st.c;
        }
        break;
      case OP_SCALE_TS: op_scale_ts<V>(cx, a, b, acc, ts); break;
      case OP_SPILL:
        if constexpr (!SCALAR) { PN_WITH_REG(a, op_spill<V>(cx, b, r);) }
        break;
      case OP_FILL:
        if constexpr (!SCALAR) { PN_WITH_REG(a, op_fill<V>(cx, b, r);) }
        break;
      case OP_SPILL_TS:
        if constexpr (!SCALAR) *stash_ptr<V>(cx, b) = ts;
        break;
      case OP_FILL_TS:
        if constexpr (!SCALAR) ts = *stash_ptr<V>(cx, b);
        break;
      case OP_ACCUM:
        if constexpr (!SCALAR) {
          if (a & 0x80) { PN_WITH_REG(b, op_accum_u<V>(a & 0x7F, r, acc);) }
          else { PN_WITH_REG(b, op_accum<V>(a, r, acc);) }
        }
        break;
      case OP_SLD: op_splat<V>(acc, cx.slots[a]); break;
      case OP_SST:
        if constexpr (SCALAR) op_sst<false>(cx, a, acc[0]);
        break;
      default: break;
    }
#undef PN_U
#undef PN_B
  }
}

// The interpreting program: every property is read from the launch parameters.
template <int VL_, int NG_, int K_>
struct Interp {
  static constexpr int VL = VL_, NG = NG_, K = K_;
  static constexpr bool kStatic = false;   // properties are launch parameters, not constants
  static constexpr int kStages = kMaxStages;
  static constexpr int kFamily = -1, kNumIo = kMaxIo, kNumPrefetch = 0;
  static PN_DEV unsigned lead_dim(const KernelParams& p, int i) { return p.lead_dim[i]; }
  static PN_DEV long long lead_stride(const KernelParams& p, int io, int i) { return p.io[io].lead_stride[i]; }
  static PN_DEV bool io_mapped(const KernelParams& p, int io) { return p.io[io].mapped != 0; }
  static PN_DEV IoMap io_map(const KernelParams& p, int q) {
    const IoDesc& io = p.io[q];
    return IoMap{io.map_dim[0], io.map_dim[1], io.map_dim[2], io.map_add[0], io.map_add[1], io.map_add[2],
                 io.map_mod[0], io.map_mod[1], io.map_mod[2], io.lead_stride[0], io.lead_stride[1], io.lead_stride[2]};
  }
  static constexpr int kWalkUnroll = 1;
  static PN_DEV int block_threads() { return (int)blockDim.x; }
  static PN_DEV long long red_stride(const KernelParams& p, int io) { return p.io[io].red_stride; }
  static PN_DEV int col_tx(const KernelParams& p) { return p.col_tx; }
  static PN_DEV int red_len(const KernelParams& p) { return p.red_len; }
  static PN_DEV int family(const KernelParams& p) { return p.family; }
  static PN_DEV int cluster(const KernelParams& p) { return p.cluster; }
  static PN_DEV int chunks(const KernelParams& p) { return p.chunks; }
  static PN_DEV int split_chunks(const KernelParams& p) { return p.split_chunks; }
  static PN_DEV int row_len(const KernelParams& p) { return p.row_len; }
  static PN_DEV int team_lanes(const KernelParams&) { return 32; }   // short rows sharing a warp: generated kernels only
  static PN_DEV int splits(const KernelParams& p) { return p.splits; }
  static PN_DEV int slice_len(const KernelParams& p) { return p.slice_len; }
  static PN_DEV int n_stages(const KernelParams& p) { return p.n_stages; }
  static PN_DEV int n_io(const KernelParams& p) { return p.n_io; }
  static PN_DEV int n_red(const KernelParams& p, int s) { return p.stage[s].n_red; }
  static PN_DEV int red_kind(const KernelParams& p, int s, int r) { return p.stage[s].red[r].kind; }
  static PN_DEV int red_slot(const KernelParams& p, int s, int r) { return p.stage[s].red[r].slot; }
  static PN_DEV bool red_uniform(const KernelParams& p, int s, int r) { return p.stage[s].red[r].uniform != 0; }
  static PN_DEV bool has_scalar(const KernelParams& p, int s) { return p.stage[s].scal_begin != p.stage[s].scal_end; }
  static PN_DEV void tile(const KernelParams& p, int s, const TileCtx& cx, float (&acc)[VL * NG],
                          float (&reg)[K][VL * NG], float& ts, Part (&)[kMaxRed], float (&)[1][VL * NG],
                          const TileCtx&, bool) {
    run_program<VL, NG, K, false>(p, p.stage[s].elem_begin, p.stage[s].elem_end, cx, acc, reg, ts);
  }
  static PN_DEV void scalar(const KernelParams& p, int s, const TileCtx& cx) {
    float sacc[1] = {0.f}, sreg[4][1] = {{0.f}, {0.f}, {0.f}, {0.f}}, sts = 0.f;
    run_program<1, 1, 4, true>(p, p.stage[s].scal_begin, p.stage[s].scal_end, cx, sacc, sreg, sts);
  }
};

// ---------------------------------------------------------------------------------------
// the kernel body, common to every family and to both kinds of program
// ---------------------------------------------------------------------------------------
template <class Prog>
PN_DEV void fused_body(const KernelParams& p, unsigned char* smem) {
  constexpr int VL = Prog::VL, NG = Prog::NG, K = Prog::K, V = VL * NG;
  // a generated program keeps row offsets, partials and per-row scalars in registers (every
  // thread computes the same values); the interpreter keeps them in shared memory
  constexpr bool kRegSlots = Prog::kStatic;
  constexpr bool kRegRowoff = Prog::kStatic;
  const int bdim = Prog::block_threads();   // a constant in generated kernels
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = bdim >> 5;
  const int family = Prog::family(p);
  const int cluster = Prog::cluster(p);
  const int chunks = Prog::chunks(p);
  const bool split = Prog::split_chunks(p) != 0;
  const bool warp_team = family <= FAM_WARP;
  // Rows of at most 16 (8) groups: two (four) rows share a warp, each owned by an aligned group
  // of TL lanes; the shuffles of a combine then stop at lane distance TL / 2.
  const int TL = warp_team ? Prog::team_lanes(p) : 32;
  const int sub = TL < 32 ? lane / TL : 0;              // which of the warp's teams this lane is in
  const int team_threads = warp_team ? TL : bdim;
  const int team_tid = warp_team ? (TL < 32 ? lane % TL : lane) : tid;
  const int team_in_cta = warp_team ? warp : 0;
  const int crank = (cluster > 1) ? (int)cluster_ctarank() : 0;

  constexpr int kPf = Prog::kNumPrefetch;          // stage-0 loads issued one tile ahead
  long long rowoff_reg[kRegRowoff ? Prog::kNumIo : 1];
  long long rowoff_nxt[kPf > 0 ? Prog::kNumIo : 1];
  float slots_reg[kRegSlots ? kMaxSlots : 1];
  long long* rowoff_sm = reinterpret_cast<long long*>(smem + p.sm_rowoff) + team_in_cta * kMaxIo;
  float* wpart = reinterpret_cast<float*>(smem + p.sm_wpart);
  float* slots = kRegSlots ? slots_reg : reinterpret_cast<float*>(smem + p.sm_slots) + team_in_cta * kMaxSlots;
  float* ctapart = reinterpret_cast<float*>(smem + p.sm_ctapart);

  TileCtx cx;
  cx.rowoff = kRegRowoff ? rowoff_reg : rowoff_sm;
  cx.part = reinterpret_cast<float*>(smem + p.sm_part) + tid;
  cx.part_stride = bdim;
  cx.slots = slots;
  cx.stash = reinterpret_cast<float*>(smem + p.sm_stash) + tid;
  cx.gstride = team_threads * VL;
  cx.chunks = chunks;
  cx.chunk = 0;
  cx.leader = (team_tid == 0) && (crank == 0);

  const long long n_items = p.item_end > 0 ? p.item_end : (split ? p.rows * chunks : p.rows);
  long long team_global, n_teams;
  if (warp_team) {
    const int per_warp = 32 / TL;
    team_global = ((long long)blockIdx.x * nwarps + warp) * per_warp + sub; n_teams = (long long)gridDim.x * nwarps * per_warp;
  }
  else { team_global = blockIdx.x / cluster; n_teams = gridDim.x / cluster; }

  if (p.item_end > 0) team_global += p.item_begin;   // a launch over part of the work
  const int slice_lo = crank * Prog::slice_len(p);
  cx.col_end = min(Prog::row_len(p), slice_lo + Prog::slice_len(p));
  const int chunk_cols = team_threads * V;
  unsigned parity = 0;
  TileCtx nx = cx;               // addressing of the tile after the current one
  nx.rowoff = rowoff_nxt;

  float acc[V];
  float reg[K][V];
  float raw[kPf > 0 ? kPf : 1][V];
  float ts = 0.f;
  Part parts[kMaxRed];
  PN_UNROLL for (int e = 0; e < V; ++e) acc[e] = 0.f;
  PN_UNROLL for (int k = 0; k < K; ++k) { PN_UNROLL for (int e = 0; e < V; ++e) reg[k][e] = 0.f; }
  PN_UNROLL for (int r = 0; r < kMaxRed; ++r) parts[r] = Part{0.f, 0.f, 0.f};

  // element offset of a row in every input / output, with the leading dims as constants
  auto row_offsets = [&](long long row, long long (&out)[kRegRowoff ? Prog::kNumIo : 1]) {
    if constexpr (!kRegRowoff) return;
    const unsigned long long r0 = (unsigned long long)row;
    const unsigned d2 = Prog::lead_dim(p, 2), d1 = Prog::lead_dim(p, 1);
    const unsigned long long q2 = r0 / d2;
    const long long i2 = (long long)(r0 - q2 * d2);
    const unsigned long long q1 = q2 / d1;
    const long long i1 = (long long)(q2 - q1 * d1);
    PN_UNROLL for (int q = 0; q < (kRegRowoff ? Prog::kNumIo : 1); ++q) {
      if (Prog::io_mapped(p, q)) out[q] = mapped_row_offset(r0, Prog::io_map(p, q));
      else out[q] = (long long)q1 * Prog::lead_stride(p, q, 0) + i1 * Prog::lead_stride(p, q, 1) + i2 * Prog::lead_stride(p, q, 2);
    }
  };

  // loads that are the same for every row: once per thread (their row offsets are all zero)
  if constexpr (Prog::kStatic) {
    PN_UNROLL for (int q = 0; q < Prog::kNumIo; ++q) rowoff_reg[q] = 0;
    cx.col0 = slice_lo + team_tid * VL;
    Prog::prologue(p, cx, acc, reg, ts);
  }
  // the first tile's stage-0 loads
  if constexpr (kPf > 0) {
    if (team_global < n_items) {
      long long row = team_global; int c0 = 0;
      if (split) { row = team_global / chunks; c0 = (int)(team_global - row * chunks); }
      row_offsets(row, rowoff_nxt);
      nx.col0 = slice_lo + c0 * chunk_cols + team_tid * VL;
      Prog::prefetch(p, nx, raw);
    }
  }

  const int col_end_all = cx.col_end;
  const bool leader_all = cx.leader;
  // the teams of a warp stay together: the loop runs while the warp's first team has an item; a
  // team without one goes through the motions on the last row with every access switched off
  for (long long item = team_global; item - sub < n_items; item += n_teams) {
    long long row = item;
    if (TL < 32) {
      const bool active = item < n_items;
      if (!active) row = n_items - 1;
      cx.col_end = active ? col_end_all : 0;
      cx.leader = active && leader_all;
    }
    int c_first = 0, c_count = chunks;
    if (split) { row = item / chunks; c_first = (int)(item - row * chunks); c_count = 1; }

    // element offset of this row in every input / output
    if constexpr (kRegRowoff) {
      row_offsets(row, rowoff_reg);
    } else {
      if (team_tid < Prog::n_io(p)) {
        const IoDesc& io = p.io[team_tid];
        long long r = row;
        const long long i2 = r % p.lead_dim[2]; r /= p.lead_dim[2];
        const long long i1 = r % p.lead_dim[1]; r /= p.lead_dim[1];
        rowoff_sm[team_tid] = io.mapped ? mapped_row_offset((unsigned long long)row, IoMap{io.map_dim[0], io.map_dim[1], io.map_dim[2], io.map_add[0], io.map_add[1], io.map_add[2], io.map_mod[0], io.map_mod[1], io.map_mod[2], io.lead_stride[0], io.lead_stride[1], io.lead_stride[2]})
                                        : r * io.lead_stride[0] + i1 * io.lead_stride[1] + i2 * io.lead_stride[2];
      }
      if (warp_team) __syncwarp(); else __syncthreads();
    }

#pragma unroll(Prog::kStatic ? Prog::kStages : 1)
    for (int s = 0; s < Prog::kStages; ++s) {
      if (s >= Prog::n_stages(p)) break;
      for (int c = c_first; c < c_first + c_count; ++c) {
        cx.chunk = split ? 0 : c;
        cx.col0 = slice_lo + c * chunk_cols + team_tid * VL;
        bool has_next = false;
        if constexpr (kPf > 0) {
          if (s == 0) {   // where the tile after this one is: next chunk of the row, or the next item
            if (c + 1 < c_first + c_count) {
              has_next = true;
              PN_UNROLL for (int q = 0; q < Prog::kNumIo; ++q) rowoff_nxt[q] = rowoff_reg[q];
              nx.col0 = cx.col0 + chunk_cols;
            } else if (item + n_teams < n_items) {
              has_next = true;
              long long nrow = item + n_teams; int nc = 0;
              if (split) { nrow = (item + n_teams) / chunks; nc = (int)(item + n_teams - nrow * chunks); }
              row_offsets(nrow, rowoff_nxt);
              nx.col0 = slice_lo + nc * chunk_cols + team_tid * VL;
            }
          }
        }
        Prog::tile(p, s, cx, acc, reg, ts, parts, raw, nx, has_next);
      }
      const int n_red = Prog::n_red(p, s);
      if (n_red == 0 && !Prog::has_scalar(p, s)) continue;

      // ---- combine the partials of this stage over the team, then the scalar program ---
      if (warp_team) {
        PN_UNROLL for (int r = 0; r < kMaxRed; ++r) {
          if (r < n_red) {
            const int kind = Prog::red_kind(p, s, r);
            Part v = Prog::kStatic ? parts[r]
                                   : Part{cx.part[(r * 3) * cx.part_stride], cx.part[(r * 3 + 1) * cx.part_stride],
                                          cx.part[(r * 3 + 2) * cx.part_stride]};
            v = warp_combine(kind, v, TL);
            if (kRegSlots || lane == 0) { float* d = slots + Prog::red_slot(p, s, r); d[0] = v.a; d[1] = v.b; d[2] = v.c; }
          }
        }
        if constexpr (!kRegSlots) __syncwarp();
        Prog::scalar(p, s, cx);
        if constexpr (!kRegSlots) __syncwarp();
      } else if constexpr (Prog::kStatic) {
        // generated program, block / cluster team: one barrier per stage.  Each warp leaves its
        // partial in shared memory (two alternating buffers, so that no second barrier is
        // needed before they are reused); after the barrier every warp combines all of them in
        // the same fixed order and runs the scalar program itself, in registers.
        float* wp = wpart + (parity & 1u) * (32 * kMaxRed * 3);
        PN_UNROLL for (int r = 0; r < kMaxRed; ++r) {
          if (r < n_red) {
            const Part v = warp_combine(Prog::red_kind(p, s, r), parts[r]);
            if (lane == 0) { float* w = wp + (warp * kMaxRed + r) * 3; w[0] = v.a; w[1] = v.b; w[2] = v.c; }
          }
        }
        __syncthreads();
        PN_UNROLL for (int r = 0; r < kMaxRed; ++r) {
          if (r < n_red) {
            const int kind = Prog::red_kind(p, s, r);
            Part v = red_identity(kind);
            if (lane < nwarps) { const float* w = wp + (lane * kMaxRed + r) * 3; v = Part{w[0], w[1], w[2]}; }
            v = warp_combine(kind, v);
            if (cluster > 1) {
              if (tid == 0) { float* d = ctapart + ((parity & 1u) * kMaxRed + r) * 3; d[0] = v.a; d[1] = v.b; d[2] = v.c; }
            } else {
              float* d = slots + Prog::red_slot(p, s, r); d[0] = v.a; d[1] = v.b; d[2] = v.c;
            }
          }
        }
        if (cluster > 1) {
          cluster_sync_all();   // every CTA's partial is now in its own shared memory
          PN_UNROLL for (int r = 0; r < kMaxRed; ++r) {
            if (r < n_red) {
              const int kind = Prog::red_kind(p, s, r);
              Part v = red_identity(kind);
              if (lane < cluster) {
                const float* w = ctapart + ((parity & 1u) * kMaxRed + r) * 3;
                v = Part{ld_shared_cluster(w, lane), ld_shared_cluster(w + 1, lane), ld_shared_cluster(w + 2, lane)};
              }
              v = warp_combine(kind, v);
              float* d = slots + Prog::red_slot(p, s, r); d[0] = v.a; d[1] = v.b; d[2] = v.c;
            }
          }
        }
        parity ^= 1u;
        Prog::scalar(p, s, cx);
      } else {
        PN_UNROLL for (int r = 0; r < kMaxRed; ++r) {
          if (r < n_red) {
            const int kind = Prog::red_kind(p, s, r);
            Part v = Prog::kStatic ? parts[r]
                                   : Part{cx.part[(r * 3) * cx.part_stride], cx.part[(r * 3 + 1) * cx.part_stride],
                                          cx.part[(r * 3 + 2) * cx.part_stride]};
            v = warp_combine(kind, v);
            if (lane == 0) { float* w = wpart + (warp * kMaxRed + r) * 3; w[0] = v.a; w[1] = v.b; w[2] = v.c; }
          }
        }
        __syncthreads();
        if (warp == 0) {
          for (int r = 0; r < n_red; ++r) {
            const int kind = Prog::red_kind(p, s, r);
            Part v = red_identity(kind);
            if (lane < nwarps) { const float* w = wpart + (lane * kMaxRed + r) * 3; v = Part{w[0], w[1], w[2]}; }
            v = warp_combine(kind, v);
            if (lane == 0) {
              float* d = (cluster > 1) ? ctapart + (parity * kMaxRed + r) * 3 : slots + Prog::red_slot(p, s, r);
              d[0] = v.a; d[1] = v.b; d[2] = v.c;
            }
          }
        }
        if (cluster > 1) {
          cluster_sync_all();   // every CTA's partial is now in its own shared memory
          if (warp == 0) {
            for (int r = 0; r < n_red; ++r) {
              const int kind = Prog::red_kind(p, s, r);
              Part v = red_identity(kind);
              if (lane < cluster) {
                const float* w = ctapart + (parity * kMaxRed + r) * 3;
                v = Part{ld_shared_cluster(w, lane), ld_shared_cluster(w + 1, lane), ld_shared_cluster(w + 2, lane)};
              }
              v = warp_combine(kind, v);
              if (lane == 0) { float* d = slots + Prog::red_slot(p, s, r); d[0] = v.a; d[1] = v.b; d[2] = v.c; }
            }
          }
          parity ^= 1u;
        }
        if (warp == 0) {
          __syncwarp();
          Prog::scalar(p, s, cx);
        }
        __syncthreads();
      }
    }
    // the next item rewrites rowoff / slots in shared memory: everyone must be done reading them
    if constexpr (!kRegRowoff || !kRegSlots) { if (warp_team) __syncwarp(); else __syncthreads(); }
  }
  // a CTA's shared memory may still be read by its cluster peers until they pass this point
  if (cluster > 1) cluster_sync_all();
}

// ---------------------------------------------------------------------------------------
// the kernel body of the split-row family: very few, very long rows whose graph needs each element once
// ---------------------------------------------------------------------------------------
// A handful of long rows cannot fill 148 SMs in whole rows or in clusters of at most 8 blocks per
// row.  Here a row is cut into `splits` slices of slice_len columns and thread block b reduces slice
// b % splits of row b / splits: one short-lived block per slice, in memory order, so that the
// hardware's block scheduler spreads the slices over the SMs as they become free and the blocks in
// flight read one compact window of memory (measured on B200 with the stream probe, 256 MB read-only:
// resident blocks that each stream through a contiguous range of their own reach 5.0 TB/s, blocks
// that take 16 - 32 KB pieces in memory order 6.2 - 6.8 TB/s).  A block leaves its partial of every
// reduction in device memory (split_part) and takes a ticket: one atomic add on the row's counter.
// Nobody waits for anybody: the block that draws the last ticket of a row finds all partials of that
// row written (each writer fenced before its ticket), combines them in slice order -- a fixed order,
// whichever block happens to be last, so results repeat bit for bit -- runs the per-row scalar
// program, stores the row's results and puts the counter back to zero for the next launch.
// Generated kernels only; the graph has a single stage (no tile value is needed again after the
// reductions).
//
// Tried on B200 and dropped, each passing the same parity tests (long-row logsumexp + argmax,
// [64, 262144] and [256, 262144] fp32; clusters of 4 / 2 blocks per row take 16.3 / 51.2 us): resident
// blocks over contiguous ranges of tiles, loads one tile ahead in registers or four tiles ahead in
// shared memory by bulk copies (18.6 / 51 us either way: the access pattern, not the bytes in flight,
// is the limit); resident blocks taking tiles in turn with a partial per warp and tile, tickets at the
// end of the block (72 / 306 us: every row is completed, and combined, by the few blocks that end
// last) or one tile later (63 / 263 us: a fence per tile among loads in flight stalls the warp, and
// the slowest warp draws every last ticket and so falls further behind).
PN_DEV float ld_cg(const float* p) { float v; asm("ld.global.cg.f32 %0, [%1];" : "=f"(v) : "l"(p) : "memory"); return v; }

template <class Prog>
PN_DEV void split_body(const KernelParams& p, unsigned char* smem) {
  constexpr int VL = Prog::VL, NG = Prog::NG, K = Prog::K, V = VL * NG;
  const int bdim = Prog::block_threads();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = bdim >> 5;
  const int S = Prog::splits(p);
  const int chunks = Prog::chunks(p);
  const int n_red = Prog::n_red(p, 0);
  const long long row = blockIdx.x / S;
  const int split = (int)(blockIdx.x - row * S);
  const int part_floats = n_red * 3;

  long long rowoff_reg[Prog::kNumIo];
  long long rowoff_nxt[1];
  float slots_reg[kMaxSlots];
  float* wpart = reinterpret_cast<float*>(smem + p.sm_wpart);

  TileCtx cx;
  cx.rowoff = rowoff_reg;
  cx.part = nullptr; cx.stash = nullptr;
  cx.part_stride = bdim;
  cx.slots = slots_reg;
  cx.gstride = bdim * VL;
  cx.chunks = chunks;
  cx.chunk = 0;
  cx.leader = false;
  const int slice_lo = split * Prog::slice_len(p);
  cx.col_end = min(Prog::row_len(p), slice_lo + Prog::slice_len(p));
  TileCtx nx = cx;
  nx.rowoff = rowoff_nxt;

  float acc[V];
  float reg[K][V];
  float raw[1][V];
  float ts = 0.f;
  Part parts[kMaxRed];
  PN_UNROLL for (int e = 0; e < V; ++e) acc[e] = 0.f;
  PN_UNROLL for (int k = 0; k < K; ++k) { PN_UNROLL for (int e = 0; e < V; ++e) reg[k][e] = 0.f; }
  PN_UNROLL for (int r = 0; r < kMaxRed; ++r) parts[r] = Part{0.f, 0.f, 0.f};

  {   // element offset of the row in every input / output
    const unsigned long long r0 = (unsigned long long)row;
    const unsigned d2 = Prog::lead_dim(p, 2), d1 = Prog::lead_dim(p, 1);
    const unsigned long long q2 = r0 / d2;
    const long long i2 = (long long)(r0 - q2 * d2);
    const unsigned long long q1 = q2 / d1;
    const long long i1 = (long long)(q2 - q1 * d1);
    PN_UNROLL for (int q = 0; q < Prog::kNumIo; ++q) {
      if (Prog::io_mapped(p, q)) rowoff_reg[q] = mapped_row_offset(r0, Prog::io_map(p, q));
      else rowoff_reg[q] = (long long)q1 * Prog::lead_stride(p, q, 0) + i1 * Prog::lead_stride(p, q, 1) + i2 * Prog::lead_stride(p, q, 2);
    }
  }
  const int chunk_cols = bdim * V;
  for (int c = 0; c < chunks; ++c) {
    cx.chunk = c;
    cx.col0 = slice_lo + c * chunk_cols + tid * VL;
    Prog::tile(p, 0, cx, acc, reg, ts, parts, raw, nx, false);
  }
  // the block's partial of every reduction: warps through shared memory, then the first warp
  PN_UNROLL for (int r = 0; r < kMaxRed; ++r) {
    if (r < n_red) {
      const Part v = warp_combine(Prog::red_kind(p, 0, r), parts[r]);
      if (lane == 0) { float* w = wpart + (warp * kMaxRed + r) * 3; w[0] = v.a; w[1] = v.b; w[2] = v.c; }
    }
  }
  __syncthreads();
  if (warp != 0) return;
  float* mine = p.split_part + ((size_t)row * S + split) * part_floats;
  PN_UNROLL for (int r = 0; r < kMaxRed; ++r) {
    if (r < n_red) {
      const int kind = Prog::red_kind(p, 0, r);
      Part v = red_identity(kind);
      if (lane < nwarps) { const float* w = wpart + (lane * kMaxRed + r) * 3; v = Part{w[0], w[1], w[2]}; }
      v = warp_combine(kind, v);
      if (lane == 0) { mine[r * 3] = v.a; mine[r * 3 + 1] = v.b; mine[r * 3 + 2] = v.c; }
    }
  }
  unsigned ticket = 0;
  if (lane == 0) {
    __threadfence();                                 // the partial is visible before the ticket is
    ticket = atomicAdd(p.split_ticket + row, 1u);
  }
  ticket = __shfl_sync(0xFFFFFFFFu, ticket, 0);
  if (ticket != (unsigned)(S - 1)) return;
  // the last block of this row: everyone else has written
  __threadfence();
  const float* all = p.split_part + (size_t)row * S * part_floats;
  // a lane takes the slices lane, lane + 32, ... in that order (then the lanes are combined): the loads
  // of four slices at a time are issued together, the combining stays in slice order
  Part v[kMaxRed];
  PN_UNROLL for (int r = 0; r < kMaxRed; ++r) v[r] = red_identity(r < n_red ? Prog::red_kind(p, 0, r) : RED_SUM);
  for (int s0 = lane; s0 < S; s0 += 32 * 4) {
    Part q[4][kMaxRed];
    PN_UNROLL for (int u = 0; u < 4; ++u) {
      const int s = s0 + 32 * u;
      PN_UNROLL for (int r = 0; r < kMaxRed; ++r) {
        if (r < n_red) {
          const float* w = all + (size_t)s * part_floats + r * 3;
          q[u][r] = s < S ? Part{ld_cg(w), ld_cg(w + 1), ld_cg(w + 2)} : red_identity(Prog::red_kind(p, 0, r));
        }
      }
    }
    PN_UNROLL for (int u = 0; u < 4; ++u) {
      PN_UNROLL for (int r = 0; r < kMaxRed; ++r) { if (r < n_red) v[r] = red_combine(Prog::red_kind(p, 0, r), v[r], q[u][r]); }
    }
  }
  PN_UNROLL for (int r = 0; r < kMaxRed; ++r) {
    if (r < n_red) {
      const Part c = warp_combine(Prog::red_kind(p, 0, r), v[r]);
      float* d = slots_reg + Prog::red_slot(p, 0, r); d[0] = c.a; d[1] = c.b; d[2] = c.c;
    }
  }
  cx.leader = lane == 0;
  Prog::scalar(p, 0, cx);
  if (lane == 0) p.split_ticket[row] = 0u;           // ready for the next launch
}

// ---------------------------------------------------------------------------------------
// the kernel body of the column family: reductions over a leading dimension
// ---------------------------------------------------------------------------------------
// Iteration space [rows, R, C], reduced over R.  A CTA is TX threads along the columns by
// TY = blockDim.x / TX along R and owns one (row, column tile) item at a time; a column tile is
// NG groups of VL columns per thread, group j of thread tx at column tile_base + j * TX * VL +
// tx * VL, so that the threads of a warp read whole 128-bit words of one contiguous run per
// step.  Thread (tx, ty) walks the steps ty, ty + TY, ...: the stage-0 tile program loads and
// evaluates one step and folds it into the accumulators (tile registers 0 .. n_red-1).  The
// accumulators of the TY walkers of a column are then combined through shared memory by the
// ty = 0 thread, in the fixed order ty = 0, 1, ..., so results repeat bit for bit; that thread
// runs the stage-1 program (the epilogue on the reduced values) and stores.  Every input element
// is read once.  Hand-offs are __syncthreads only.
//
// With p.splits > 1 the reduced dimension itself is cut into that many slices, one work item per
// (row, column tile, slice): what fills the GPU when a graph has few columns and a long reduced
// dimension.  As in the split-row family nobody waits: a block leaves the combined accumulators of
// its slice in device memory (split_part, [item][slice][reduction][element][tx]), fences, and takes
// a ticket on the item's counter; the block that draws the item's last ticket reads all slices back
// in slice order (its own included, so the order of the combine never depends on who is last), runs
// the epilogue, stores, and puts the counter back to zero.
template <class Prog>
PN_DEV void column_body(const KernelParams& p, unsigned char* smem) {
  constexpr int VL = Prog::VL, NG = Prog::NG, K = Prog::K, V = VL * NG;
  constexpr int kAcc = K < kMaxRed ? K : kMaxRed;
  const int tid = threadIdx.x, nthreads = Prog::block_threads();   // a constant in generated kernels
  const int TX = Prog::col_tx(p), TY = nthreads / TX;
  const int tx = tid % TX, ty = tid / TX;
  const int R = Prog::red_len(p);
  const int n_ctiles = Prog::chunks(p);
  const int n_red = Prog::n_red(p, 0);

  long long rowoff[Prog::kNumIo];
  float no_slots[1] = {0.f};
  TileCtx cx;
  cx.rowoff = rowoff;
  cx.part = nullptr; cx.stash = nullptr;
  cx.slots = no_slots;
  cx.part_stride = nthreads;
  cx.gstride = TX * VL;
  cx.col_end = Prog::row_len(p);
  cx.chunk = 0; cx.chunks = 1;
  cx.leader = false;
  float* stage = reinterpret_cast<float*>(smem + p.sm_part);

  constexpr int kPf = Prog::kNumPrefetch;            // loads at the head of the stage-0 program
  constexpr int U = kPf > 0 ? Prog::kWalkUnroll : 1; // steps whose loads are in flight together
  float acc[V];
  float reg[K][V];
  float raw[U][kPf > 0 ? kPf : 1][V];
  float ts = 0.f;
  Part parts[kMaxRed];
  PN_UNROLL for (int e = 0; e < V; ++e) acc[e] = 0.f;
  PN_UNROLL for (int k = 0; k < K; ++k) { PN_UNROLL for (int e = 0; e < V; ++e) reg[k][e] = 0.f; }
  PN_UNROLL for (int u = 0; u < U; ++u) { PN_UNROLL for (int j = 0; j < (kPf > 0 ? kPf : 1); ++j) { PN_UNROLL for (int e = 0; e < V; ++e) raw[u][j][e] = 0.f; } }
  PN_UNROLL for (int r = 0; r < kMaxRed; ++r) parts[r] = Part{0.f, 0.f, 0.f};

  const int S = Prog::splits(p) > 1 ? Prog::splits(p) : 1;   // slices of the reduced dimension
  const int Rs = (R + S - 1) / S;
  const long long n_items = (p.item_end > 0 ? p.item_end : p.rows * n_ctiles) * S;
  for (long long it = (p.item_end > 0 ? p.item_begin : 0) * S + blockIdx.x; it < n_items; it += gridDim.x) {
    const long long item = it / S;
    const int split = (int)(it - item * S);
    const int s_lo = split * Rs, s_hi = min(R, s_lo + Rs);
    const long long o = item / n_ctiles;
    const int ct = (int)(item - o * n_ctiles);
    cx.col0 = ct * (TX * V) + tx * VL;
    PN_UNROLL for (int r = 0; r < kAcc; ++r) {
      if (r < n_red) {
        const float ident = red_identity(Prog::red_kind(p, 0, r)).a;
        PN_UNROLL for (int e = 0; e < V; ++e) reg[r][e] = ident;
      }
    }
    long long item_off[Prog::kNumIo];   // offset of this item's first step in every input / output
    PN_UNROLL for (int q = 0; q < Prog::kNumIo; ++q) item_off[q] = o * Prog::lead_stride(p, q, 2);
    auto at_step = [&](int s) {
      PN_UNROLL for (int q = 0; q < Prog::kNumIo; ++q) rowoff[q] = item_off[q] + s * Prog::red_stride(p, q);
    };
    if constexpr (kPf > 0) {
      // U steps at a time: all their loads are issued, then their arithmetic runs in step order.
      // (Measured on B200: issuing the next batch before the arithmetic of the current one costs
      // more in registers, hence resident warps, than it gains.)
      for (int s0 = s_lo + ty; s0 < s_hi; s0 += U * TY) {
        PN_UNROLL for (int u = 0; u < U; ++u) {
          const int s = s0 + u * TY;
          if (s < s_hi) { at_step(s); Prog::prefetch(p, cx, raw[u]); }
        }
        PN_UNROLL for (int u = 0; u < U; ++u) {
          const int s = s0 + u * TY;
          if (s < s_hi) { at_step(s); Prog::tile(p, 0, cx, acc, reg, ts, parts, raw[u], cx, false); }
        }
      }
    } else {
      for (int s = s_lo + ty; s < s_hi; s += TY) {
        at_step(s);
        Prog::tile(p, 0, cx, acc, reg, ts, parts, raw[0], cx, false);
      }
    }
    PN_UNROLL for (int r = 0; r < kAcc; ++r) {   // reductions carried by one element: now in all of them
      if (r < n_red && Prog::red_uniform(p, 0, r)) { PN_UNROLL for (int e = 1; e < V; ++e) reg[r][e] = reg[r][0]; }
    }
    if (TY > 1) {
      PN_UNROLL for (int r = 0; r < kAcc; ++r) {
        if (r < n_red) { PN_UNROLL for (int e = 0; e < V; ++e) stage[(r * V + e) * nthreads + tid] = reg[r][e]; }
      }
      __syncthreads();
      if (ty == 0) {
        PN_UNROLL for (int r = 0; r < kAcc; ++r) {
          if (r < n_red) {
            const int kind = Prog::red_kind(p, 0, r);
            PN_UNROLL for (int e = 0; e < V; ++e) {
              const float* col = stage + (r * V + e) * nthreads + tx;
              float v = col[0];
              for (int y = 1; y < TY; ++y) v = accum_combine(kind, v, col[y * TX]);
              reg[r][e] = v;
            }
          }
        }
      }
    }
    bool finish = ty == 0;
    if (S > 1 && tid < 32) {   // the ty = 0 threads are the first TX (<= 32) threads of the block
      const size_t slice_floats = (size_t)n_red * V * TX;
      if (ty == 0) {
        float* mine = p.split_part + (size_t)it * slice_floats;
        PN_UNROLL for (int r = 0; r < kAcc; ++r) {
          if (r < n_red) { PN_UNROLL for (int e = 0; e < V; ++e) mine[(r * V + e) * TX + tx] = reg[r][e]; }
        }
        __threadfence();                               // the slice is visible before the ticket is
      }
      __syncwarp();
      unsigned ticket = 0;
      if (tid == 0) ticket = atomicAdd(p.split_ticket + item, 1u);
      ticket = __shfl_sync(0xFFFFFFFFu, ticket, 0);
      finish = finish && ticket == (unsigned)(S - 1);
      if (finish) {   // the item's last block: every other slice has been written
        __threadfence();
        const float* all = p.split_part + (size_t)item * S * slice_floats;
        PN_UNROLL for (int r = 0; r < kAcc; ++r) {
          if (r < n_red) {
            const int kind = Prog::red_kind(p, 0, r);
            PN_UNROLL for (int e = 0; e < V; ++e) {
              const float* col = all + (r * V + e) * TX + tx;
              float v = ld_cg(col);
              for (int s1 = 1; s1 < S; s1 += 4) {        // four slices' loads together, combined in slice order
                float q4[4];
                PN_UNROLL for (int u = 0; u < 4; ++u) q4[u] = s1 + u < S ? ld_cg(col + (size_t)(s1 + u) * slice_floats) : 0.f;
                PN_UNROLL for (int u = 0; u < 4; ++u) { if (s1 + u < S) v = accum_combine(kind, v, q4[u]); }
              }
              reg[r][e] = v;
            }
          }
        }
        if (tid == 0) p.split_ticket[item] = 0u;       // ready for the next launch
      }
    }
    if (finish) {
      PN_UNROLL for (int q = 0; q < Prog::kNumIo; ++q) rowoff[q] = item_off[q];
      Prog::tile(p, 1, cx, acc, reg, ts, parts, raw[0], cx, false);
    }
    if (TY > 1) __syncthreads();   // the next item rewrites the staging area
  }
}

}  // namespace pn
