// Device-side primitives shared by the kernels: counter-based generator, normals,
// lattice quantizer (constructive form of Corollary 1), 256-bit global accesses and
// warp reductions. sm_100a only.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "swarm_internal.h"

namespace swarm {

constexpr int kBlockCoords = 1024;   // coordinates sharing one lattice exponent
constexpr int kExpMin = -126;
constexpr int kExpMax = 119;

// Generator stream ids (fourth counter word).
enum : uint32_t {
  kStreamInit = 1, kStreamDataA = 2, kStreamDataNoise = 3, kStreamXStar = 4,
  kStreamNodeScalars = 5, kStreamTopology = 6, kStreamPairs = 7,
  kStreamMinibatch = 8, kStreamSynthGrad = 9, kStreamRounding = 10, kStreamStepCount = 11, kStreamOwnRounding = 12
};

// ---------------------------------------------------------------------------------------
// Philox-4x32, 10 rounds (Salmon et al., SC'11). Two 32x32->64 multiplies per round.
// ---------------------------------------------------------------------------------------
__host__ __device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                        uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
    const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
    const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    c1 = (uint32_t)p1;
    c3 = (uint32_t)p0;
    c0 = n0;
    c2 = n2;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return make_uint4(c0, c1, c2, c3);
}

// The ten round keys of a generator key (struct in swarm_internal.h): the kernels on the hot path take them
// ready-made from their parameters instead of deriving them in every call.
__host__ __device__ __forceinline__ PhiloxRoundKeys philox_round_keys(uint32_t k0, uint32_t k1) {
  PhiloxRoundKeys rk;
#pragma unroll
  for (int r = 0; r < 10; ++r) { rk.k0[r] = k0 + (uint32_t)r * 0x9E3779B9u; rk.k1[r] = k1 + (uint32_t)r * 0xBB67AE85u; }
  return rk;
}
__host__ __device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                        const PhiloxRoundKeys& rk) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
    const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ rk.k0[r];
    const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ rk.k1[r];
    c1 = (uint32_t)p1;
    c3 = (uint32_t)p0;
    c0 = n0;
    c2 = n2;
  }
  return make_uint4(c0, c1, c2, c3);
}

__host__ __device__ __forceinline__ uint32_t uniform_int(uint32_t word, uint32_t m) {
  return (uint32_t)(((uint64_t)word * m) >> 32);
}

__device__ __forceinline__ float uniform_float(uint32_t word) { return (float)(word >> 8) * 0x1p-24f; }

// Box-Muller on two generator words: u1 in (0, 1], u2 in [0, 1).
__device__ __forceinline__ void normal_pair(uint32_t w0, uint32_t w1, float& z0, float& z1) {
  const float u1 = (float)((w0 >> 8) + 1u) * 0x1p-24f;
  const float u2 = (float)(w1 >> 8) * 0x1p-24f;
  const float r = sqrtf(-2.0f * logf(u1));
  float s, c;
  sincospif(2.0f * u2, &s, &c);
  z0 = r * c;
  z1 = r * s;
}

// Box-Muller with the hardware approximations (lg2, sqrt, sin, cos on the special-function unit),
// for the local-step gradient noise only. Absolute error of a normal: a few 1e-6 (sin/cos: 2^-20.9
// absolute times a radius <= 5.8; radius: relative 4e-6). The noise enters a model coordinate
// multiplied by lr * grad_std, so the model error is lr * grad_std * 4e-6 per step.
//   -ln(u1) for u1 close to 1 comes from the series of -ln(1 - v), v = 1 - u1 (exact in fp32), because
//   lg2 of a number next to 1 has no relative accuracy; the angle 2*pi*u2 is folded to [-pi, pi).
__device__ __forceinline__ float mufu_lg2(float x) { float r; asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x)); return r; }
__device__ __forceinline__ float mufu_sqrt(float x) { float r; asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x)); return r; }
__device__ __forceinline__ float mufu_sin(float x) { float r; asm("sin.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x)); return r; }
__device__ __forceinline__ float mufu_cos(float x) { float r; asm("cos.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x)); return r; }

__device__ __forceinline__ void normal_pair_fast(uint32_t w0, uint32_t w1, float& z0, float& z1) {
  const float u1 = fmaf((float)(w0 >> 8), 0x1p-24f, 0x1p-24f);     // ((w0 >> 8) + 1) * 2^-24, exact
  const float v = 1.0f - u1;                                        // exact: both are multiples of 2^-24
  const float series = v * fmaf(v, fmaf(v, fmaf(v, 0.25f, 0.33333334f), 0.5f), 1.0f);
  const float viaLg2 = -0.69314718f * mufu_lg2(u1);                 // u1 >= 2^-24 is a normal float
  const float nl = v < 0x1p-6f ? series : viaLg2;
  const float r = mufu_sqrt(nl + nl);                               // 0 or >= 3.4e-4: no subnormals
  const float ang = (float)(int32_t)(w1 & 0xFFFFFF00u) * (6.2831853071795865f * 0x1p-32f);
  z0 = r * mufu_cos(ang);
  z1 = r * mufu_sin(ang);
}

__device__ __forceinline__ void normal4_fast(uint32_t group, uint32_t row, uint32_t event, uint32_t stream,
                                             const PhiloxRoundKeys& rk, float z[4]) {
  const uint4 w = philox4x32_10(group, row, event, stream, rk);
  normal_pair_fast(w.x, w.y, z[0], z[1]);
  normal_pair_fast(w.z, w.w, z[2], z[3]);
}

// Four normals of generator call (group, row, event, stream).
__device__ __forceinline__ void normal4(uint32_t group, uint32_t row, uint32_t event, uint32_t stream,
                                        uint32_t k0, uint32_t k1, float z[4]) {
  const uint4 w = philox4x32_10(group, row, event, stream, k0, k1);
  normal_pair(w.x, w.y, z[0], z[1]);
  normal_pair(w.z, w.w, z[2], z[3]);
}

// Residual of one sampled row: least squares <a, x> - b, or logistic regression sigmoid(<a, x>) - y.
__device__ __forceinline__ float row_residual(float dot, float label, int logistic) {
  const float pred = logistic ? 1.0f / (1.0f + expf(-dot)) : dot;
  return pred - label;
}

// ---------------------------------------------------------------------------------------
// Quantizer: lattice of step 2^e, colour = index mod 2^b, L = 2^(b-1) - 1.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ float pow2f_exact(int e) {   // e in [-126, 127]
  return __uint_as_float((uint32_t)(e + 127) << 23);
}

// Least e with L * 2^e >= rho, raised so that M * 2^-e < 2^23, clamped to [-126, 119].
// rho = m * 2^E with m in [0.5, 1): L * 2^(E-b+1) = 2^E (1 - 2^(1-b)) covers rho iff
// m <= 1 - 2^(1-b), i.e. iff the 23-bit mantissa field is <= 2^23 - 2^(25-b); otherwise
// one more doubling is needed. Subnormal or zero rho ends at the lower clamp.
template <int BITS>
__device__ __forceinline__ int exponent_rule(float rho, float M) {
  const uint32_t rb = __float_as_uint(rho);
  int e = kExpMin;
  if (rb >= 0x00800000u) {
    const int E = (int)(rb >> 23) - 126;
    const uint32_t man = rb & 0x007FFFFFu;
    constexpr uint32_t lim = (1u << 23) - (1u << (25 - BITS));
    e = E - BITS + (man <= lim ? 1 : 2);
  }
  const uint32_t mb = __float_as_uint(M);
  if (mb >= 0x00800000u) e = max(e, (int)(mb >> 23) - 126 - 23);
  e = max(e, kExpMin);
  e = min(e, kExpMax);
  return e;
}

// Stochastic rounding onto the lattice with a 16-bit uniform: up with probability
// floor(frac * 2^16) / 2^16. Returns the lattice index; `cell` receives floor(x * 2^-e).
__device__ __forceinline__ int32_t encode_index(float x, float inv_step, uint32_t u16, int32_t& cell) {
  const float t = __fmul_rn(x, inv_step);
  const float f = floorf(t);
  const float frac = __fsub_rn(t, f);
  const uint32_t thr = __float2uint_rz(__fmul_rn(frac, 65536.0f));
  cell = __float2int_rd(t);                     // saturating, like the reference definition
  return (int32_t)((uint32_t)cell + (u16 < thr ? 1u : 0u));
}

// ---------------------------------------------------------------------------------------
// The same lattice arithmetic without conversion instructions. Float<->integer conversions and
// floorf share one quarter-rate unit, which the 8..18 conversions per coordinate of the interaction
// kernels keep busier than HBM does. While every scaled value and lattice index of a block stays inside
// (-2^21, 2^21) and the exponent is at most 100, the same results come from full-rate instructions with
// directed rounding:
//   s = t + C rounded toward -inf, C an integer in [2^23, 2^24) - 2^21, is floor(t) + C exactly (floats are
//   spaced 1 in [2^23, 2^24)). With C = 1.5 * 2^23 its bit pattern is 0x4B400000 + floor(t): a lattice cell
//   "biased" by 0x4B400000. The bias has no low 22 bits, so colours (cell & mask) and the window arithmetic
//   of the decoder work on biased cells unchanged, and a biased index i turns into the value
//   (i - bias) * 2^e with one exact fused multiply-add: as_float(i) * 2^e - 1.5*2^23 * 2^e.
//   Encoder: with C = 1.5 * 2^23 + 192, frac = t + (C - s) is RN(t - floor t), the definition's fraction (it
//   can round up to 1 for a tiny negative t, as there). The 16-bit uniform u becomes the float
//   um = 192 + u / 2^16 by splicing its half word under the bytes 0x43 0x40 with one byte permute; 192 keeps
//   um - frac inside [128, 256), where floats are spaced 2^-16, so um - frac rounded toward +inf is
//   192 + (u - thr) / 2^16 with thr = floor(frac * 2^16), the definition's threshold, and s minus that,
//   again rounded toward +inf, is floor(t) + 1.5 * 2^23 + [u < thr]: the biased lattice index.
// Two fast forms. For e <= 0 the scaled value t = x * 2^-e is an exact product (subnormal x included), so the
// multiply folds into the adds: s = fma(x, 2^-e, C) and frac = fma(x, 2^-e, C - s), six instructions per encoded
// coordinate (kFastFma). For 0 < e <= 100 a tiny x can make the product inexact (a subnormal result), and the
// definition rounds it before taking the floor, so t is formed by a multiply of its own first: seven
// instructions (kFastMul, valid for every e <= 100). LatticeOps<kDefining> is the defining form with saturating
// conversions. All give bit-identical results wherever a fast form is valid; the caller picks the form,
// warp-uniformly, per block.
// ---------------------------------------------------------------------------------------
constexpr float kCellBias = 12582912.0f;            // 1.5 * 2^23
constexpr uint32_t kCellBiasBits = 0x4B400000u;
constexpr float kEncBias = 12583104.0f;             // 1.5 * 2^23 + 192: running sum of the encoder
constexpr float kFastRange = 2097152.0f;            // 2^21: bound on |x| * 2^-e for the fast forms (half the
                                                    // exact limit, which leaves room for the decode window)
constexpr int kFastExpMax = 100;                    // keeps 1.5*2^23 * 2^e finite
enum : int { kDefining = 0, kFastFma = 1, kFastMul = 2 };

template <int MODE>
struct LatticeOps {
  static constexpr bool kFast = MODE != kDefining;
  // x * 2^-e plus an integer constant, rounded toward -inf: floor(t) + c
  static __device__ __forceinline__ float floor_plus(float x, float inv_step, float c, float& t_out) {
    if constexpr (MODE == kFastFma) { t_out = 0.0f; return __fmaf_rd(x, inv_step, c); }
    else { t_out = __fmul_rn(x, inv_step); return __fadd_rd(t_out, c); }
  }
  // (biased) cell of a key: floor(key * 2^-e)
  static __device__ __forceinline__ uint32_t cell(float key, float inv_step) {
    if constexpr (kFast) { float t; return __float_as_uint(floor_plus(key, inv_step, kCellBias, t)); }
    else return (uint32_t)__float2int_rd(__fmul_rn(key, inv_step));
  }
  // (biased) lattice index of x after stochastic rounding with half `hi` (0 low, 1 high) of generator
  // word `w`; `cell` receives the (biased) cell of x.
  static __device__ __forceinline__ uint32_t encode(float x, float inv_step, uint32_t w, int hi, uint32_t& cell_out) {
    if constexpr (kFast) {
      float t;
      const float sft = floor_plus(x, inv_step, kEncBias, t);                          // floor(t) + kEncBias
      const float neg_floor = __fsub_rn(kEncBias, sft);
      const float frac = MODE == kFastFma ? __fmaf_rn(x, inv_step, neg_floor)          // RN(t - floor t), in [0, 1]
                                          : __fadd_rn(t, neg_floor);
      const float um = __uint_as_float(__byte_perm(w, 0x43400000u, hi ? 0x7632 : 0x7610));   // 192 + u / 2^16
      const float gap = __fsub_ru(um, frac);                                           // 192 + (u - thr) / 2^16
      cell_out = __float_as_uint(sft) - 192u;
      return __float_as_uint(__fsub_ru(sft, gap));                                     // floor(t) + bias + [u < thr]
    } else {
      const float t = __fmul_rn(x, inv_step);
      const float f = floorf(t);
      const float frac = __fsub_rn(t, f);
      const uint32_t thr = __float2uint_rz(__fmul_rn(frac, 65536.0f));
      const uint32_t u = hi ? (w >> 16) : (w & 0xFFFFu);
      cell_out = (uint32_t)__float2int_rd(t);
      return cell_out + (u < thr ? 1u : 0u);
    }
  }
  // (biased) index congruent to colour c (mod 2^BITS) in the window [cell - L, cell + L + 1]:
  // cell - L + ((c - cell + L) mod 2^BITS), L = 2^(BITS-1) - 1. Bits of c above the colour are ignored.
  template <int BITS>
  static __device__ __forceinline__ uint32_t decode(uint32_t c, uint32_t cell_in) {
    constexpr uint32_t mask = (1u << BITS) - 1u, L = (1u << (BITS - 1)) - 1u;
    return cell_in - L + ((c - cell_in + L) & mask);
  }
  static __device__ __forceinline__ uint32_t decode_bits(uint32_t c, uint32_t cell_in, int bits) {
    const uint32_t mask = (1u << bits) - 1u, L = (1u << (bits - 1)) - 1u;
    return cell_in - L + ((c - cell_in + L) & mask);
  }
  // value of a (biased) index; `unbias` = -1.5*2^23 * step (fast forms only)
  static __device__ __forceinline__ float value(uint32_t idx, float step, float unbias) {
    if constexpr (kFast) return __fmaf_rn(__uint_as_float(idx), step, unbias);
    else return __fmul_rn(__int2float_rn((int32_t)idx), step);
  }
  // Fast forms: half the sum of the values of two biased indices of magnitude <= 2^21 each (an encoder's own
  // output), (qa + qb) * 2^(e-1). That is what RN(0.5 * RN(Qa + Qb)) comes to, because each product and the sum
  // are exact and (qa + qb) * 2^(e-1) is a float for every e >= -126 (a subnormal at worst). One integer
  // add-add (the sum of two biased patterns minus one bias is the biased sum while |qa + qb| <= 2^22) and one
  // fused multiply-add; `half_step` = 2^(e-1), `half_unbias` = -1.5*2^23 * 2^(e-1).
  static __device__ __forceinline__ float mean_of_own(uint32_t ia, uint32_t ib, float half_step, float half_unbias) {
    static_assert(kFast, "biased indices only");
    return __fmaf_rn(__uint_as_float(ia + ib - kCellBiasBits), half_step, half_unbias);
  }
};

// Eight colours (the low BITS bits of eight lattice indices, coordinate order) as one little-endian bit
// stream of 8 * BITS bits. Widths 2, 4 and 8 merge neighbours with shift-and-select steps that leave
// garbage above each partial byte and drop it with byte permutes.
template <int BITS>
__device__ __forceinline__ uint64_t pack_colours(const uint32_t (&q)[8]) {
  if constexpr (BITS == 8) {
    const uint32_t lo = __byte_perm(__byte_perm(q[0], q[1], 0x0040), __byte_perm(q[2], q[3], 0x0040), 0x5410);
    const uint32_t hi = __byte_perm(__byte_perm(q[4], q[5], 0x0040), __byte_perm(q[6], q[7], 0x0040), 0x5410);
    return (uint64_t)lo | ((uint64_t)hi << 32);
  } else if constexpr (BITS == 4) {
    uint32_t b[4];
#pragma unroll
    for (int t = 0; t < 4; ++t) b[t] = (q[2 * t] & 0xFu) | (q[2 * t + 1] << 4);         // byte t (garbage above bit 7)
    return __byte_perm(__byte_perm(b[0], b[1], 0x0040), __byte_perm(b[2], b[3], 0x0040), 0x5410);
  } else if constexpr (BITS == 2) {
    uint32_t n[4];
#pragma unroll
    for (int t = 0; t < 4; ++t) n[t] = (q[2 * t] & 0x3u) | (q[2 * t + 1] << 2);         // nibble t (garbage above bit 3)
    const uint32_t b0 = (n[0] & 0xFu) | (n[1] << 4), b1 = (n[2] & 0xFu) | (n[3] << 4);
    return __byte_perm(b0, b1, 0x0040) & 0xFFFFu;
  } else {
    constexpr uint32_t mask = (1u << BITS) - 1u;
    uint64_t pk = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) pk |= (uint64_t)(q[i] & mask) << (i * BITS);
    return pk;
  }
}

// The form of the lattice arithmetic that covers a block whose largest magnitude is `maxabs` at exponent e:
// a fast form while maxabs * 2^-e stays below 2^21 and e <= 100, the fused one for e <= 0.
__device__ __forceinline__ int lattice_mode(float maxabs, float inv_step, int e) {
  if (!(__fmul_rn(maxabs, inv_step) < kFastRange) || e > kFastExpMax) return kDefining;
  return e <= 0 ? kFastFma : kFastMul;
}
// For kernels that are built without the multiply form (their fast path is the fused one or none).
__device__ __forceinline__ int lattice_mode_fused_only(float maxabs, float inv_step, int e) {
  return lattice_mode(maxabs, inv_step, e) == kFastFma ? kFastFma : kDefining;
}
// The form that serves two scalings at once.
__device__ __forceinline__ int lattice_mode_both(int m1, int m2) {
  return (m1 == kDefining || m2 == kDefining) ? kDefining : ((m1 == kFastFma && m2 == kFastFma) ? kFastFma : kFastMul);
}
// Runs CALL with the compile-time constant M set to the run-time form `mode`.
#define SWARM_LATTICE_DISPATCH(mode, ...)                                   \
  switch (mode) {                                                           \
    case kFastFma: { constexpr int M = kFastFma; __VA_ARGS__; } break;      \
    case kFastMul: { constexpr int M = kFastMul; __VA_ARGS__; } break;      \
    default: { constexpr int M = kDefining; __VA_ARGS__; } break;           \
  }

// Generator word holding the 16-bit rounding uniform of coordinate i (0..7) of a call covering 8
// consecutive coordinates (low half for even i, high half for odd i).
__device__ __forceinline__ uint32_t sr_word(const uint4& w, int i) {
  return (i < 2) ? w.x : (i < 4) ? w.y : (i < 6) ? w.z : w.w;
}
// 16-bit rounding uniform i (0..7) of a generator call covering 8 consecutive coordinates.
__device__ __forceinline__ uint32_t sr_u16(const uint4& w, int i) {
  const uint32_t word = (i < 2) ? w.x : (i < 4) ? w.y : (i < 6) ? w.z : w.w;
  return (i & 1) ? (word >> 16) : (word & 0xFFFFu);
}

// ---------------------------------------------------------------------------------------
// 256-bit global accesses (one lane moves 8 consecutive floats; 32-byte aligned).
// ---------------------------------------------------------------------------------------
struct alignas(32) f8 { float v[8]; };

__device__ __forceinline__ f8 ld256(const float* p) {
  f8 r;
  asm volatile("ld.global.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=f"(r.v[0]), "=f"(r.v[1]), "=f"(r.v[2]), "=f"(r.v[3]),
                 "=f"(r.v[4]), "=f"(r.v[5]), "=f"(r.v[6]), "=f"(r.v[7])
               : "l"(p));
  return r;
}

__device__ __forceinline__ void st256(float* p, const f8& r) {
  asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
               :: "l"(p), "f"(r.v[0]), "f"(r.v[1]), "f"(r.v[2]), "f"(r.v[3]),
                  "f"(r.v[4]), "f"(r.v[5]), "f"(r.v[6]), "f"(r.v[7])
               : "memory");
}

// One synthetic-gradient local step x <- x - lr * (c + grad_std * z) on the 8 consecutive coordinates of
// coordinate group g8 (first coordinate / 8): two generator calls, every operation rounded on its own.
// The one definition serves the stand-alone local-step kernel and the steps fused into an interaction.
__device__ __forceinline__ void synth_step8(f8& v, uint32_t g8, uint32_t node, uint32_t event, float lr,
                                            float grad_std, float c, const PhiloxRoundKeys& rk) {
  float z[8];
  normal4_fast(2u * g8, node, event, kStreamSynthGrad, rk, z);
  normal4_fast(2u * g8 + 1u, node, event, kStreamSynthGrad, rk, z + 4);
#pragma unroll
  for (int t = 0; t < 8; ++t) {
    const float grad = __fadd_rn(c, __fmul_rn(grad_std, z[t]));
    v.v[t] = __fsub_rn(v.v[t], __fmul_rn(lr, grad));
  }
}

// Eight packed codes of one lane: BITS bytes at `p` = (the warp's 32*BITS-byte run) + lane*BITS. A block's
// codes are a little-endian bit stream (code of local coordinate k at bits [k*BITS, (k+1)*BITS)), so a lane's
// 8 coordinates always fill whole bytes. Widths 2, 4, 8 give naturally aligned 2-, 4-, 8-byte accesses.
// Widths 3, 5, 6, 7 are called by all 32 lanes together: the store regroups the run into aligned 32-bit
// words through shuffles (each word takes bytes from at most two neighbouring lanes); the load reads the two
// aligned 8-byte words that cover the lane's bytes (rows keep >= 128 spare bytes behind the last run).
template <int BITS>
__device__ __forceinline__ void store_codes(uint8_t* p, int lane, uint64_t packed) {
  if constexpr (BITS == 8) *reinterpret_cast<uint2*>(p) = make_uint2((uint32_t)packed, (uint32_t)(packed >> 32));
  else if constexpr (BITS == 4) *reinterpret_cast<uint32_t*>(p) = (uint32_t)packed;
  else if constexpr (BITS == 2) *reinterpret_cast<uint16_t*>(p) = (uint16_t)packed;
  else {
    uint32_t* run = reinterpret_cast<uint32_t*>(p - lane * BITS);
    constexpr int kWords = 8 * BITS;                 // 32-bit words in the run
#pragma unroll
    for (int r = 0; r < (kWords + 31) / 32; ++r) {
      const int w = r * 32 + lane;
      const int src = (4 * w) / BITS;                // lane holding the word's first byte
      const int off = 4 * w - src * BITS;            // ... at this byte of its BITS bytes
      const uint64_t p0 = __shfl_sync(0xFFFFFFFFu, packed, min(src, 31));
      const uint64_t p1 = __shfl_sync(0xFFFFFFFFu, packed, min(src + 1, 31));
      const uint64_t both = (p0 >> (8 * off)) | (p1 << (8 * (BITS - off)));
      if (w < kWords) run[w] = (uint32_t)both;
    }
  }
}
template <int BITS>
__device__ __forceinline__ uint64_t load_codes(const uint8_t* p) {
  if constexpr (BITS == 8) { const uint2 v = *reinterpret_cast<const uint2*>(p); return (uint64_t)v.x | ((uint64_t)v.y << 32); }
  else if constexpr (BITS == 4) return *reinterpret_cast<const uint32_t*>(p);
  else if constexpr (BITS == 2) return *reinterpret_cast<const uint16_t*>(p);
  else {
    const uintptr_t addr = reinterpret_cast<uintptr_t>(p);
    const uint64_t* q = reinterpret_cast<const uint64_t*>(addr & ~(uintptr_t)7);
    const int sh = (int)(addr & 7) * 8;
    const uint64_t lo = q[0], hi = q[1];
    const uint64_t v = sh ? ((lo >> sh) | (hi << (64 - sh))) : lo;
    return v & ((1ull << (8 * BITS)) - 1ull);
  }
}

// Warp-wide maximum of non-negative floats (bit pattern order equals value order).
__device__ __forceinline__ float warp_max_nonneg(float v) {
  return __uint_as_float(__reduce_max_sync(0xFFFFFFFFu, __float_as_uint(v)));
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}

}  // namespace swarm
