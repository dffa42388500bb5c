// Per-block bodies shared by the interaction kernels and the single-launch sequence kernel: one warp
// handles one 1024-coordinate block of one pair; a lane owns 8 consecutive coordinates in each of the
// block's four 256-coordinate sub-blocks.
#pragma once
#include "swarm_dev.cuh"
#include "swarm_internal.h"

namespace swarm {

constexpr int kSub = 4;          // sub-blocks per block
constexpr int kSubCoords = 256;  // coordinates per sub-block

// Local steps fused into an interaction (synthetic objective): H steps on the lane's 4 x 8 coordinates of
// block blk of `node`, then the padding behind coordinate d of the last block is put back to zero.
__device__ __forceinline__ void fused_steps_block(f8 (&v)[kSub], const StoreView& s, const FusedSteps& fs, int node,
                                                  uint32_t event, int64_t blk, int lane) {
  const float c = fs.scalars[node * 3 + 1];
  const PhiloxRoundKeys& rk = s.rk;
  const uint32_t g0 = (uint32_t)(blk * (kBlockCoords / 8) + lane);
  for (int q = 0; q < fs.H; ++q) {
#pragma unroll
    for (int j = 0; j < kSub; ++j)
      synth_step8(v[j], g0 + j * (kSubCoords / 8), (uint32_t)node, event + (uint32_t)q, fs.lr, fs.grad_std, c, rk);
  }
  if (blk == s.nblk - 1) {
#pragma unroll
    for (int j = 0; j < kSub; ++j)
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if (blk * kBlockCoords + j * kSubCoords + lane * 8 + i >= s.d) v[j].v[i] = 0.0f;
  }
}

// The responder's local steps when the interaction itself does not touch its model.
__device__ __forceinline__ void fused_steps_responder(const StoreView& s, const FusedSteps& fs, const PairDesc& pd,
                                                      int64_t blk, int lane) {
  float* xb = s.X + (int64_t)pd.b * s.pitch + blk * kBlockCoords + lane * 8;
  f8 vb[kSub];
#pragma unroll
  for (int j = 0; j < kSub; ++j) vb[j] = ld256(xb + j * kSubCoords);
  fused_steps_block(vb, s, fs, pd.b, pd.lsb, blk, lane);
#pragma unroll
  for (int j = 0; j < kSub; ++j) st256(xb + j * kSubCoords, vb[j]);
}

// Encode / cross-decode / average of the 8 coordinate pairs a lane owns in one sub-block, in a fast or the
// defining form of the lattice arithmetic (LatticeOps). ra, rb: the generator calls that hold the rounding
// uniforms of the two buffers. ELIDE (fast forms only) leaves the cross-decodes out: when the block's range
// satisfies rho < L * 2^e strictly, |X^a - X^b| < L * 2^e holds for the exact difference of every coordinate
// pair (rho is a maximum of rounded differences, and rounding to nearest cannot carry a value from L * 2^e or
// above to below it), so the two scaled values differ by less than L, their floors by at most L, and the
// encoder's index, floor or floor + 1, lies in the decoder's window [cell - L, cell + L + 1] around the
// partner's cell: Dec returns the encoder's own lattice point (Corollary 1, the case where the writer knows
// the distance to the decoding key). At equality, or with the exponent clamped, the decode stays.
struct ExchangeScale {
  float step, inv_step, unbias, half_step, half_unbias;
};
template <int MODE>
__device__ __forceinline__ ExchangeScale exchange_scale(int e) {
  ExchangeScale sc;
  sc.step = pow2f_exact(e);
  sc.inv_step = pow2f_exact(-e);
  sc.unbias = MODE != kDefining ? -__fmul_rn(kCellBias, sc.step) : 0.0f;
  sc.half_step = __fmul_rn(0.5f, sc.step);                  // 2^(e-1): a subnormal for e = -126, still exact
  sc.half_unbias = __fmul_rn(0.5f, sc.unbias);
  return sc;
}
template <int BITS, int MODE, bool ELIDE>
__device__ __forceinline__ void exchange8(const f8& va, const f8& vb, const uint4& ra, const uint4& rb,
                                          const ExchangeScale& sc, f8& out, uint64_t& pka, uint64_t& pkb) {
  using Ops = LatticeOps<MODE>;
  static_assert(MODE != kDefining || !ELIDE, "the decode is left out in the fast forms only");
  uint32_t ia[8], ib[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    uint32_t cell_a, cell_b;
    ia[i] = Ops::encode(va.v[i], sc.inv_step, sr_word(ra, i), i & 1, cell_a);
    ib[i] = Ops::encode(vb.v[i], sc.inv_step, sr_word(rb, i), i & 1, cell_b);
    // b decodes a's codes with X^b as key and vice versa; the key's cell is already known
    if constexpr (ELIDE) {
      out.v[i] = Ops::mean_of_own(ia[i], ib[i], sc.half_step, sc.half_unbias);
    } else {
      const float Qa = Ops::value(Ops::template decode<BITS>(ia[i], cell_b), sc.step, sc.unbias);
      const float Qb = Ops::value(Ops::template decode<BITS>(ib[i], cell_a), sc.step, sc.unbias);
      out.v[i] = __fmul_rn(0.5f, __fadd_rn(Qa, Qb));
    }
  }
  pka = pack_colours<BITS>(ia);
  pkb = pack_colours<BITS>(ib);
}

template <int BITS, int MODE, bool ELIDE>
__device__ __forceinline__ void blocking_exchange(const f8 (&va)[kSub], const f8 (&vb)[kSub], float* xa, float* xb,
                                                  uint8_t* ca, uint8_t* cb, uint32_t group0, const StoreView& s,
                                                  const PairDesc& pd, int lane, int e) {
  const ExchangeScale sc = exchange_scale<MODE>(e);
#pragma unroll
  for (int j = 0; j < kSub; ++j) {
    const uint32_t g = group0 + j * (kSubCoords / 8);
    const uint4 ra = philox4x32_10(g, (uint32_t)pd.a, pd.wa, kStreamRounding, s.rk);
    const uint4 rb = philox4x32_10(g, (uint32_t)pd.b, pd.wb, kStreamRounding, s.rk);
    uint64_t pka, pkb;
    f8 out;
    exchange8<BITS, MODE, ELIDE>(va[j], vb[j], ra, rb, sc, out, pka, pkb);
    st256(xa + j * kSubCoords, out);
    st256(xb + j * kSubCoords, out);
    store_codes<BITS>(ca + j * (kSubCoords * BITS / 8), lane, pka);
    store_codes<BITS>(cb + j * (kSubCoords * BITS / 8), lane, pkb);
  }
}

// Whether a blocking block may leave the cross-decodes out: rho < L * 2^e strictly (see exchange8).
template <int BITS>
__device__ __forceinline__ bool decode_elidable(float rho, int e) {
  constexpr float L = (float)((1 << (BITS - 1)) - 1);
  return rho < __fmul_rn(L, pow2f_exact(e));
}

// Blocking interaction of one block (Algorithm 1, interaction lines, with both models present): exact
// range of X^a - X^b gives the common exponent; both models are encoded into their buffers; each side
// decodes the partner's codes against its own model and both adopt Q(X^a)/2 + Q(X^b)/2.
template <int BITS, bool FUSED>
__device__ __forceinline__ void blocking_block(const StoreView& s, const PairDesc& pd, int64_t blk, int lane,
                                               const FusedSteps& fs) {
  float* xa = s.X + (int64_t)pd.a * s.pitch + blk * kBlockCoords + lane * 8;
  float* xb = s.X + (int64_t)pd.b * s.pitch + blk * kBlockCoords + lane * 8;

  f8 va[kSub], vb[kSub];
#pragma unroll
  for (int j = 0; j < kSub; ++j) va[j] = ld256(xa + j * kSubCoords);
#pragma unroll
  for (int j = 0; j < kSub; ++j) vb[j] = ld256(xb + j * kSubCoords);
  if constexpr (FUSED) {
    fused_steps_block(va, s, fs, pd.a, pd.lsa, blk, lane);
    if (fs.responders) fused_steps_block(vb, s, fs, pd.b, pd.lsb, blk, lane);
  }

  float rho = 0.0f, M = 0.0f;
#pragma unroll
  for (int j = 0; j < kSub; ++j)
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      rho = fmaxf(rho, fabsf(__fsub_rn(va[j].v[i], vb[j].v[i])));
      M = fmaxf(M, fmaxf(fabsf(va[j].v[i]), fabsf(vb[j].v[i])));
    }
  rho = warp_max_nonneg(rho);
  M = warp_max_nonneg(M);
  const int e = exponent_rule<BITS>(rho, M);

  const uint32_t group0 = (uint32_t)(blk * (kBlockCoords / 8) + lane);   // generator call index of sub-block 0
  uint8_t* ca = s.codes + (int64_t)pd.a * s.nblk * kBlockCoords + blk * (kBlockCoords * BITS / 8) + lane * BITS;
  uint8_t* cb = s.codes + (int64_t)pd.b * s.nblk * kBlockCoords + blk * (kBlockCoords * BITS / 8) + lane * BITS;
  const int mode = lattice_mode(M, pow2f_exact(-e), e);
  const bool elide = mode != kDefining && decode_elidable<BITS>(rho, e);
  if (mode == kFastFma && elide) blocking_exchange<BITS, kFastFma, true>(va, vb, xa, xb, ca, cb, group0, s, pd, lane, e);
  else if (mode == kFastFma) blocking_exchange<BITS, kFastFma, false>(va, vb, xa, xb, ca, cb, group0, s, pd, lane, e);
  else if (mode == kFastMul && elide) blocking_exchange<BITS, kFastMul, true>(va, vb, xa, xb, ca, cb, group0, s, pd, lane, e);
  else if (mode == kFastMul) blocking_exchange<BITS, kFastMul, false>(va, vb, xa, xb, ca, cb, group0, s, pd, lane, e);
  else blocking_exchange<BITS, kDefining, false>(va, vb, xa, xb, ca, cb, group0, s, pd, lane, e);
  if (lane == 0) {
    s.exps[(int64_t)pd.a * s.nblk + blk] = (int8_t)e;
    s.exps[(int64_t)pd.b * s.nblk + blk] = (int8_t)e;
  }
}

template <int BITS, int MODE, bool ELIDE>
__device__ __forceinline__ void subblock_exchange(const f8& va, const f8& vb, float* xa, float* xb, uint8_t* ca,
                                                  uint8_t* cb, const uint4& ra, const uint4& rb, int lane, int e) {
  const ExchangeScale sc = exchange_scale<MODE>(e);
  uint64_t pka, pkb;
  f8 out;
  exchange8<BITS, MODE, ELIDE>(va, vb, ra, rb, sc, out, pka, pkb);
  st256(xa, out);
  st256(xb, out);
  store_codes<BITS>(ca, lane, pka);
  store_codes<BITS>(cb, lane, pkb);
}

// The same interaction with the block spread over four warps of one CTA (warp j takes sub-block j): for
// launches too small to fill the GPU, where the length of one warp's instruction chain is what counts.
// `red` holds 8 floats of shared memory; the four warps meet at named barrier `bar_id` (128 threads).
// Results are identical to blocking_block: the block maxima are order-independent and every coordinate
// keeps its rounding uniform.
template <int BITS>
__device__ __forceinline__ void blocking_subblock(const StoreView& s, const PairDesc& pd, int64_t blk, int j, int lane,
                                                  float* red, int bar_id) {
  float* xa = s.X + (int64_t)pd.a * s.pitch + blk * kBlockCoords + j * kSubCoords + lane * 8;
  float* xb = s.X + (int64_t)pd.b * s.pitch + blk * kBlockCoords + j * kSubCoords + lane * 8;
  const f8 va = ld256(xa), vb = ld256(xb);
  float rho = 0.0f, M = 0.0f;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    rho = fmaxf(rho, fabsf(__fsub_rn(va.v[i], vb.v[i])));
    M = fmaxf(M, fmaxf(fabsf(va.v[i]), fabsf(vb.v[i])));
  }
  rho = warp_max_nonneg(rho);
  M = warp_max_nonneg(M);
  if (lane == 0) { red[j] = rho; red[4 + j] = M; }
  asm volatile("bar.sync %0, 128;" :: "r"(bar_id) : "memory");
  rho = fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3]));
  M = fmaxf(fmaxf(red[4], red[5]), fmaxf(red[6], red[7]));
  const int e = exponent_rule<BITS>(rho, M);
  const uint32_t g = (uint32_t)(blk * (kBlockCoords / 8) + j * (kSubCoords / 8) + lane);
  uint8_t* ca = s.codes + (int64_t)pd.a * s.nblk * kBlockCoords + blk * (kBlockCoords * BITS / 8) +
                j * (kSubCoords * BITS / 8) + lane * BITS;
  uint8_t* cb = s.codes + (int64_t)pd.b * s.nblk * kBlockCoords + blk * (kBlockCoords * BITS / 8) +
                j * (kSubCoords * BITS / 8) + lane * BITS;
  const uint4 ra = philox4x32_10(g, (uint32_t)pd.a, pd.wa, kStreamRounding, s.rk);
  const uint4 rb = philox4x32_10(g, (uint32_t)pd.b, pd.wb, kStreamRounding, s.rk);
  const int mode = lattice_mode(M, pow2f_exact(-e), e);
  const bool elide = mode != kDefining && decode_elidable<BITS>(rho, e);
  if (mode == kFastFma && elide) subblock_exchange<BITS, kFastFma, true>(va, vb, xa, xb, ca, cb, ra, rb, lane, e);
  else if (mode == kFastFma) subblock_exchange<BITS, kFastFma, false>(va, vb, xa, xb, ca, cb, ra, rb, lane, e);
  else if (mode == kFastMul && elide) subblock_exchange<BITS, kFastMul, true>(va, vb, xa, xb, ca, cb, ra, rb, lane, e);
  else if (mode == kFastMul) subblock_exchange<BITS, kFastMul, false>(va, vb, xa, xb, ca, cb, ra, rb, lane, e);
  else subblock_exchange<BITS, kDefining, false>(va, vb, xa, xb, ca, cb, ra, rb, lane, e);
  if (j == 0 && lane == 0) {
    s.exps[(int64_t)pd.a * s.nblk + blk] = (int8_t)e;
    s.exps[(int64_t)pd.b * s.nblk + blk] = (int8_t)e;
  }
  // red[] is rewritten only after the next cluster-wide barrier of the caller
}

}  // namespace swarm
