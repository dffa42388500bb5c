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
  const PhiloxRoundKeys rk = philox_round_keys(s.key0, s.key1);
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

// Encode / cross-decode / average / store phase of a blocking block, in the fast or the defining form of
// the lattice arithmetic (LatticeOps).
template <int BITS, bool FAST>
__device__ __forceinline__ void blocking_exchange(const f8 (&va)[kSub], const f8 (&vb)[kSub], float* xa, float* xb,
                                                  uint8_t* ca, uint8_t* cb, uint32_t group0, const StoreView& s,
                                                  const PairDesc& pd, int lane, int e) {
  using Ops = LatticeOps<FAST>;
  const float step = pow2f_exact(e), inv_step = pow2f_exact(-e);
  const float unbias = FAST ? -__fmul_rn(kCellBias, step) : 0.0f;
  constexpr uint32_t mask = (1u << BITS) - 1u;
#pragma unroll
  for (int j = 0; j < kSub; ++j) {
    const uint32_t g = group0 + j * (kSubCoords / 8);
    const uint4 ra = philox4x32_10(g, (uint32_t)pd.a, pd.wa, kStreamRounding, s.key0, s.key1);
    const uint4 rb = philox4x32_10(g, (uint32_t)pd.b, pd.wb, kStreamRounding, s.key0, s.key1);
    uint64_t pka = 0, pkb = 0;
    f8 out;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      uint32_t cell_a, cell_b;
      const uint32_t code_a = Ops::encode(va[j].v[i], inv_step, sr_word(ra, i), i & 1, cell_a) & mask;
      const uint32_t code_b = Ops::encode(vb[j].v[i], inv_step, sr_word(rb, i), i & 1, cell_b) & mask;
      pka |= (uint64_t)code_a << (i * BITS);
      pkb |= (uint64_t)code_b << (i * BITS);
      // b decodes a's codes with X^b as key and vice versa; the key's cell is already known
      const float Qa = Ops::value(Ops::template decode<BITS>(code_a, cell_b), step, unbias);
      const float Qb = Ops::value(Ops::template decode<BITS>(code_b, cell_a), step, unbias);
      out.v[i] = __fmul_rn(0.5f, __fadd_rn(Qa, Qb));
    }
    st256(xa + j * kSubCoords, out);
    st256(xb + j * kSubCoords, out);
    store_codes<BITS>(ca + j * (kSubCoords * BITS / 8), lane, pka);
    store_codes<BITS>(cb + j * (kSubCoords * BITS / 8), lane, pkb);
  }
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
  if (fast_range(M, pow2f_exact(-e), e)) blocking_exchange<BITS, true>(va, vb, xa, xb, ca, cb, group0, s, pd, lane, e);
  else blocking_exchange<BITS, false>(va, vb, xa, xb, ca, cb, group0, s, pd, lane, e);
  if (lane == 0) {
    s.exps[(int64_t)pd.a * s.nblk + blk] = (int8_t)e;
    s.exps[(int64_t)pd.b * s.nblk + blk] = (int8_t)e;
  }
}

template <int BITS, bool FAST>
__device__ __forceinline__ void subblock_exchange(const f8& va, const f8& vb, float* xa, float* xb, uint8_t* ca,
                                                  uint8_t* cb, const uint4& ra, const uint4& rb, int lane, int e) {
  using Ops = LatticeOps<FAST>;
  const float step = pow2f_exact(e), inv_step = pow2f_exact(-e);
  const float unbias = FAST ? -__fmul_rn(kCellBias, step) : 0.0f;
  constexpr uint32_t mask = (1u << BITS) - 1u;
  uint64_t pka = 0, pkb = 0;
  f8 out;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    uint32_t cell_a, cell_b;
    const uint32_t code_a = Ops::encode(va.v[i], inv_step, sr_word(ra, i), i & 1, cell_a) & mask;
    const uint32_t code_b = Ops::encode(vb.v[i], inv_step, sr_word(rb, i), i & 1, cell_b) & mask;
    pka |= (uint64_t)code_a << (i * BITS);
    pkb |= (uint64_t)code_b << (i * BITS);
    const float Qa = Ops::value(Ops::template decode<BITS>(code_a, cell_b), step, unbias);
    const float Qb = Ops::value(Ops::template decode<BITS>(code_b, cell_a), step, unbias);
    out.v[i] = __fmul_rn(0.5f, __fadd_rn(Qa, Qb));
  }
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
  const uint4 ra = philox4x32_10(g, (uint32_t)pd.a, pd.wa, kStreamRounding, s.key0, s.key1);
  const uint4 rb = philox4x32_10(g, (uint32_t)pd.b, pd.wb, kStreamRounding, s.key0, s.key1);
  if (fast_range(M, pow2f_exact(-e), e)) subblock_exchange<BITS, true>(va, vb, xa, xb, ca, cb, ra, rb, lane, e);
  else subblock_exchange<BITS, false>(va, vb, xa, xb, ca, cb, ra, rb, lane, e);
  if (j == 0 && lane == 0) {
    s.exps[(int64_t)pd.a * s.nblk + blk] = (int8_t)e;
    s.exps[(int64_t)pd.b * s.nblk + blk] = (int8_t)e;
  }
  // red[] is rewritten only after the next cluster-wide barrier of the caller
}

}  // namespace swarm
