// Fused pairwise-interaction kernels (Algorithm 1, interaction lines; Corollary 1 Enc/Dec).
//
// Work decomposition: one warp owns one 1024-coordinate block of one pair. The block is
// four 256-coordinate sub-blocks; in each, a lane owns 8 consecutive coordinates, so that
//   * one 256-bit load/store per lane moves its coordinates (a warp covers 1 KiB contiguous),
//   * one Philox call yields exactly the lane's eight 16-bit rounding uniforms,
//   * the lane's eight b-bit codes pack into b contiguous bytes of the buffer.
// Rows are padded with zeros to a multiple of 1024, and zeros encode to code 0 and decode
// to 0, so the tail block needs no bounds checks and its padding stays zero.
#include "swarm_dev.cuh"
#include "swarm_internal.h"
#include "swarm_blocks.cuh"

namespace swarm {

constexpr int kWarpsPerCta = 4;

// Programmatic dependent launch: a kernel launched with the stream-serialization attribute may become
// resident while its predecessor in the stream drains; it must not touch global memory before
// grid_dependency_wait() returns (predecessor complete and flushed). Signalling early lets the
// successor's CTAs occupy SM slots as soon as this grid has none left to schedule, which hides the
// launch latency between back-to-back interaction launches.
// L2 prefetch of one 128-byte line. Before its own loads a warp asks for the lines of the block that the
// warp a few hundred warp indices later will work on (a fraction of the resident wave), so that block's
// demand loads hit L2 instead of waiting on HBM; this adds memory-level parallelism without holding registers.
__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" :: "l"(p)); }
constexpr int64_t kPrefetchDistance = 444;            // warps ahead; swept 148..2368 on B200 (best 300..600)
constexpr int64_t kPrefetchDistanceRegisters = 296;   // the register-protocol kernel keeps fewer warps resident

// The (pair, block) that the warp `ahead` warp indices after this one works on; false past the end of the
// launch. A launch has fewer than 2^31 warps (checked by the launch wrappers), for which the multiplier and
// shift in the store view give the exact quotient by the number of blocks per row.
__device__ __forceinline__ bool warp_slot(int64_t total_warps, const StoreView& s, uint32_t ahead, uint32_t& pair,
                                          uint32_t& blk) {
  uint32_t warp = blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5) + ahead;
  if (warp >= (uint32_t)total_warps) return false;
  if (s.backwards) warp = (uint32_t)total_warps - 1u - warp;
  pair = s.nblk_magic ? __umulhi(warp, s.nblk_magic) >> s.nblk_shift : warp;
  blk = warp - pair * (uint32_t)s.nblk;
  return true;
}

// The first warps of a launch have no earlier warp that asks for their lines; they ask themselves, and do so before
// they wait for the previous launch: a prefetch only moves a line into L2, the point of coherence, so it may
// precede the last writes to that line. (Not in the two-register kernel, which ran 1 % slower with it.)
__device__ __forceinline__ bool first_warps(int64_t distance) {
  return (int64_t)blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5) < distance;
}
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_signal() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
// -----------------------------------------------------------------------------------------
// Blocking interaction: both models are present. Per block: exact range of X^a - X^b gives
// the common exponent; both are encoded into their buffers; each side decodes the partner's
// codes against its own model and both adopt Q(X^a)/2 + Q(X^b)/2.
// Traffic per coordinate: 8 B read, 8 B written, 2*b/8 B of codes written.
// -----------------------------------------------------------------------------------------
template <int BITS, bool FUSED>
__global__ void __launch_bounds__(kWarpsPerCta * 32, 4)   // 128 registers: four CTAs per SM at every code width
interact_blocking_kernel(StoreView s, const PairList pairs, int64_t total_warps, const FusedSteps fs) {
  grid_dependency_signal();
  const int lane = threadIdx.x & 31;
  auto prefetch_block = [&](uint32_t ahead) {
    uint32_t pair2, blk2_32;
    if (warp_slot(total_warps, s, ahead, pair2, blk2_32)) {
      const int64_t blk2 = blk2_32;
      const PairDesc p2 = pairs.get(pair2);
      prefetch_l2(s.X + (int64_t)p2.a * s.pitch + blk2 * kBlockCoords + lane * 32);     // 32 lines of 128 B
      prefetch_l2(s.X + (int64_t)p2.b * s.pitch + blk2 * kBlockCoords + lane * 32);
    }
  };
  if (first_warps(kPrefetchDistance)) prefetch_block(0);
  grid_dependency_wait();
  uint32_t pair, blk32;
  if (!warp_slot(total_warps, s, 0, pair, blk32)) return;
  const int64_t blk = blk32;
  const PairDesc pd = pairs.get(pair);
  prefetch_block((uint32_t)kPrefetchDistance);

  blocking_block<BITS, FUSED>(s, pd, blk, lane, fs);
}

// Identity quantizer (Corollary 2): plain averaging, buffers untouched.
__global__ void __launch_bounds__(kWarpsPerCta * 32)
interact_identity_kernel(StoreView s, const PairList pairs, int64_t total_warps, const FusedSteps fs) {
  grid_dependency_signal();
  const int lane = threadIdx.x & 31;
  auto prefetch_block = [&](uint32_t ahead) {
    uint32_t pair2, blk2_32;
    if (warp_slot(total_warps, s, ahead, pair2, blk2_32)) {
      const int64_t blk2 = blk2_32;
      const PairDesc p2 = pairs.get(pair2);
      prefetch_l2(s.X + (int64_t)p2.a * s.pitch + blk2 * kBlockCoords + lane * 32);
      prefetch_l2(s.X + (int64_t)p2.b * s.pitch + blk2 * kBlockCoords + lane * 32);
    }
  };
  if (first_warps(kPrefetchDistance)) prefetch_block(0);
  grid_dependency_wait();
  uint32_t pair, blk32;
  if (!warp_slot(total_warps, s, 0, pair, blk32)) return;
  const int64_t blk = blk32;
  const PairDesc pd = pairs.get(pair);
  prefetch_block((uint32_t)kPrefetchDistance);
  float* xa = s.X + (int64_t)pd.a * s.pitch + blk * kBlockCoords + lane * 8;
  float* xb = s.X + (int64_t)pd.b * s.pitch + blk * kBlockCoords + lane * 8;
  f8 va[kSub], vb[kSub];
#pragma unroll
  for (int j = 0; j < kSub; ++j) va[j] = ld256(xa + j * kSubCoords);
#pragma unroll
  for (int j = 0; j < kSub; ++j) vb[j] = ld256(xb + j * kSubCoords);
  if (fs.H > 0) {
    fused_steps_block(va, s, fs, pd.a, pd.lsa, blk, lane);
    if (fs.responders) fused_steps_block(vb, s, fs, pd.b, pd.lsb, blk, lane);
  }
#pragma unroll
  for (int j = 0; j < kSub; ++j) {
    f8 out;
#pragma unroll
    for (int i = 0; i < 8; ++i) out.v[i] = __fmul_rn(0.5f, __fadd_rn(va[j].v[i], vb[j].v[i]));
    st256(xa + j * kSubCoords, out);
    st256(xb + j * kSubCoords, out);
  }
}

// Decode phase of a non-blocking block: nx holds X^a and av the snapshot B^a (the key) on entry; on return
// nx holds the new model and av the average. Block maxima for the guard rule come back warp-reduced.
template <int BITS, int MODE>
__device__ __forceinline__ void nonblocking_decode(f8 (&nx)[kSub], f8 (&av)[kSub], const uint64_t (&pa)[kSub],
                                                   const uint64_t (&pb)[kSub], int e_own, int e_oth, float& spread_out,
                                                   float& dmax_out, float& M_out) {
  using Ops = LatticeOps<MODE>;
  const float step_own = pow2f_exact(e_own), inv_own = pow2f_exact(-e_own);
  const float step_oth = pow2f_exact(e_oth), inv_oth = pow2f_exact(-e_oth);
  const float unb_own = Ops::kFast ? -__fmul_rn(kCellBias, step_own) : 0.0f;
  const float unb_oth = Ops::kFast ? -__fmul_rn(kCellBias, step_oth) : 0.0f;
  float spread = 0.0f, dmax = 0.0f, M = 0.0f;
#pragma unroll
  for (int j = 0; j < kSub; ++j)
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float key = av[j].v[i];
      // colours with whatever follows them in the stream above: the decoder reads the low BITS bits only
      const uint32_t code_own = (uint32_t)(pa[j] >> (i * BITS)), code_oth = (uint32_t)(pb[j] >> (i * BITS));
      const float own = Ops::value(Ops::template decode<BITS>(code_own, Ops::cell(key, inv_own)), step_own, unb_own);
      const float oth = Ops::value(Ops::template decode<BITS>(code_oth, Ops::cell(key, inv_oth)), step_oth, unb_oth);
      const float avg = __fmul_rn(0.5f, __fadd_rn(own, oth));
      const float D = __fsub_rn(key, nx[j].v[i]);
      const float x_new = __fsub_rn(avg, D);
      spread = fmaxf(spread, fabsf(__fsub_rn(own, oth)));
      dmax = fmaxf(dmax, fabsf(D));
      M = fmaxf(M, fmaxf(fabsf(x_new), fabsf(avg)));
      nx[j].v[i] = x_new;
      av[j].v[i] = avg;
    }
  spread_out = warp_max_nonneg(spread);
  dmax_out = warp_max_nonneg(dmax);
  M_out = warp_max_nonneg(M);
}

// Encode phase: the new model goes to X^a, B^a and (encoded) to a's buffer, the average (encoded) to b's.
template <int BITS, int MODE>
__device__ __forceinline__ void nonblocking_encode(const f8 (&nx)[kSub], const f8 (&av)[kSub], float* xa, float* ba,
                                                   uint8_t* ca, uint8_t* cb, uint32_t group0, const StoreView& s,
                                                   const PairDesc& pd, int lane, int e) {
  using Ops = LatticeOps<MODE>;
  const float inv_step = pow2f_exact(-e);
#pragma unroll
  for (int j = 0; j < kSub; ++j) {
    const uint32_t g = group0 + j * (kSubCoords / 8);
    const uint4 ra = philox4x32_10(g, (uint32_t)pd.a, pd.wa, kStreamRounding, s.rk);
    const uint4 rb = philox4x32_10(g, (uint32_t)pd.b, pd.wb, kStreamRounding, s.rk);
    uint32_t qa[8], qb[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      uint32_t cell;
      qa[i] = Ops::encode(nx[j].v[i], inv_step, sr_word(ra, i), i & 1, cell);
      qb[i] = Ops::encode(av[j].v[i], inv_step, sr_word(rb, i), i & 1, cell);
    }
    st256(xa + j * kSubCoords, nx[j]);
    st256(ba + j * kSubCoords, nx[j]);
    store_codes<BITS>(ca + j * (kSubCoords * BITS / 8), lane, pack_colours<BITS>(qa));
    store_codes<BITS>(cb + j * (kSubCoords * BITS / 8), lane, pack_colours<BITS>(qb));
  }
}

// -----------------------------------------------------------------------------------------
// Non-blocking interaction (the single-buffer form of Algorithm 1): the initiator a decodes
// its own buffer and the responder's buffer with its base snapshot B^a as key, averages,
// subtracts its pending local update D = B^a - X^a, adopts the result as X^a and B^a, and
// writes Enc(new X^a) to its own buffer and Enc(average) to the responder's buffer.
// X^b and B^b are not read or written. The new exponent comes from the guard rule
// rho' = 2 max|own - oth| + max|D| over the block.
// Traffic per coordinate: 8 B + 2*b/8 B read, 8 B + 2*b/8 B written.
// -----------------------------------------------------------------------------------------
template <int BITS, bool FUSED>
__global__ void __launch_bounds__(kWarpsPerCta * 32, 4)     // 128 registers: four CTAs per SM
interact_nonblocking_kernel(StoreView s, const PairList pairs, int64_t total_warps, const FusedSteps fs) {
  grid_dependency_signal();
  const int lane = threadIdx.x & 31;
  auto prefetch_block = [&](uint32_t ahead) {
    uint32_t pair2, blk2_32;
    if (warp_slot(total_warps, s, ahead, pair2, blk2_32)) {
      const int64_t blk2 = blk2_32;
      const PairDesc p2 = pairs.get(pair2);
      prefetch_l2(s.X + (int64_t)p2.a * s.pitch + blk2 * kBlockCoords + lane * 32);     // 32 lines of 128 B
      prefetch_l2(s.B + (int64_t)p2.a * s.pitch + blk2 * kBlockCoords + lane * 32);
      if (lane < BITS) {                                                                 // 128 * BITS bytes of codes
        prefetch_l2(s.codes + (int64_t)p2.a * s.nblk * kBlockCoords + blk2 * (kBlockCoords * BITS / 8) + lane * 128);
        prefetch_l2(s.codes + (int64_t)p2.b * s.nblk * kBlockCoords + blk2 * (kBlockCoords * BITS / 8) + lane * 128);
      }
    }
  };
  if (first_warps(kPrefetchDistance)) prefetch_block(0);
  grid_dependency_wait();
  uint32_t pair, blk32;
  if (!warp_slot(total_warps, s, 0, pair, blk32)) return;
  const int64_t blk = blk32;
  const PairDesc pd = pairs.get(pair);
  prefetch_block((uint32_t)kPrefetchDistance);

  float* xa = s.X + (int64_t)pd.a * s.pitch + blk * kBlockCoords + lane * 8;
  float* ba = s.B + (int64_t)pd.a * s.pitch + blk * kBlockCoords + lane * 8;
  uint8_t* ca = s.codes + (int64_t)pd.a * s.nblk * kBlockCoords + blk * (kBlockCoords * BITS / 8) + lane * BITS;
  uint8_t* cb = s.codes + (int64_t)pd.b * s.nblk * kBlockCoords + blk * (kBlockCoords * BITS / 8) + lane * BITS;
  int8_t* ea_p = s.exps + (int64_t)pd.a * s.nblk + blk;
  int8_t* eb_p = s.exps + (int64_t)pd.b * s.nblk + blk;

  f8 nx[kSub], av[kSub];       // loaded as X^a / B^a, overwritten with new model / average
  uint64_t pa[kSub], pb[kSub];
#pragma unroll
  for (int j = 0; j < kSub; ++j) nx[j] = ld256(xa + j * kSubCoords);
  if constexpr (FUSED) {
    if (fs.responders) fused_steps_responder(s, fs, pd, blk, lane);
    fused_steps_block(nx, s, fs, pd.a, pd.lsa, blk, lane);
  }
#pragma unroll
  for (int j = 0; j < kSub; ++j) av[j] = ld256(ba + j * kSubCoords);
#pragma unroll
  for (int j = 0; j < kSub; ++j) {
    pa[j] = load_codes<BITS>(ca + j * (kSubCoords * BITS / 8));
    pb[j] = load_codes<BITS>(cb + j * (kSubCoords * BITS / 8));
  }
  const int e_own = *ea_p, e_oth = *eb_p;

  // largest key magnitude of the block: decides, for the whole warp, which form of the lattice arithmetic
  // the decodes take
  float kmax = 0.0f;
#pragma unroll
  for (int j = 0; j < kSub; ++j)
#pragma unroll
    for (int i = 0; i < 8; ++i) kmax = fmaxf(kmax, fabsf(av[j].v[i]));
  kmax = warp_max_nonneg(kmax);
  float spread, dmax, M_blk;
  const int dec_mode = lattice_mode_both(lattice_mode(kmax, pow2f_exact(-e_own), e_own), lattice_mode(kmax, pow2f_exact(-e_oth), e_oth));
  SWARM_LATTICE_DISPATCH(dec_mode, nonblocking_decode<BITS, M>(nx, av, pa, pb, e_own, e_oth, spread, dmax, M_blk))
  const float rho = __fadd_rn(__fmul_rn(2.0f, spread), dmax);
  const int e = exponent_rule<BITS>(rho, M_blk);

  const uint32_t group0 = (uint32_t)(blk * (kBlockCoords / 8) + lane);
  SWARM_LATTICE_DISPATCH(lattice_mode(M_blk, pow2f_exact(-e), e),
                         nonblocking_encode<BITS, M>(nx, av, xa, ba, ca, cb, group0, s, pd, lane, e))
  if (lane == 0) { *ea_p = (int8_t)e; *eb_p = (int8_t)e; }
}

// -----------------------------------------------------------------------------------------
// Publish: every buffer receives an encoding of its node's base snapshot; the exponent of a
// block is set by the spread of all snapshots in that block, so that any node can decode any
// buffer with its own snapshot as key.
// -----------------------------------------------------------------------------------------
template <int BITS>
__global__ void __launch_bounds__(kWarpsPerCta * 32)
publish_range_kernel(StoreView s, int8_t* __restrict__ out_exps) {
  const int lane = threadIdx.x & 31;
  const int64_t blk = (int64_t)blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5);
  if (blk >= s.nblk) return;
  const float* base = s.B + blk * kBlockCoords + lane * 8;
  f8 lo[kSub], hi[kSub];
  float M = 0.0f;
#pragma unroll
  for (int j = 0; j < kSub; ++j) { lo[j] = ld256(base + j * kSubCoords); hi[j] = lo[j]; }
  for (int i = 0; i < s.n; ++i) {
    const float* row = base + (int64_t)i * s.pitch;
#pragma unroll
    for (int j = 0; j < kSub; ++j) {
      const f8 v = ld256(row + j * kSubCoords);
#pragma unroll
      for (int t = 0; t < 8; ++t) {
        lo[j].v[t] = fminf(lo[j].v[t], v.v[t]);
        hi[j].v[t] = fmaxf(hi[j].v[t], v.v[t]);
        M = fmaxf(M, fabsf(v.v[t]));
      }
    }
  }
  float rho = 0.0f;
#pragma unroll
  for (int j = 0; j < kSub; ++j)
#pragma unroll
    for (int t = 0; t < 8; ++t) rho = fmaxf(rho, __fsub_rn(hi[j].v[t], lo[j].v[t]));
  rho = warp_max_nonneg(rho);
  M = warp_max_nonneg(M);
  const int e = exponent_rule<BITS>(rho, M);
  for (int i = lane; i < s.n; i += 32) out_exps[(int64_t)i * s.nblk + blk] = (int8_t)e;
}

template <int BITS>
__global__ void __launch_bounds__(kWarpsPerCta * 32)
publish_encode_kernel(StoreView s, const uint32_t* __restrict__ wctr, int64_t total_warps) {
  const int lane = threadIdx.x & 31;
  const int64_t warp = (int64_t)blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5);
  if (warp >= total_warps) return;
  const int64_t node = warp / s.nblk;
  const int64_t blk = warp - node * s.nblk;
  const float* row = s.B + node * s.pitch + blk * kBlockCoords + lane * 8;
  uint8_t* c = s.codes + node * s.nblk * kBlockCoords + blk * (kBlockCoords * BITS / 8) + lane * BITS;
  const int e = s.exps[node * s.nblk + blk];
  const float inv_step = pow2f_exact(-e);
  const uint32_t w = wctr[node];
  constexpr uint32_t mask = (1u << BITS) - 1u;
  const uint32_t group0 = (uint32_t)(blk * (kBlockCoords / 8) + lane);
  f8 v[kSub];
#pragma unroll
  for (int j = 0; j < kSub; ++j) v[j] = ld256(row + j * kSubCoords);
#pragma unroll
  for (int j = 0; j < kSub; ++j) {
    const uint4 r = philox4x32_10(group0 + j * (kSubCoords / 8), (uint32_t)node, w, kStreamRounding, s.rk);
    uint64_t pk = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      int32_t cell;
      pk |= (uint64_t)((uint32_t)encode_index(v[j].v[i], inv_step, sr_u16(r, i), cell) & mask) << (i * BITS);
    }
    store_codes<BITS>(c + j * (kSubCoords * BITS / 8), lane, pk);
  }
}

// -----------------------------------------------------------------------------------------
// Two-register protocol (Section 3, "The Communication Registers"; Algorithm 1 with its chain of
// three decodes). Node k's own register O_k holds a 16-bit encoding of its snapshot, written only by
// k with the step of an 8-bit code of the guard distance (its readers' keys are unknown to it); its
// current register P_k holds a b-bit encoding written by whoever last interacted with k and scaled by
// the exact distance to its decoding key Q(X^_k), which that writer knows.
//   Q(X^_a) = Dec16(B_a, O_a)            local
//   Q(X_a)  = Dec_b(Q(X^_a), P_a)        Algorithm 1, first decode
//   Q(X^_b) = Dec16(B_a, O_b)            second decode: the partner's own register, key = own snapshot
//   Q(X_b)  = Dec_b(Q(X^_b), P_b)        third decode
//   X_a <- Q(X_a)/2 + Q(X_b)/2 - (B_a - X_a);  B_a <- X_a;  O_a, P_a <- Enc(X_a);  P_b <- Enc(average)
// Traffic per coordinate: 8 + 4 + 2b/8 B read, 8 + 2 + 2b/8 B written.
// -----------------------------------------------------------------------------------------
// own registers hold 16-bit colours (two byte planes)
constexpr int kOwnResolutionBits = 8;

// Own registers are stored in two byte planes per 1024-coordinate block (1024 low bytes, then 1024 high
// bytes of the 16-bit colours), so that a reader which needs only the 8-bit prefix touches the first
// plane alone. A lane's 8 coordinates of a sub-block are 8 consecutive bytes in each plane.
constexpr int kOwnBlockBytes = 2 * kBlockCoords;
// Byte i of a lane's 8 plane bytes in the low byte of the result; whatever follows it stays above (decoders read
// the low bits they need).
__device__ __forceinline__ uint32_t plane_byte(const uint2& v, int i) {
  return ((i < 4) ? v.x : v.y) >> ((i & 3) * 8);
}
// 16-bit colour i from the low-byte and high-byte planes in the low half of the result (upper half: garbage).
__device__ __forceinline__ uint32_t plane_colour16(const uint2& lo, const uint2& hi, int i) {
  return __byte_perm((i < 4) ? lo.x : lo.y, (i < 4) ? hi.x : hi.y, (i & 3) | ((4 + (i & 3)) << 4));
}
// Split eight 16-bit colours (two per word) into their low-byte and high-byte planes.
__device__ __forceinline__ void split_planes(const uint32_t (&ow)[4], uint2& lo, uint2& hi) {
  lo.x = __byte_perm(ow[0], ow[1], 0x6420); hi.x = __byte_perm(ow[0], ow[1], 0x7531);
  lo.y = __byte_perm(ow[2], ow[3], 0x6420); hi.y = __byte_perm(ow[2], ow[3], 0x7531);
}

// Decode chain of a two-register block. On entry nx = X^a, av = snapshot B^a; on return nx = new model,
// av = average. Returns the warp-reduced block maxima for the exponents of the three writes. FAST_LAST: the form
// of the lattice arithmetic in the last decode (b's current register, keyed by Q(X^_b)).
template <int BITS, int MODE, int MODE_LAST>
__device__ __forceinline__ void registers_decode(f8 (&nx)[kSub], f8 (&av)[kSub], const uint2 (&va)[kSub],
                                                 const uint2 (&vb)[kSub], const uint2 (&vbh)[kSub],
                                                 const uint64_t (&pa)[kSub], const uint64_t (&pb)[kSub], int prefix,
                                                 int eoa, int eob, int epa, int epb, float& spread_out, float& dmax_out,
                                                 float& M_out, float& rho_b_out, float& M_b_out) {
  using Ops = LatticeOps<MODE>;
  using LastOps = LatticeOps<MODE_LAST>;
  static_assert(MODE != kDefining || MODE_LAST == kDefining, "the last decode follows the others into the defining form");
  const float so_a = pow2f_exact(eoa), io_a = pow2f_exact(-eoa), so_b = pow2f_exact(eob), io_b = pow2f_exact(-eob);
  const float sp_a = pow2f_exact(epa), ip_a = pow2f_exact(-epa), sp_b = pow2f_exact(epb), ip_b = pow2f_exact(-epb);
  const float uo_a = Ops::kFast ? -__fmul_rn(kCellBias, so_a) : 0.0f, uo_b = Ops::kFast ? -__fmul_rn(kCellBias, so_b) : 0.0f;
  const float up_a = Ops::kFast ? -__fmul_rn(kCellBias, sp_a) : 0.0f, up_b = LastOps::kFast ? -__fmul_rn(kCellBias, sp_b) : 0.0f;
  float spread = 0.0f, dmax = 0.0f, M = 0.0f, rho_b = 0.0f, M_b = 0.0f;
#pragma unroll
  for (int j = 0; j < kSub; ++j)
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float snap = av[j].v[i];
      // own key: less than one step away, the 8-bit prefix always suffices
      const float qhat_a = Ops::value(Ops::template decode<8>(plane_byte(va[j], i), Ops::cell(snap, io_a)), so_a, uo_a);
      const float Qa = Ops::value(Ops::template decode<BITS>((uint32_t)(pa[j] >> (i * BITS)), Ops::cell(qhat_a, ip_a)), sp_a, up_a);
      const float qhat_b = Ops::value(Ops::decode_bits(plane_colour16(vb[j], vbh[j], i), Ops::cell(snap, io_b), prefix), so_b, uo_b);
      const float Qb = LastOps::value(LastOps::template decode<BITS>((uint32_t)(pb[j] >> (i * BITS)), LastOps::cell(qhat_b, ip_b)), sp_b, up_b);
      const float avg = __fmul_rn(0.5f, __fadd_rn(Qa, Qb));
      const float D = __fsub_rn(snap, nx[j].v[i]);
      const float x_new = __fsub_rn(avg, D);
      spread = fmaxf(spread, fabsf(__fsub_rn(Qa, Qb)));
      dmax = fmaxf(dmax, fabsf(D));
      M = fmaxf(M, fmaxf(fabsf(x_new), fabsf(avg)));             // (three-input maxima: one instruction each)
      rho_b = fmaxf(rho_b, fabsf(__fsub_rn(avg, qhat_b)));        // distance of the average to b's decoding key
      M_b = fmaxf(M_b, fmaxf(fabsf(avg), fabsf(qhat_b)));
      nx[j].v[i] = x_new;
      av[j].v[i] = avg;
    }
  spread_out = warp_max_nonneg(spread);
  dmax_out = warp_max_nonneg(dmax);
  M_out = warp_max_nonneg(M);
  rho_b_out = warp_max_nonneg(rho_b);
  M_b_out = warp_max_nonneg(M_b);
}

// Writes a's own register (16-bit colours of the new model, two byte planes) and b's current register
// (b-bit colours of the average); returns the distance of the new model to the lattice point just written.
template <int BITS, int MODE>
__device__ __forceinline__ void registers_encode_own(const f8 (&nx)[kSub], const f8 (&av)[kSub], uint8_t* oa, uint8_t* cb,
                                                     uint32_t group0, const StoreView& s, const PairDesc& pd, int lane,
                                                     int eo, int ep_b, float& rho_a_out, float& M_a_out) {
  using Ops = LatticeOps<MODE>;
  const float so = pow2f_exact(eo), io = pow2f_exact(-eo), ipb_new = pow2f_exact(-ep_b);
  const float uo = Ops::kFast ? -__fmul_rn(kCellBias, so) : 0.0f;
  float rho_a = 0.0f, M_a = 0.0f;
#pragma unroll
  for (int j = 0; j < kSub; ++j) {
    const uint32_t g = group0 + j * (kSubCoords / 8);
    const uint4 ro = philox4x32_10(g, (uint32_t)pd.a, pd.woa, kStreamOwnRounding, s.rk);
    const uint4 rb = philox4x32_10(g, (uint32_t)pd.b, pd.wb, kStreamRounding, s.rk);
    uint32_t qo[8], qb[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      uint32_t cell;
      qo[i] = Ops::encode(nx[j].v[i], io, sr_word(ro, i), i & 1, cell);
      const float qhat_new = Ops::value(qo[i], so, uo);
      rho_a = fmaxf(rho_a, fabsf(__fsub_rn(nx[j].v[i], qhat_new)));
      M_a = fmaxf(M_a, fmaxf(fabsf(nx[j].v[i]), fabsf(qhat_new)));
      qb[i] = Ops::encode(av[j].v[i], ipb_new, sr_word(rb, i), i & 1, cell);
    }
    uint32_t ow[4];
#pragma unroll
    for (int t = 0; t < 4; ++t) ow[t] = __byte_perm(qo[2 * t], qo[2 * t + 1], 0x5410);   // two 16-bit colours per word
    uint2 lo, hi;
    split_planes(ow, lo, hi);
    *reinterpret_cast<uint2*>(oa + j * kSubCoords) = lo;
    *reinterpret_cast<uint2*>(oa + kBlockCoords + j * kSubCoords) = hi;
    store_codes<BITS>(cb + j * (kSubCoords * BITS / 8), lane, pack_colours<BITS>(qb));
  }
  rho_a_out = warp_max_nonneg(rho_a);
  M_a_out = warp_max_nonneg(M_a);
}

// Writes the new model to X^a and B^a and its b-bit colours to a's current register.
template <int BITS, int MODE>
__device__ __forceinline__ void registers_encode_current(const f8 (&nx)[kSub], float* xa, float* ba, uint8_t* ca,
                                                         uint32_t group0, const StoreView& s, const PairDesc& pd,
                                                         int lane, int ep_a) {
  using Ops = LatticeOps<MODE>;
  const float ipa_new = pow2f_exact(-ep_a);
#pragma unroll
  for (int j = 0; j < kSub; ++j) {
    const uint32_t g = group0 + j * (kSubCoords / 8);
    const uint4 ra = philox4x32_10(g, (uint32_t)pd.a, pd.wa, kStreamRounding, s.rk);
    uint32_t qa[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      uint32_t cell;
      qa[i] = Ops::encode(nx[j].v[i], ipa_new, sr_word(ra, i), i & 1, cell);
    }
    st256(xa + j * kSubCoords, nx[j]);
    st256(ba + j * kSubCoords, nx[j]);
    store_codes<BITS>(ca + j * (kSubCoords * BITS / 8), lane, pack_colours<BITS>(qa));
  }
}

// (Local steps are not fused into this kernel: at 168 registers it keeps three warps per scheduler, and the steps'
// instruction stream on top of its own ran slower than the two kernels one after the other.)
template <int BITS>
__global__ void __launch_bounds__(kWarpsPerCta * 32)
interact_registers_kernel(StoreView s, const PairList pairs, int64_t total_warps, const FusedSteps fs) {
  grid_dependency_signal();
  grid_dependency_wait();
  const int lane = threadIdx.x & 31;
  uint32_t pair, blk32;
  if (!warp_slot(total_warps, s, 0, pair, blk32)) return;
  const int64_t blk = blk32;
  const PairDesc pd = pairs.get(pair);

  {
    uint32_t pair2, blk2_32;
    if (warp_slot(total_warps, s, (uint32_t)kPrefetchDistanceRegisters, pair2, blk2_32)) {
      const int64_t blk2 = blk2_32;
      const PairDesc p2 = pairs.get(pair2);
      const int64_t k2 = blk2 * kBlockCoords;
      prefetch_l2(s.X + (int64_t)p2.a * s.pitch + k2 + lane * 32);                      // 32 lines of 128 B
      prefetch_l2(s.B + (int64_t)p2.a * s.pitch + k2 + lane * 32);
      if (lane < 8)                                                                      // a's low-byte plane (1 KiB)
        prefetch_l2(s.own + ((int64_t)p2.a * s.nblk + blk2) * kOwnBlockBytes + lane * 128);
      if (lane < (int)p2.prefix)                                                         // b's plane(s): 8 or 16 lines
        prefetch_l2(s.own + ((int64_t)p2.b * s.nblk + blk2) * kOwnBlockBytes + lane * 128);
      if (lane < BITS) {
        prefetch_l2(s.codes + (int64_t)p2.a * s.nblk * kBlockCoords + blk2 * (kBlockCoords * BITS / 8) + lane * 128);
        prefetch_l2(s.codes + (int64_t)p2.b * s.nblk * kBlockCoords + blk2 * (kBlockCoords * BITS / 8) + lane * 128);
      }
    }
  }
  const int64_t koff = blk * kBlockCoords + lane * 8;
  float* xa = s.X + (int64_t)pd.a * s.pitch + koff;
  float* ba = s.B + (int64_t)pd.a * s.pitch + koff;
  uint8_t* oa = s.own + ((int64_t)pd.a * s.nblk + blk) * kOwnBlockBytes + lane * 8;       // low plane; high at +1024
  const uint8_t* ob = s.own + ((int64_t)pd.b * s.nblk + blk) * kOwnBlockBytes + lane * 8;
  const int prefix = (int)pd.prefix;      // the reader's statement about its distance to b's snapshot
  uint8_t* ca = s.codes + (int64_t)pd.a * s.nblk * kBlockCoords + blk * (kBlockCoords * BITS / 8) + lane * BITS;
  uint8_t* cb = s.codes + (int64_t)pd.b * s.nblk * kBlockCoords + blk * (kBlockCoords * BITS / 8) + lane * BITS;

  f8 nx[kSub], av[kSub];       // loaded as X^a / B^a, overwritten with new model / average
  uint2 va[kSub], vb[kSub], vbh[kSub];   // low bytes of a's and b's own registers, high bytes of b's
  uint64_t pa[kSub], pb[kSub];
#pragma unroll
  for (int j = 0; j < kSub; ++j) nx[j] = ld256(xa + j * kSubCoords);
#pragma unroll
  for (int j = 0; j < kSub; ++j) av[j] = ld256(ba + j * kSubCoords);
#pragma unroll
  for (int j = 0; j < kSub; ++j) {
    va[j] = *reinterpret_cast<const uint2*>(oa + j * kSubCoords);
    vb[j] = *reinterpret_cast<const uint2*>(ob + j * kSubCoords);
    vbh[j] = prefix == 16 ? *reinterpret_cast<const uint2*>(ob + kBlockCoords + j * kSubCoords) : make_uint2(0u, 0u);
    pa[j] = load_codes<BITS>(ca + j * (kSubCoords * BITS / 8));
    pb[j] = load_codes<BITS>(cb + j * (kSubCoords * BITS / 8));
  }
  const int eoa = s.oexps[(int64_t)pd.a * s.nblk + blk], eob = s.oexps[(int64_t)pd.b * s.nblk + blk];
  const int epa = s.exps[(int64_t)pd.a * s.nblk + blk], epb = s.exps[(int64_t)pd.b * s.nblk + blk];

  // Which form of the lattice arithmetic the decode chain takes is decided for the whole warp from bounds on the
  // keys: the snapshot (largest magnitude kmax) for the two own registers; for a's current register Q(X^_a),
  // which the 8-bit own decode leaves within 130 own steps of the snapshot; for b's current register Q(X^_b), which
  // can lie anywhere in the reader's window (32768 own steps with the full register: usually too far for the bound
  // to pass, though the value itself never is). That last decode therefore takes its form on its own: with the
  // full register it normally runs in the defining form (two conversions) while the other three stay fast.
  float kmax = 0.0f;
#pragma unroll
  for (int j = 0; j < kSub; ++j)
#pragma unroll
    for (int i = 0; i < 8; ++i) kmax = fmaxf(kmax, fabsf(av[j].v[i]));
  kmax = warp_max_nonneg(kmax);
  const float qa_max = __fmaf_rn(130.0f, pow2f_exact(eoa), kmax);
  const float qb_max = __fmaf_rn(prefix == 16 ? 32770.0f : 130.0f, pow2f_exact(eob), kmax);
  // (This kernel is built with the fused fast form only: with the multiply form as a third set of variants it ran
  // 3 % slower on its main workload, for the sake of blocks with positive exponents, which take the defining form.)
  const int mode_keys = lattice_mode_both(
      lattice_mode_both(lattice_mode_fused_only(kmax, pow2f_exact(-eoa), eoa), lattice_mode_fused_only(kmax, pow2f_exact(-eob), eob)),
      lattice_mode_fused_only(qa_max, pow2f_exact(-epa), epa));
  const int mode_last = lattice_mode_fused_only(qb_max, pow2f_exact(-epb), epb);
  float spread, dmax, M, rho_b, M_b;
#define SWARM_CHAIN(MK, ML) registers_decode<BITS, MK, ML>(nx, av, va, vb, vbh, pa, pb, prefix, eoa, eob, epa, epb, spread, dmax, M, rho_b, M_b)
  if (mode_keys == kFastFma && mode_last == kFastFma) SWARM_CHAIN(kFastFma, kFastFma);
  else if (mode_keys == kFastFma) SWARM_CHAIN(kFastFma, kDefining);
  else SWARM_CHAIN(kDefining, kDefining);
#undef SWARM_CHAIN
  const int eo = exponent_rule<kOwnResolutionBits>(__fadd_rn(__fmul_rn(2.0f, spread), dmax), M);
  const int ep_b = exponent_rule<BITS>(rho_b, M_b);

  // own register of a (16 bits) and current register of b; distance of the new model to its own key
  const uint32_t group0 = (uint32_t)(blk * (kBlockCoords / 8) + lane);
  float rho_a, M_a;
  if (lattice_mode_both(lattice_mode_fused_only(M, pow2f_exact(-eo), eo), lattice_mode_fused_only(M_b, pow2f_exact(-ep_b), ep_b)) == kFastFma)
    registers_encode_own<BITS, kFastFma>(nx, av, oa, cb, group0, s, pd, lane, eo, ep_b, rho_a, M_a);
  else
    registers_encode_own<BITS, kDefining>(nx, av, oa, cb, group0, s, pd, lane, eo, ep_b, rho_a, M_a);
  const int ep_a = exponent_rule<BITS>(rho_a, M_a);
  if (lattice_mode_fused_only(M_a, pow2f_exact(-ep_a), ep_a) == kFastFma)
    registers_encode_current<BITS, kFastFma>(nx, xa, ba, ca, group0, s, pd, lane, ep_a);
  else
    registers_encode_current<BITS, kDefining>(nx, xa, ba, ca, group0, s, pd, lane, ep_a);
  if (lane == 0) {
    s.oexps[(int64_t)pd.a * s.nblk + blk] = (int8_t)eo;
    s.exps[(int64_t)pd.a * s.nblk + blk] = (int8_t)ep_a;
    s.exps[(int64_t)pd.b * s.nblk + blk] = (int8_t)ep_b;
  }
}

// Initial register contents: own register = 16-bit encoding of the snapshot with the block's common
// exponent (already in oexps), current register = b-bit encoding scaled by the distance to that point.
template <int BITS>
__global__ void __launch_bounds__(kWarpsPerCta * 32)
register_publish_encode_kernel(StoreView s, const uint32_t* __restrict__ wctr, int64_t total_warps) {
  const int lane = threadIdx.x & 31;
  const int64_t warp = (int64_t)blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5);
  if (warp >= total_warps) return;
  const int64_t node = warp / s.nblk;
  const int64_t blk = warp - node * s.nblk;
  const int64_t koff = blk * kBlockCoords + lane * 8;
  const float* row = s.B + node * s.pitch + koff;
  uint8_t* o = s.own + (node * s.nblk + blk) * kOwnBlockBytes + lane * 8;
  uint8_t* c = s.codes + node * s.nblk * kBlockCoords + blk * (kBlockCoords * BITS / 8) + lane * BITS;
  const int eo = s.oexps[node * s.nblk + blk];
  const float so = pow2f_exact(eo), io = pow2f_exact(-eo);
  const uint32_t w = wctr[node], wo = wctr[s.n + node];
  constexpr uint32_t mask = (1u << BITS) - 1u;
  const uint32_t group0 = (uint32_t)(blk * (kBlockCoords / 8) + lane);
  f8 v[kSub];
#pragma unroll
  for (int j = 0; j < kSub; ++j) v[j] = ld256(row + j * kSubCoords);
  float rho = 0.0f, M = 0.0f;
#pragma unroll
  for (int j = 0; j < kSub; ++j) {
    const uint4 ro = philox4x32_10(group0 + j * (kSubCoords / 8), (uint32_t)node, wo, kStreamOwnRounding, s.rk);
    uint32_t ow[4] = {0u, 0u, 0u, 0u};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      int32_t cell;
      const int32_t q = encode_index(v[j].v[i], io, sr_u16(ro, i), cell);
      ow[i >> 1] |= ((uint32_t)q & 0xFFFFu) << ((i & 1) * 16);
      const float qhat = __fmul_rn(__int2float_rn(q), so);
      rho = fmaxf(rho, fabsf(__fsub_rn(v[j].v[i], qhat)));
      M = fmaxf(M, fmaxf(fabsf(v[j].v[i]), fabsf(qhat)));
    }
    uint2 lo, hi;
    split_planes(ow, lo, hi);
    *reinterpret_cast<uint2*>(o + j * kSubCoords) = lo;
    *reinterpret_cast<uint2*>(o + kBlockCoords + j * kSubCoords) = hi;
  }
  rho = warp_max_nonneg(rho);
  M = warp_max_nonneg(M);
  const int ep = exponent_rule<BITS>(rho, M);
  const float ip = pow2f_exact(-ep);
#pragma unroll
  for (int j = 0; j < kSub; ++j) {
    const uint4 r = philox4x32_10(group0 + j * (kSubCoords / 8), (uint32_t)node, w, kStreamRounding, s.rk);
    uint64_t pk = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      int32_t cell;
      pk |= (uint64_t)((uint32_t)encode_index(v[j].v[i], ip, sr_u16(r, i), cell) & mask) << (i * BITS);
    }
    store_codes<BITS>(c + j * (kSubCoords * BITS / 8), lane, pk);
  }
  if (lane == 0) s.exps[node * s.nblk + blk] = (int8_t)ep;
}

// -----------------------------------------------------------------------------------------
// Launch wrappers
// -----------------------------------------------------------------------------------------
static inline unsigned ctas_for(int64_t warps) { return (unsigned)((warps + kWarpsPerCta - 1) / kWarpsPerCta); }
constexpr int64_t kMaxLaunchWarps = (int64_t)1 << 31;   // the kernels index warps, and the warp a prefetch looks at, in 32 bits

// Code widths with a compiled kernel: SWARM_FOR_WIDTH(bits, BODY) runs BODY with the constant W = bits.
#define SWARM_WIDTH_CASE(w, ...) case w: { constexpr int W = w; __VA_ARGS__; } break;
#define SWARM_FOR_WIDTH(bits, ...)                                                          \
  switch (bits) {                                                                           \
    SWARM_WIDTH_CASE(2, __VA_ARGS__) SWARM_WIDTH_CASE(3, __VA_ARGS__) SWARM_WIDTH_CASE(4, __VA_ARGS__) \
    SWARM_WIDTH_CASE(5, __VA_ARGS__) SWARM_WIDTH_CASE(6, __VA_ARGS__) SWARM_WIDTH_CASE(7, __VA_ARGS__) \
    SWARM_WIDTH_CASE(8, __VA_ARGS__)                                                        \
    default: return cudaErrorInvalidValue;                                                  \
  }

template <typename Kernel>
static cudaError_t launch_dependent(Kernel kernel, dim3 grid, dim3 block, cudaStream_t st, const StoreView& s,
                                    const PairList& pairs, int64_t warps, const FusedSteps& fs) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, s, pairs, warps, fs);
}

cudaError_t launch_interact_blocking(const StoreView& s, const PairList& pairs, int npairs, int bits,
                                     const FusedSteps& fs, cudaStream_t st, int* launches) {
  if (npairs == 0) return cudaSuccess;
  const int64_t warps = (int64_t)npairs * s.nblk;
  if (warps + kPrefetchDistance >= kMaxLaunchWarps) return cudaErrorInvalidValue;
  const dim3 grid(ctas_for(warps)), block(kWarpsPerCta * 32);
  cudaError_t e = cudaSuccess;
  if (bits == 32) {
    e = launch_dependent(interact_identity_kernel, grid, block, st, s, pairs, warps, fs);
  } else {
    SWARM_FOR_WIDTH(bits, e = (fs.H > 0 ? launch_dependent(interact_blocking_kernel<W, true>, grid, block, st, s, pairs, warps, fs)
                                         : launch_dependent(interact_blocking_kernel<W, false>, grid, block, st, s, pairs, warps, fs)))
  }
  ++*launches;
  return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_interact_nonblocking(const StoreView& s, const PairList& pairs, int npairs, int bits,
                                        const FusedSteps& fs, cudaStream_t st, int* launches) {
  if (npairs == 0) return cudaSuccess;
  const int64_t warps = (int64_t)npairs * s.nblk;
  if (warps + kPrefetchDistance >= kMaxLaunchWarps) return cudaErrorInvalidValue;
  const dim3 grid(ctas_for(warps)), block(kWarpsPerCta * 32);
  cudaError_t e = cudaSuccess;
  SWARM_FOR_WIDTH(bits, e = (fs.H > 0 ? launch_dependent(interact_nonblocking_kernel<W, true>, grid, block, st, s, pairs, warps, fs)
                                         : launch_dependent(interact_nonblocking_kernel<W, false>, grid, block, st, s, pairs, warps, fs)))
  ++*launches;
  return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_publish(const StoreView& s, const uint32_t* wctr_dev, int bits, cudaStream_t st, int* launches) {
  const dim3 block(kWarpsPerCta * 32);
  const dim3 grid_r(ctas_for(s.nblk));
  const int64_t warps = (int64_t)s.n * s.nblk;
  const dim3 grid_e(ctas_for(warps));
  SWARM_FOR_WIDTH(bits, publish_range_kernel<W><<<grid_r, block, 0, st>>>(s, s.exps);
                        publish_encode_kernel<W><<<grid_e, block, 0, st>>>(s, wctr_dev, warps))
  *launches += 2;
  return cudaGetLastError();
}

cudaError_t launch_interact_registers(const StoreView& s, const PairList& pairs, int npairs, int bits,
                                      const FusedSteps& fs, cudaStream_t st, int* launches) {
  if (npairs == 0) return cudaSuccess;
  const int64_t warps = (int64_t)npairs * s.nblk;
  if (warps + kPrefetchDistance >= kMaxLaunchWarps) return cudaErrorInvalidValue;
  const dim3 grid(ctas_for(warps)), block(kWarpsPerCta * 32);
  cudaError_t e = cudaSuccess;
  if (fs.H > 0) return cudaErrorInvalidValue;       // the caller runs the local steps as a kernel of their own
  SWARM_FOR_WIDTH(bits, e = launch_dependent(interact_registers_kernel<W>, grid, block, st, s, pairs, warps, fs))
  ++*launches;
  return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_register_publish(const StoreView& s, const uint32_t* wctr_dev, int bits, cudaStream_t st,
                                    int* launches) {
  const dim3 block(kWarpsPerCta * 32);
  const dim3 grid_r(ctas_for(s.nblk));
  const int64_t warps = (int64_t)s.n * s.nblk;
  const dim3 grid_e(ctas_for(warps));
  // the own registers of a block share the step of an 8-bit code of the spread of all snapshots
  publish_range_kernel<kOwnResolutionBits><<<grid_r, block, 0, st>>>(s, s.oexps);
  SWARM_FOR_WIDTH(bits, register_publish_encode_kernel<W><<<grid_e, block, 0, st>>>(s, wctr_dev, warps))
  *launches += 2;
  return cudaGetLastError();
}

}  // namespace swarm
