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

namespace swarm {

constexpr int kWarpsPerCta = 4;

// Programmatic dependent launch: a kernel launched with the stream-serialization attribute may become
// resident while its predecessor in the stream drains; it must not touch global memory before
// grid_dependency_wait() returns (predecessor complete and flushed). Signalling early lets the
// successor's CTAs occupy SM slots as soon as this grid has none left to schedule, which hides the
// launch latency between back-to-back interaction launches.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_signal() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
constexpr int kSub = 4;          // sub-blocks per block
constexpr int kSubCoords = 256;  // coordinates per sub-block

// -----------------------------------------------------------------------------------------
// Blocking interaction: both models are present. Per block: exact range of X^a - X^b gives
// the common exponent; both are encoded into their buffers; each side decodes the partner's
// codes against its own model and both adopt Q(X^a)/2 + Q(X^b)/2.
// Traffic per coordinate: 8 B read, 8 B written, 2*b/8 B of codes written.
// -----------------------------------------------------------------------------------------
template <int BITS>
__global__ void __launch_bounds__(kWarpsPerCta * 32)
interact_blocking_kernel(StoreView s, const PairList pairs, int64_t total_warps) {
  grid_dependency_signal();
  grid_dependency_wait();
  const int lane = threadIdx.x & 31;
  const int64_t warp = (int64_t)blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5);
  if (warp >= total_warps) return;
  const int64_t pair = warp / s.nblk;
  const int64_t blk = warp - pair * s.nblk;
  const PairDesc pd = pairs.get(pair);

  float* xa = s.X + (int64_t)pd.a * s.pitch + blk * kBlockCoords + lane * 8;
  float* xb = s.X + (int64_t)pd.b * s.pitch + blk * kBlockCoords + lane * 8;

  f8 va[kSub], vb[kSub];
#pragma unroll
  for (int j = 0; j < kSub; ++j) va[j] = ld256(xa + j * kSubCoords);
#pragma unroll
  for (int j = 0; j < kSub; ++j) vb[j] = ld256(xb + j * kSubCoords);

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
  const float step = pow2f_exact(e), inv_step = pow2f_exact(-e);

  constexpr uint32_t mask = (1u << BITS) - 1u;
  const uint32_t group0 = (uint32_t)(blk * (kBlockCoords / 8) + lane);   // generator call index of sub-block 0
  uint8_t* ca = s.codes + (int64_t)pd.a * s.nblk * kBlockCoords + blk * (kBlockCoords * BITS / 8) + lane * BITS;
  uint8_t* cb = s.codes + (int64_t)pd.b * s.nblk * kBlockCoords + blk * (kBlockCoords * BITS / 8) + lane * BITS;

#pragma unroll
  for (int j = 0; j < kSub; ++j) {
    const uint32_t g = group0 + j * (kSubCoords / 8);
    const uint4 ra = philox4x32_10(g, (uint32_t)pd.a, pd.wa, kStreamRounding, s.key0, s.key1);
    const uint4 rb = philox4x32_10(g, (uint32_t)pd.b, pd.wb, kStreamRounding, s.key0, s.key1);
    uint64_t pka = 0, pkb = 0;
    f8 out;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      int32_t cell_a, cell_b;
      const int32_t qa = encode_index(va[j].v[i], inv_step, sr_u16(ra, i), cell_a);
      const int32_t qb = encode_index(vb[j].v[i], inv_step, sr_u16(rb, i), cell_b);
      const uint32_t code_a = (uint32_t)qa & mask, code_b = (uint32_t)qb & mask;
      pka |= (uint64_t)code_a << (i * BITS);
      pkb |= (uint64_t)code_b << (i * BITS);
      // b decodes a's codes with X^b as key and vice versa; the key's cell is already known
      const float Qa = __fmul_rn(__int2float_rn(decode_index<BITS>(code_a, cell_b)), step);
      const float Qb = __fmul_rn(__int2float_rn(decode_index<BITS>(code_b, cell_a)), step);
      out.v[i] = __fmul_rn(0.5f, __fadd_rn(Qa, Qb));
    }
    st256(xa + j * kSubCoords, out);
    st256(xb + j * kSubCoords, out);
    store_codes<BITS>(ca + j * (kSubCoords * BITS / 8), pka);
    store_codes<BITS>(cb + j * (kSubCoords * BITS / 8), pkb);
  }
  if (lane == 0) {
    s.exps[(int64_t)pd.a * s.nblk + blk] = (int8_t)e;
    s.exps[(int64_t)pd.b * s.nblk + blk] = (int8_t)e;
  }
}

// Identity quantizer (Corollary 2): plain averaging, buffers untouched.
__global__ void __launch_bounds__(kWarpsPerCta * 32)
interact_identity_kernel(StoreView s, const PairList pairs, int64_t total_warps) {
  const int lane = threadIdx.x & 31;
  const int64_t warp = (int64_t)blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5);
  if (warp >= total_warps) return;
  const int64_t pair = warp / s.nblk;
  const int64_t blk = warp - pair * s.nblk;
  const PairDesc pd = pairs.get(pair);
  float* xa = s.X + (int64_t)pd.a * s.pitch + blk * kBlockCoords + lane * 8;
  float* xb = s.X + (int64_t)pd.b * s.pitch + blk * kBlockCoords + lane * 8;
  f8 va[kSub], vb[kSub];
#pragma unroll
  for (int j = 0; j < kSub; ++j) va[j] = ld256(xa + j * kSubCoords);
#pragma unroll
  for (int j = 0; j < kSub; ++j) vb[j] = ld256(xb + j * kSubCoords);
#pragma unroll
  for (int j = 0; j < kSub; ++j) {
    f8 out;
#pragma unroll
    for (int i = 0; i < 8; ++i) out.v[i] = __fmul_rn(0.5f, __fadd_rn(va[j].v[i], vb[j].v[i]));
    st256(xa + j * kSubCoords, out);
    st256(xb + j * kSubCoords, out);
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
template <int BITS>
__global__ void __launch_bounds__(kWarpsPerCta * 32)
interact_nonblocking_kernel(StoreView s, const PairList pairs, int64_t total_warps) {
  grid_dependency_signal();
  grid_dependency_wait();
  const int lane = threadIdx.x & 31;
  const int64_t warp = (int64_t)blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5);
  if (warp >= total_warps) return;
  const int64_t pair = warp / s.nblk;
  const int64_t blk = warp - pair * s.nblk;
  const PairDesc pd = pairs.get(pair);

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
#pragma unroll
  for (int j = 0; j < kSub; ++j) av[j] = ld256(ba + j * kSubCoords);
#pragma unroll
  for (int j = 0; j < kSub; ++j) {
    pa[j] = load_codes<BITS>(ca + j * (kSubCoords * BITS / 8));
    pb[j] = load_codes<BITS>(cb + j * (kSubCoords * BITS / 8));
  }
  const int e_own = *ea_p, e_oth = *eb_p;
  const float step_own = pow2f_exact(e_own), inv_own = pow2f_exact(-e_own);
  const float step_oth = pow2f_exact(e_oth), inv_oth = pow2f_exact(-e_oth);

  constexpr uint32_t mask = (1u << BITS) - 1u;
  float spread = 0.0f, dmax = 0.0f, M = 0.0f;
#pragma unroll
  for (int j = 0; j < kSub; ++j)
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float key = av[j].v[i];
      const float own = decode_value<BITS>(key, (uint32_t)(pa[j] >> (i * BITS)) & mask, inv_own, step_own);
      const float oth = decode_value<BITS>(key, (uint32_t)(pb[j] >> (i * BITS)) & mask, inv_oth, step_oth);
      const float avg = __fmul_rn(0.5f, __fadd_rn(own, oth));
      const float D = __fsub_rn(key, nx[j].v[i]);
      const float x_new = __fsub_rn(avg, D);
      spread = fmaxf(spread, fabsf(__fsub_rn(own, oth)));
      dmax = fmaxf(dmax, fabsf(D));
      M = fmaxf(M, fmaxf(fabsf(x_new), fabsf(avg)));
      nx[j].v[i] = x_new;
      av[j].v[i] = avg;
    }
  spread = warp_max_nonneg(spread);
  dmax = warp_max_nonneg(dmax);
  M = warp_max_nonneg(M);
  const float rho = __fadd_rn(__fmul_rn(2.0f, spread), dmax);
  const int e = exponent_rule<BITS>(rho, M);
  const float inv_step = pow2f_exact(-e);

  const uint32_t group0 = (uint32_t)(blk * (kBlockCoords / 8) + lane);
#pragma unroll
  for (int j = 0; j < kSub; ++j) {
    const uint32_t g = group0 + j * (kSubCoords / 8);
    const uint4 ra = philox4x32_10(g, (uint32_t)pd.a, pd.wa, kStreamRounding, s.key0, s.key1);
    const uint4 rb = philox4x32_10(g, (uint32_t)pd.b, pd.wb, kStreamRounding, s.key0, s.key1);
    uint64_t pka = 0, pkb = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      int32_t cell;
      pka |= (uint64_t)((uint32_t)encode_index(nx[j].v[i], inv_step, sr_u16(ra, i), cell) & mask) << (i * BITS);
      pkb |= (uint64_t)((uint32_t)encode_index(av[j].v[i], inv_step, sr_u16(rb, i), cell) & mask) << (i * BITS);
    }
    st256(xa + j * kSubCoords, nx[j]);
    st256(ba + j * kSubCoords, nx[j]);
    store_codes<BITS>(ca + j * (kSubCoords * BITS / 8), pka);
    store_codes<BITS>(cb + j * (kSubCoords * BITS / 8), pkb);
  }
  if (lane == 0) { *ea_p = (int8_t)e; *eb_p = (int8_t)e; }
}

// -----------------------------------------------------------------------------------------
// Publish: every buffer receives an encoding of its node's base snapshot; the exponent of a
// block is set by the spread of all snapshots in that block, so that any node can decode any
// buffer with its own snapshot as key.
// -----------------------------------------------------------------------------------------
template <int BITS>
__global__ void __launch_bounds__(kWarpsPerCta * 32)
publish_range_kernel(StoreView s) {
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
  for (int i = lane; i < s.n; i += 32) s.exps[(int64_t)i * s.nblk + blk] = (int8_t)e;
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
    const uint4 r = philox4x32_10(group0 + j * (kSubCoords / 8), (uint32_t)node, w, kStreamRounding, s.key0, s.key1);
    uint64_t pk = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      int32_t cell;
      pk |= (uint64_t)((uint32_t)encode_index(v[j].v[i], inv_step, sr_u16(r, i), cell) & mask) << (i * BITS);
    }
    store_codes<BITS>(c + j * (kSubCoords * BITS / 8), pk);
  }
}

// -----------------------------------------------------------------------------------------
// Launch wrappers
// -----------------------------------------------------------------------------------------
static inline unsigned ctas_for(int64_t warps) { return (unsigned)((warps + kWarpsPerCta - 1) / kWarpsPerCta); }

template <typename Kernel>
static cudaError_t launch_dependent(Kernel kernel, dim3 grid, dim3 block, cudaStream_t st, const StoreView& s,
                                    const PairList& pairs, int64_t warps) {
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
  return cudaLaunchKernelEx(&cfg, kernel, s, pairs, warps);
}

cudaError_t launch_interact_blocking(const StoreView& s, const PairList& pairs, int npairs, int bits,
                                     cudaStream_t st, int* launches) {
  if (npairs == 0) return cudaSuccess;
  const int64_t warps = (int64_t)npairs * s.nblk;
  const dim3 grid(ctas_for(warps)), block(kWarpsPerCta * 32);
  cudaError_t e = cudaSuccess;
  switch (bits) {
    case 2: e = launch_dependent(interact_blocking_kernel<2>, grid, block, st, s, pairs, warps); break;
    case 4: e = launch_dependent(interact_blocking_kernel<4>, grid, block, st, s, pairs, warps); break;
    case 8: e = launch_dependent(interact_blocking_kernel<8>, grid, block, st, s, pairs, warps); break;
    case 32: interact_identity_kernel<<<grid, block, 0, st>>>(s, pairs, warps); break;
    default: return cudaErrorInvalidValue;
  }
  ++*launches;
  return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_interact_nonblocking(const StoreView& s, const PairList& pairs, int npairs, int bits,
                                        cudaStream_t st, int* launches) {
  if (npairs == 0) return cudaSuccess;
  const int64_t warps = (int64_t)npairs * s.nblk;
  const dim3 grid(ctas_for(warps)), block(kWarpsPerCta * 32);
  cudaError_t e = cudaSuccess;
  switch (bits) {
    case 2: e = launch_dependent(interact_nonblocking_kernel<2>, grid, block, st, s, pairs, warps); break;
    case 4: e = launch_dependent(interact_nonblocking_kernel<4>, grid, block, st, s, pairs, warps); break;
    case 8: e = launch_dependent(interact_nonblocking_kernel<8>, grid, block, st, s, pairs, warps); break;
    default: return cudaErrorInvalidValue;
  }
  ++*launches;
  return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_publish(const StoreView& s, const uint32_t* wctr_dev, int bits, cudaStream_t st, int* launches) {
  const dim3 block(kWarpsPerCta * 32);
  const dim3 grid_r(ctas_for(s.nblk));
  const int64_t warps = (int64_t)s.n * s.nblk;
  const dim3 grid_e(ctas_for(warps));
  switch (bits) {
    case 2:
      publish_range_kernel<2><<<grid_r, block, 0, st>>>(s);
      publish_encode_kernel<2><<<grid_e, block, 0, st>>>(s, wctr_dev, warps);
      break;
    case 4:
      publish_range_kernel<4><<<grid_r, block, 0, st>>>(s);
      publish_encode_kernel<4><<<grid_e, block, 0, st>>>(s, wctr_dev, warps);
      break;
    case 8:
      publish_range_kernel<8><<<grid_r, block, 0, st>>>(s);
      publish_encode_kernel<8><<<grid_e, block, 0, st>>>(s, wctr_dev, warps);
      break;
    default: return cudaErrorInvalidValue;
  }
  *launches += 2;
  return cudaGetLastError();
}

}  // namespace swarm
