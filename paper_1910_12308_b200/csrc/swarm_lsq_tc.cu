// Least-squares local steps on bf16 data, batched over the nodes that share a data matrix and a
// minibatch, on the 5th-generation tensor cores (tcgen05.mma, accumulators in tensor memory).
//
// Section 3, "The Communication Procedure": x <- x - lr * g~(x), g~ = (1/B) sum_s (<a_s, x> - b_s) a_s
// over the B sampled rows a_s. For a unit of up to 16 nodes with the same rows this is two skinny
// contractions per step:
//   scores     P[s][j] = sum_k A[r_s][k] * X_j[k]          (64 x 16 output, K = d)
//   update     X_j[k] -= (lr/B) * sum_s resid[s][j] A[r_s][k]   (d x 16 output, K = 64)
// Both stream the sampled rows once per unit (instead of once per node) and are HBM-bound; the
// tensor cores keep the 2*64*16 flops per coordinate off the critical path.
//
// Steps in groups. A node's G consecutive steps q = 0 .. G-1 (G <= 4) draw row sets S_q that are known in
// advance, and each step moves x along the sampled rows only: x_q = x_0 - (lr/B) sum_{p<q} A_{S_p}^T resid_p.
// The scores of step q are therefore
//   A_{S_q} x_q = A_{S_q} x_0 - (lr/B) sum_{p<q} (A_{S_q} A_{S_p}^T) resid_p,
// where A_{S_q} A_{S_p}^T is a 64 x 64 block of the data matrix's Gram matrix A A^T (m x m, a constant of
// the data, computed once when the data is made). One pass over the models then gives the scores of all G
// steps against x_0, a small kernel walks the recursion, and one pass applies all G updates:
// (G * rows + models) + (G * rows + 2 * models) bytes instead of G * (2 * rows + 3 * models).
// The result differs from G separately rounded steps only in rounding (the models are rounded once instead
// of G times). Without a Gram matrix (too large to keep) G = 1.
//
// Precision: fp32 operands are split into bf16 hi + bf16 lo (x = hi + lo up to 2^-17 relative), both
// halves multiplied against the same data tile, accumulated in fp32.
//
// Three kernels per group of steps:
//   lsq_tc_scores_kernel    CTA = (k-chunk, unit): split-K partial scores of the G steps into scratch
//   lsq_tc_finalize_kernel  CTA = unit: sums the chunk partials in chunk order, applies the Gram
//                           corrections step by step, subtracts labels, writes resid as bf16 hi/lo
//   lsq_tc_update_kernel    CTA = (k-chunk, unit): D = sum_q A_{S_q}^T resid_q per 128-coordinate tile,
//                           x -= scale * D
// Operand tiles are staged with cp.async into the 128-byte-swizzled shared-memory layouts the MMA
// descriptors name; a stage holds the rows of one step for one tile, and the stages of a tile follow one
// another. Every wait on an mbarrier is bounded (spin_limit polls). A wait's outcome is made
// warp-uniform by a vote and CTA-uniform at the stage loop's barrier, so all threads of a CTA leave the loop
// together; the CTA then raises the status word, drains its copies, waits (bounded by the full default limit,
// whatever spin_limit says) for the last MMA commit so that no MMA is in flight, frees its tensor memory and
// returns without writing results. Kernels that find the status word set on entry return at once, so a step
// that gave up is not built upon.
#include <mutex>

#include <cuda_bf16.h>

#include "swarm_dev.cuh"
#include "swarm_internal.h"

namespace swarm {

namespace {

constexpr int kTcThreads = 256;
constexpr int kUnitNodes = 16;            // N of the MMA
constexpr int kTcBatch = 64;              // rows of the minibatch tile (M of the residual MMA, K of the update MMA)
constexpr uint32_t kSpinLimit = 1u << 22;

// ---- small PTX wrappers ---------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" :: "n"(N) : "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait, called by whole warps: false for every lane when the limit expired in any lane.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint32_t limit) {
  bool done = false;
  for (uint32_t i = 0; i < limit && !done; ++i) done = mbar_try_wait(bar, parity);
  return __all_sync(0xFFFFFFFFu, done);
}
// True (for the whole CTA) when an earlier kernel on this context gave up; called by all threads.
__device__ __forceinline__ bool status_raised(const int* status, int* flag_smem) {
  if (threadIdx.x == 0) *flag_smem = *reinterpret_cast<const volatile int*>(status);
  __syncthreads();
  return *flag_smem != 0;
}
__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(slot_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(bar) : "memory");
}
// D[tmem] (+)= A[smem desc] * B[smem desc], bf16 inputs, fp32 accumulation.
__device__ __forceinline__ void tc_mma(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      :: "r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate) : "memory");
}
// 32 lanes x 8 consecutive 32-bit columns: thread t of the warp receives lane (base lane + t).
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float v[8]) {
  uint32_t r[8];
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory matrix descriptor, 128-byte swizzle, Blackwell version field = 1.
// Fields are in 16-byte units: start address [0,14), leading byte offset [16,30), stride byte offset
// [32,46), version [46,48), layout type [61,64) (2 = 128-byte swizzle).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
// Instruction descriptor for kind::f16: fp32 accumulator (bit 4), bf16 A (bit 7) and B (bit 10),
// A/B major (bits 15/16, 1 = MN-major), N/8 at [17,23), M/16 at [24,29).
__host__ __device__ constexpr uint32_t instr_desc_bf16(int M, int N, int a_mn_major, int b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) |
         ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

__device__ __forceinline__ int tc_minibatch_row(int s_idx, int group, uint32_t event, int m, uint32_t k0, uint32_t k1) {
  const uint4 w = philox4x32_10((uint32_t)(s_idx / 4), (uint32_t)group, event, kStreamMinibatch, k0, k1);
  const int t = s_idx & 3;
  const uint32_t word = t == 0 ? w.x : t == 1 ? w.y : t == 2 ? w.z : w.w;
  return (int)uniform_int(word, (uint32_t)m);
}

__device__ __forceinline__ void split_bf16(float x, __nv_bfloat16& hi, __nv_bfloat16& lo) {
  hi = __float2bfloat16_rn(x);
  lo = __float2bfloat16_rn(x - __bfloat162float(hi));
}

}  // namespace

constexpr int kTcMaxGroup = 4;            // steps folded into one pair of passes

// The rows of steps step0 .. step0 + G - 1 of a unit, as element offsets of the rows within their data matrix
// (row * pitch), so that a copy's source address is one addition away (slots beyond the batch size hold row 0
// and are never read as data: their tiles are zero and their residuals are zero).
template <int G>
__device__ __forceinline__ void draw_rows(int64_t* row_off, const LsqView& l, int group, uint32_t event0,
                                          const StoreView& s) {
  for (int i = threadIdx.x; i < G * kTcBatch; i += blockDim.x) {
    const int q = i / kTcBatch, sidx = i % kTcBatch;
    const int row = sidx < l.batch ? tc_minibatch_row(sidx, group, event0 + (uint32_t)q, l.m, s.key0, s.key1) : 0;
    row_off[i] = (int64_t)row * s.pitch;
  }
}

// =================================================================================================
// Score partials. Tile = 128 coordinates (2 swizzle atoms of 64). Shared memory per stage:
//   A    : 2 atoms x [64 rows x 128 B]   (K-major, 128B swizzle, 8-row groups 1024 B apart)  16 KiB
// plus two operand buffers of 2 atoms x [32 rows x 128 B]: rows 0..15 the bf16 hi halves of the 16 nodes' models,
// rows 16..31 the lo halves, so that one MMA (N = 32) multiplies a data tile against both; the two products are
// added in the epilogue. Stage f holds the rows of step f % G for tile f / G; the model tile is converted once
// per tile and multiplied against the G stages of the tile, step q accumulating into tensor-memory columns
// 32 q .. 32 q + 31. The MMAs of a stage are issued after the copies of a later stage, so that the issuing thread's
// warp does not fall behind with its copies. The fp32 models are loaded one
// tile ahead into registers (8 coordinates per thread) and converted to bf16 hi/lo straight into the
// operand buffers. Three stages of A: 65 KiB per CTA, three CTAs per SM, so that one CTA's barrier and
// operand conversion hide behind the copies of the other two. (Measured on the 256-node workload and dropped: a
// fourth stage with a single operand buffer, which each new tile must wait for, 3 % slower; L2 prefetches of the
// rows of a stage 2 to 8 stages further on, 6 % slower.)
// Order of completion: the wait at the end of iteration f covers the commit of stage f - 1, and commits complete
// in order; so when iteration f starts, every MMA up to stage f - 2 has completed, among them (G >= 1) all that
// read the operand buffer which a new tile is about to overwrite (the tile two before).
// =================================================================================================
constexpr int kResTile = 128;
constexpr int kResAtoms = kResTile / 64;
constexpr int kResStages = 3;
constexpr int kResABytes = kResAtoms * kTcBatch * 128;         // 16384
constexpr int kResXopBytes = kResAtoms * kUnitNodes * 128;     // 4096 (one of hi / lo)
constexpr int kResSmem = kResStages * kResABytes + 2 * 2 * kResXopBytes + 1024 /*align*/ + 64;

template <int G>
__global__ void __launch_bounds__(kTcThreads, 3)
lsq_tc_scores_kernel(StoreView s, LsqView l, const LsqUnit* __restrict__ units, int step, float* __restrict__ partial,
                     int64_t chunk_coords, int64_t nchunks, int* __restrict__ status, uint32_t spin_limit) {
  constexpr uint32_t kCols = G == 1 ? 32 : G == 2 ? 64 : 128;   // tensor-memory columns: 32 per step, a power of two
  __shared__ int poisoned;
  if (status_raised(status, &poisoned)) return;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* sA = smem;                                           // stages of A
  uint8_t* sXop = sA + kResStages * kResABytes;                 // [buf][hi|lo]
  uint64_t* bars = (uint64_t*)(sXop + 4 * kResXopBytes);        // mma_done[2]
  uint32_t* tmem_slot = (uint32_t*)(bars + 2);
  __shared__ int64_t row_off[G * kTcBatch];
  __shared__ int unodes[kUnitNodes];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const LsqUnit* up = units + blockIdx.y;
  struct { int group, count; } u = {up->group, up->count};
  if (tid < kUnitNodes) unodes[tid] = up->nodes[tid];
  const int64_t kbase = (int64_t)blockIdx.x * chunk_coords;
  const int64_t kend = min(kbase + chunk_coords, s.pitch);
  const int ntiles = (int)((kend - kbase) / kResTile);
  const int nstages = ntiles * G;
  const __nv_bfloat16* A = reinterpret_cast<const __nv_bfloat16*>(l.A) + (int64_t)u.group * l.m * s.pitch;

  draw_rows<G>(row_off, l, u.group, up->event + (uint32_t)step, s);
  if (tid == 0) {
    mbar_init(smem_u32(&bars[0]), 1);
    mbar_init(smem_u32(&bars[1]), 1);
    fence_mbar_init();
  }
  if (warp == 0) { tmem_alloc(smem_u32(tmem_slot), kCols); tmem_relinquish(); }
  // rows of the minibatch tile beyond the batch size are never copied: they must read as zero
  if (l.batch < kTcBatch)
    for (int i = tid; i < kResStages * kResABytes / 16; i += kTcThreads) reinterpret_cast<uint4*>(sA)[i] = make_uint4(0, 0, 0, 0);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_d = *tmem_slot;

  // A: 64 rows x 16 chunks of 16 B per stage; this thread copies chunk tid % 16 (16 B of the 256-byte row slice) of
  // rows tid / 16 + 16 it, it = 0..3: the same place within an 8-row group every time, 2048 B further per it
  const int crow = tid >> 4, cchunk = tid & 15;
  const uint32_t cdst = smem_u32(sA) + (cchunk >> 3) * (kTcBatch * 128) + (crow >> 3) * 1024 + (crow & 7) * 128 +
                        (((cchunk & 7) ^ (crow & 7)) << 4);
  int cmask = 0;                                                // which of its four rows exist (batch size)
#pragma unroll
  for (int it = 0; it < 4; ++it) cmask |= (crow + 16 * it < l.batch) << it;
  // the stage that the next call copies: destination, source tile, step within the tile, stage buffer, stages left
  uint32_t ld_dst = cdst;
  const __nv_bfloat16* ld_src = A + kbase + cchunk * 8;
  int ld_q = 0, ld_st = 0, ld_left = nstages;
  auto issue_loads = [&]() {
    if (ld_left > 0) {
      const int64_t* off = row_off + ld_q * kTcBatch + crow;
#pragma unroll
      for (int it = 0; it < kTcBatch * 16 / kTcThreads; ++it)
        if (cmask & (1 << it)) cp_async16(ld_dst + it * 2048, ld_src + off[16 * it]);
      --ld_left;
      if (++ld_q == G) { ld_q = 0; ld_src += kResTile; }
      if (++ld_st == kResStages) { ld_st = 0; ld_dst = cdst; } else ld_dst += kResABytes;
    }
    cp_async_commit();
  };

  // this thread's slice of the model tile: node row tid / 16, coordinates 8 * (tid % 16) .. +7
  const int xr = tid >> 4, xc8 = tid & 15;
  const float* xsrc = s.X + (int64_t)unodes[xr < u.count ? xr : 0] * s.pitch + kbase + xc8 * 8;
  auto load_x = [&](int tile, float4 v[2]) {
    if (tile < ntiles && xr < u.count) {
      v[0] = *reinterpret_cast<const float4*>(xsrc + (int64_t)tile * kResTile);
      v[1] = *reinterpret_cast<const float4*>(xsrc + (int64_t)tile * kResTile + 4);
    } else {
      v[0] = v[1] = make_float4(0.f, 0.f, 0.f, 0.f);          // node rows beyond the unit stay zero
    }
  };

  bool ok = true;                  // this warp's waits so far
  int committed = -1;              // last stage whose MMAs were committed (the same in every thread)
  for (int f = 0; f < kResStages - 1; ++f) issue_loads();
  constexpr uint32_t idesc = instr_desc_bf16(kTcBatch, 2 * kUnitNodes, 0, 0);   // N = 32: hi and lo side by side
  const uint64_t desc_a0 = smem_desc_sw128(smem_u32(sA), 16, 1024), desc_x0 = smem_desc_sw128(smem_u32(sXop), 16, 1024);
  float4 xcur[2], xnext[2];
  load_x(0, xcur);
  for (int f = 0, t = 0, q = 0, st = 0; f < nstages; ++f) {
    const int buf = t & 1;
    if (q == 0) load_x(t + 1, xnext);                       // consumed one tile later
    cp_async_wait<kResStages - 2>();                        // this thread's copies of stage f have landed
    if (q == 0 && ok) {
      // fp32 -> bf16 hi/lo into the swizzled operand layout
      const int r = xr, c8 = xc8;                           // c8: group of 8 coordinates = one 16-byte bf16 chunk
      __align__(16) __nv_bfloat16 hi[8], lo[8];
#pragma unroll
      for (int p = 0; p < 2; ++p) {
        const float4 v = xcur[p];
        split_bf16(v.x, hi[p * 4 + 0], lo[p * 4 + 0]);
        split_bf16(v.y, hi[p * 4 + 1], lo[p * 4 + 1]);
        split_bf16(v.z, hi[p * 4 + 2], lo[p * 4 + 2]);
        split_bf16(v.w, hi[p * 4 + 3], lo[p * 4 + 3]);
      }
      // operand rows 0..15 = hi of the 16 nodes, rows 16..31 = lo (two 8-row groups further on)
      const int atom = c8 >> 3, cc = c8 & 7;
      const int off = buf * (2 * kResXopBytes) + atom * (2 * kUnitNodes * 128) + (r >> 3) * 1024 + (r & 7) * 128 +
                      ((cc ^ (r & 7)) << 4);
      *reinterpret_cast<uint4*>(sXop + off) = *reinterpret_cast<const uint4*>(hi);
      *reinterpret_cast<uint4*>(sXop + off + 2048) = *reinterpret_cast<const uint4*>(lo);
      xcur[0] = xnext[0]; xcur[1] = xnext[1];
    }
    fence_proxy_async();                                    // generic-proxy writes (cp.async, st.shared) -> MMA reads
    tc_fence_before();
    ok = __syncthreads_and(ok);                             // the loop's one barrier also makes the give-up decision CTA-uniform
    if (!ok) break;
    // refill the stage that stage f-1 used (its MMAs were committed one iteration ago) before this stage's MMAs
    // are issued, so that the issue does not hold back warp 0's copies; a warp whose wait expired leaves that stage
    // alone and reports at the next barrier
    if (f >= 1) ok = mbar_wait(smem_u32(&bars[(f - 1) & 1]), ((f - 1) >> 1) & 1, spin_limit);
    if (ok) issue_loads(); else cp_async_commit();
    if (tid == 0) {
      tc_fence_after();
      // a descriptor's low bits hold the operand's shared-memory address / 16 (all of shared memory fits them), so
      // the descriptors of a stage, an atom and a 16-coordinate slice are additions to the first one
      const uint64_t da0 = desc_a0 + (uint64_t)((st * kResABytes) >> 4);
      const uint64_t dx0 = desc_x0 + (uint64_t)((buf * 2 * kResXopBytes) >> 4);
      const uint32_t d_addr = tmem_d + (uint32_t)(q * 2 * kUnitNodes);
#pragma unroll
      for (int atom = 0; atom < kResAtoms; ++atom)
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)                      // 16 coordinates (32 bytes) per MMA
          tc_mma(d_addr, da0 + (uint64_t)((atom * (kTcBatch * 128) + ks * 32) >> 4),
                 dx0 + (uint64_t)((atom * (2 * kUnitNodes * 128) + ks * 32) >> 4), idesc, (t | atom | ks) != 0);
      tc_commit(smem_u32(&bars[f & 1]));
    }
    committed = f;
    if (++q == G) { q = 0; ++t; }
    if (++st == kResStages) st = 0;
  }
  cp_async_wait<0>();
  if (ok && committed >= 0) ok = mbar_wait(smem_u32(&bars[committed & 1]), (committed >> 1) & 1, spin_limit);
  if (ok && committed >= 1) ok = mbar_wait(smem_u32(&bars[(committed - 1) & 1]), ((committed - 1) >> 1) & 1, spin_limit);
  ok = __syncthreads_and(ok);
  if (!ok) {
    if (tid == 0) atomicExch(status, 1);
    // gave up: the last commit covers every MMA issued before it; wait for it with the full default bound
    // so that tensor memory is not released under an MMA
    if (committed >= 0) mbar_wait(smem_u32(&bars[committed & 1]), (committed >> 1) & 1, kSpinLimit);
  }
  tc_fence_after();
  // accumulator rows 16w..16w+15 live in lanes 32w..32w+15: warps 0..3, lanes 0..15
  if (warp < 4) {
#pragma unroll
    for (int q = 0; q < G; ++q) {
      float v[16], w[16];                                   // products with the hi halves, with the lo halves
#pragma unroll
      for (int p = 0; p < 2; ++p) {
        tmem_ld8(tmem_d + ((uint32_t)(warp * 32) << 16) + (uint32_t)(q * 2 * kUnitNodes + p * 8), v + p * 8);
        tmem_ld8(tmem_d + ((uint32_t)(warp * 32) << 16) + (uint32_t)(q * 2 * kUnitNodes + kUnitNodes + p * 8), w + p * 8);
      }
#pragma unroll
      for (int p = 0; p < 16; ++p) v[p] += w[p];
      if (lane < 16 && ok) {
        float* dst = partial +
                     ((((int64_t)blockIdx.y * nchunks + blockIdx.x) * G + q) * kTcBatch + warp * 16 + lane) * kUnitNodes;
#pragma unroll
        for (int p = 0; p < 4; ++p)
          reinterpret_cast<float4*>(dst)[p] = ntiles > 0 ? make_float4(v[p * 4], v[p * 4 + 1], v[p * 4 + 2], v[p * 4 + 3])
                                                         : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_d, kCols);
}

// =================================================================================================
// Finalize, thread = (sampled row s, node j). kFinSplit CTAs per unit each add a contiguous run of the unit's
// chunk partials (in chunk order) and leave one second-level partial per step; the CTA of a unit that finishes
// last (a ticket counter per unit, left at zero) adds the second-level partials in run order, so the sum has one
// fixed association whichever CTA that is, and then walks the steps q = 0 .. G-1 in turn:
//   score[s][j] = the sum of step q - scale * sum_{p<q} sum_{s'} gram[row_q[s]][row_p[s']] * resid_p[s'][j]
//   resid_q[s][j] = score - label (least squares) or sigmoid(score) - label (logistic)
// stored K-major per node as bf16 hi / lo: R[unit][q][hi|lo][j][s]. The corrections use the residuals as the
// update kernel will see them (hi + lo).
// =================================================================================================
constexpr int kFinSplit = 8;

__global__ void __launch_bounds__(kTcBatch * kUnitNodes)
lsq_tc_finalize_kernel(StoreView s, LsqView l, const LsqUnit* __restrict__ units, int step, int G, float scale,
                       const float* __restrict__ partial, int64_t nchunks, float* __restrict__ level2,
                       unsigned int* __restrict__ tickets, __nv_bfloat16* __restrict__ resid,
                       const int* __restrict__ status) {
  if (*reinterpret_cast<const volatile int*>(status) != 0) return;    // the partials of a step that gave up are not complete
  __shared__ int rows[kTcMaxGroup * kTcBatch];
  __shared__ float seen[kTcMaxGroup - 1][kTcBatch][kUnitNodes];       // residuals of the earlier steps of the group
  __shared__ float block[kTcBatch][kTcBatch + 1];                     // one 64 x 64 block of the Gram matrix
  __shared__ bool last;
  const int unit = blockIdx.y, part = blockIdx.x;
  constexpr int kCell = kTcBatch * kUnitNodes;
  // the scores of every step against the model before the group; the steps' sums are independent of one another,
  // which keeps G times as many loads in flight
  float sum[kTcMaxGroup] = {0.0f, 0.0f, 0.0f, 0.0f};
  {
    const int64_t per = (nchunks + kFinSplit - 1) / kFinSplit;
    const int64_t c0 = part * per, c1 = min(c0 + per, nchunks);
    const float* p = partial + (int64_t)unit * nchunks * G * kCell + threadIdx.x;
#pragma unroll 4
    for (int64_t c = c0; c < c1; ++c) {
#pragma unroll
      for (int q = 0; q < kTcMaxGroup; ++q)
        if (q < G) sum[q] += p[(c * G + q) * kCell];
    }
    float* mine = level2 + ((int64_t)unit * kFinSplit + part) * kTcMaxGroup * kCell + threadIdx.x;
#pragma unroll
    for (int q = 0; q < kTcMaxGroup; ++q)
      if (q < G) mine[q * kCell] = sum[q];
  }
  __threadfence();                                                    // this thread's partials before the ticket
  __syncthreads();
  if (threadIdx.x == 0) {
    last = atomicAdd(&tickets[unit], 1u) == kFinSplit - 1;
    if (last) tickets[unit] = 0;                                      // every CTA of the unit has drawn: ready for the next launch
  }
  __syncthreads();
  if (!last) return;
  __threadfence();                                                    // the other CTAs' partials after the ticket
  {
    const volatile float* all = level2 + (int64_t)unit * kFinSplit * kTcMaxGroup * kCell + threadIdx.x;
#pragma unroll
    for (int q = 0; q < kTcMaxGroup; ++q) {
      sum[q] = 0.0f;
      if (q < G)
        for (int r = 0; r < kFinSplit; ++r) sum[q] += all[(r * kTcMaxGroup + q) * kCell];
    }
  }
  const LsqUnit u = units[unit];
  const int sidx = threadIdx.x / kUnitNodes, j = threadIdx.x % kUnitNodes;
  for (int i = threadIdx.x; i < G * kTcBatch; i += blockDim.x) {
    const int q = i / kTcBatch, r = i % kTcBatch;
    rows[i] = r < l.batch ? tc_minibatch_row(r, u.group, u.event + (uint32_t)(step + q), l.m, s.key0, s.key1) : 0;
  }
  __syncthreads();
  const float* gram = l.gram + (int64_t)u.group * l.m * l.m;
  const bool valid = sidx < l.batch && j < u.count;
#pragma unroll
  for (int q = 0; q < kTcMaxGroup; ++q) {
    if (q >= G) break;
    float acc = sum[q];
    float corr = 0.0f;
    for (int pq = 0; pq < q; ++pq) {
      __syncthreads();                                                // the block's previous readers are done
      for (int i = threadIdx.x; i < kTcBatch * kTcBatch; i += blockDim.x) {
        const int a = i / kTcBatch, b = i % kTcBatch;
        block[a][b] = gram[(int64_t)rows[q * kTcBatch + a] * l.m + rows[pq * kTcBatch + b]];
      }
      __syncthreads();
#pragma unroll 8
      for (int b = 0; b < kTcBatch; ++b) corr = fmaf(block[sidx][b], seen[pq][b][j], corr);
    }
    acc = fmaf(-scale, corr, acc);
    float r = 0.0f;
    if (valid) r = row_residual(acc, l.bvec[(int64_t)u.nodes[j] * l.m + rows[q * kTcBatch + sidx]], l.logistic);
    __nv_bfloat16 hi, lo;
    split_bf16(r, hi, lo);
    __nv_bfloat16* out = resid + ((int64_t)unit * G + q) * (2 * kUnitNodes * kTcBatch);
    out[j * kTcBatch + sidx] = hi;
    out[kUnitNodes * kTcBatch + j * kTcBatch + sidx] = lo;
    if (q + 1 < G) seen[q][sidx][j] = __bfloat162float(hi) + __bfloat162float(lo);
  }
}

// =================================================================================================
// Update. Tile = 128 coordinates. A operand = A_S^T, MN-major: per stage
//   [half h of 64 coordinates][8 groups of 8 sampled rows][8 rows x 128 B], 128B swizzle
//   (leading byte offset = 8192 between halves, stride byte offset = 1024 between row groups).
// B operand = resid of the stage's step, K-major [32 x 64 rows]: rows 0..15 the hi halves of the 16 nodes'
// residuals, rows 16..31 the lo halves (N = 32; the two products are added in the epilogue).
// Stage f holds the rows of step f % G for tile f / G; the G stages of a tile accumulate into one accumulator
// (128 lanes x 32 columns, two buffers), read back once the tile's last stage has completed.
// Four stages (three for groups of more than two steps, whose residuals take more room): at most 75 KiB per
// CTA, three CTAs per SM (72 registers).
// =================================================================================================
constexpr int kUpdTile = 128;
constexpr int kUpdABytes = kTcBatch * kUpdTile * 2;             // 16384
constexpr int kUpdRBytes = kUnitNodes * 128;                   // 2048 (one of hi / lo)
__host__ __device__ constexpr int upd_stages(int G) { return G <= 2 ? 4 : 3; }
__host__ __device__ constexpr int upd_smem(int G) { return upd_stages(G) * kUpdABytes + G * 2 * kUpdRBytes + 1024 + 64; }

template <int G>
__global__ void __launch_bounds__(kTcThreads, 3)
lsq_tc_update_kernel(StoreView s, LsqView l, const LsqUnit* __restrict__ units, int step, float lr,
                     const __nv_bfloat16* __restrict__ resid, int64_t chunk_coords, int* __restrict__ status,
                     uint32_t spin_limit) {
  constexpr int kStages = upd_stages(G);
  __shared__ int poisoned;
  if (status_raised(status, &poisoned)) return;               // no model is touched after a step gave up
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* sA = smem;
  uint8_t* sR = sA + kStages * kUpdABytes;                      // per step: hi then lo
  uint64_t* bars = (uint64_t*)(sR + G * 2 * kUpdRBytes);
  uint32_t* tmem_slot = (uint32_t*)(bars + 2);
  __shared__ int64_t row_off[G * kTcBatch];
  __shared__ int unodes[kUnitNodes];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const LsqUnit* up = units + blockIdx.y;
  struct { int group, count; } u = {up->group, up->count};
  if (tid < kUnitNodes) unodes[tid] = up->nodes[tid];
  const int64_t kbase = (int64_t)blockIdx.x * chunk_coords;
  const int64_t kend = min(kbase + chunk_coords, s.pitch);
  const int ntiles = (int)((kend - kbase) / kUpdTile);
  const int nstages = ntiles * G;
  const __nv_bfloat16* A = reinterpret_cast<const __nv_bfloat16*>(l.A) + (int64_t)u.group * l.m * s.pitch;
  const float scale = lr / (float)l.batch;

  draw_rows<G>(row_off, l, u.group, up->event + (uint32_t)step, s);
  if (tid == 0) {
    mbar_init(smem_u32(&bars[0]), 1);
    mbar_init(smem_u32(&bars[1]), 1);
    fence_mbar_init();
  }
  if (warp == 0) { tmem_alloc(smem_u32(tmem_slot), 64); tmem_relinquish(); }
  if (l.batch < kTcBatch)     // sampled-row slots beyond the batch are never copied: they must read as zero
    for (int i = tid; i < kStages * kUpdABytes / 16; i += kTcThreads) reinterpret_cast<uint4*>(sA)[i] = make_uint4(0, 0, 0, 0);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_d = *tmem_slot;

  // resid hi / lo of every step: 2 x [16 rows x 8 chunks], K-major swizzled (part of the first copy group)
  {
    const int which = tid / (kUnitNodes * 8), r = (tid / 8) % kUnitNodes, c = tid & 7;
#pragma unroll
    for (int q = 0; q < G; ++q)
      cp_async16(smem_u32(sR + (q * 2 + which) * kUpdRBytes + (r >> 3) * 1024 + (r & 7) * 128 + ((c ^ (r & 7)) << 4)),
                 resid + ((int64_t)blockIdx.y * G + q) * (2 * kUnitNodes * kTcBatch) + which * (kUnitNodes * kTcBatch) +
                     r * kTcBatch + c * 8);
  }
  // 64 rows x 16 chunks of 16 B per stage; this thread copies chunk tid % 16 of rows tid / 16 + 16 it, it = 0..3:
  // the same place within an 8-row group every time, 2048 B further per it
  const int crow = tid >> 4, cchunk = tid & 15;
  const uint32_t cdst = smem_u32(sA) + (cchunk >> 3) * 8192 + (crow >> 3) * 1024 + (crow & 7) * 128 +
                        (((cchunk & 7) ^ (crow & 7)) << 4);
  int cmask = 0;                                                // which of its four rows exist (batch size)
#pragma unroll
  for (int it = 0; it < 4; ++it) cmask |= (crow + 16 * it < l.batch) << it;
  // the stage that the next call copies: destination, source tile, step within the tile, stage buffer, stages left
  uint32_t ld_dst = cdst;
  const __nv_bfloat16* ld_src = A + kbase + cchunk * 8;
  int ld_q = 0, ld_st = 0, ld_left = nstages;
  auto issue_loads = [&]() {
    if (ld_left > 0) {
      const int64_t* off = row_off + ld_q * kTcBatch + crow;
#pragma unroll
      for (int it = 0; it < kTcBatch * 16 / kTcThreads; ++it)
        if (cmask & (1 << it)) cp_async16(ld_dst + it * 2048, ld_src + off[16 * it]);
      --ld_left;
      if (++ld_q == G) { ld_q = 0; ld_src += kUpdTile; }
      if (++ld_st == kStages) { ld_st = 0; ld_dst = cdst; } else ld_dst += kUpdABytes;
    }
    cp_async_commit();
  };

  // this thread's share of the epilogue: coordinate lane of quadrant (warp % 4), nodes 8*(warp/4)..+7
  const int quad = warp & 3, jbase = (warp >> 2) * 8;
  auto epilogue = [&](int tile, const float xin[8]) {
    float dacc[8], dlo[8];                                  // products with the hi halves of the residuals, with the lo halves
    tmem_ld8(tmem_d + ((uint32_t)(quad * 32) << 16) + (uint32_t)((tile & 1) * 2 * kUnitNodes + jbase), dacc);
    tmem_ld8(tmem_d + ((uint32_t)(quad * 32) << 16) + (uint32_t)((tile & 1) * 2 * kUnitNodes + kUnitNodes + jbase), dlo);
#pragma unroll
    for (int p = 0; p < 8; ++p) dacc[p] += dlo[p];
    const int64_t k = kbase + (int64_t)tile * kUpdTile + quad * 32 + lane;
    if (k < s.d) {
#pragma unroll
      for (int p = 0; p < 8; ++p)
        if (jbase + p < u.count) s.X[(int64_t)unodes[jbase + p] * s.pitch + k] = xin[p] - scale * dacc[p];
    }
  };
  auto load_x = [&](int tile, float xin[8]) {
    const int64_t k = kbase + (int64_t)tile * kUpdTile + quad * 32 + lane;
#pragma unroll
    for (int p = 0; p < 8; ++p)
      xin[p] = (tile < ntiles && jbase + p < u.count) ? s.X[(int64_t)unodes[jbase + p] * s.pitch + k] : 0.0f;
  };

  bool ok = true;                  // this warp's waits so far
  int committed = -1;              // last stage whose MMAs were committed (the same in every thread)
  for (int f = 0; f < kStages - 1; ++f) issue_loads();
  constexpr uint32_t idesc = instr_desc_bf16(kUpdTile, 2 * kUnitNodes, 1, 0);   // N = 32: hi and lo residuals side by side
  const uint64_t desc_a0 = smem_desc_sw128(smem_u32(sA), 8192, 1024), desc_r0 = smem_desc_sw128(smem_u32(sR), 16, 1024);
  float xprev[8], xcur[8];
  for (int f = 0, t = 0, q = 0, st = 0; f < nstages; ++f) {
    const int buf = t & 1;
    if (q == 0) load_x(t, xcur);                            // consumed when the tile's last stage has completed
    cp_async_wait<kStages - 2>();
    fence_proxy_async();
    tc_fence_before();
    ok = __syncthreads_and(ok);                             // stage f landed; epilogue of tile t-2 has drained buffer `buf`;
    if (!ok) break;                                         // and the give-up decision is CTA-uniform
    if (tid == 0) {
      tc_fence_after();
      // descriptors of a stage and of a 16-row slice: additions to the first one (address / 16 in the low bits)
      const uint64_t da0 = desc_a0 + (uint64_t)((st * kUpdABytes) >> 4);
      const uint64_t dr0 = desc_r0 + (uint64_t)((q * 2 * kUpdRBytes) >> 4);   // rows 0..15 hi, rows 16..31 lo
#pragma unroll
      for (int ks = 0; ks < 4; ++ks)                        // 16 sampled rows per MMA = two 8-row groups
        tc_mma(tmem_d + buf * 2 * kUnitNodes, da0 + (uint64_t)((ks * 2048) >> 4), dr0 + (uint64_t)((ks * 32) >> 4), idesc,
               (q | ks) != 0);
      tc_commit(smem_u32(&bars[f & 1]));
    }
    committed = f;
    if (f >= 1) {
      ok = mbar_wait(smem_u32(&bars[(f - 1) & 1]), ((f - 1) >> 1) & 1, spin_limit);
      tc_fence_after();
      if (ok && q == 0) epilogue(t - 1, xprev);             // stage f-1 was the last of tile t-1
      tc_fence_before();
    }
    if (q == 0) {
#pragma unroll
      for (int p = 0; p < 8; ++p) xprev[p] = xcur[p];
    }
    if (ok) issue_loads();                                  // into the stage of f-1: its MMAs have completed
    else cp_async_commit();
    if (++q == G) { q = 0; ++t; }
    if (++st == kStages) st = 0;
  }
  cp_async_wait<0>();
  if (ok && committed >= 0) {
    ok = mbar_wait(smem_u32(&bars[committed & 1]), (committed >> 1) & 1, spin_limit);
    tc_fence_after();
    if (ok) epilogue(committed / G, xprev);
  }
  ok = __syncthreads_and(ok);
  if (!ok) {
    if (tid == 0) atomicExch(status, 1);
    // gave up: wait for the last commit (it covers every MMA issued before it) with the full default bound,
    // so that tensor memory is not released under an MMA
    if (committed >= 0) mbar_wait(smem_u32(&bars[committed & 1]), (committed >> 1) & 1, kSpinLimit);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_d, 64);
}

// =================================================================================================
// Gram matrix of a bf16 data matrix on the tensor cores: gram = A A^T, a dense contraction with m x m outputs over
// the row length. CTA = one 128 x 128 tile of the lower triangle (mirrored on store) over the whole row length;
// stage = 64 coordinates of the tile's 128 + 128 rows (two K-major 128-byte-swizzled operand tiles of 16 KiB; a
// diagonal tile uses one for both operands); M = N = 128, K = 16 per MMA. The accumulator runs in tensor memory
// for 32 stages (2048 coordinates, 128 MMAs) at a time and is then added to per-thread double sums (thread = one
// row of the tile x 64 columns): the fp32 additions in tensor memory were measured to lose up to 3e-8 of the running
// sum each, all in one direction (1.9e-6 of a diagonal entry after 64 MMAs), so a run is kept to 128 of them
// (< 8e-6 of the entry; what reaches a residual is that times lr/B). Waits are bounded as in the step kernels. Runs once per data matrix (when the data is made or rewritten), not in the step.
// =================================================================================================
constexpr int kGtRows = 128;
constexpr int kGtStages = 4;
constexpr int kGtTileBytes = kGtRows * 128;                      // 16384
constexpr int kGtRun = 32;                                       // stages per accumulation run in tensor memory
constexpr int kGtSmem = kGtStages * 2 * kGtTileBytes + 1024 + 64;

__global__ void __launch_bounds__(kTcThreads, 1)
lsq_gram_tc_kernel(const __nv_bfloat16* __restrict__ A, int m, int64_t pitch, int first_matrix, float* __restrict__ gram,
                   int* __restrict__ status, uint32_t spin_limit) {
  __shared__ int poisoned;
  if (status_raised(status, &poisoned)) return;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* sA = smem;                                            // per stage: the tile of rows i, then of rows j
  uint64_t* bars = (uint64_t*)(sA + kGtStages * 2 * kGtTileBytes);
  uint32_t* tmem_slot = (uint32_t*)(bars + 2);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  int ti = 0;
  while ((ti + 1) * (ti + 2) / 2 <= (int)blockIdx.x) ++ti;       // tile (ti, tj) of the lower triangle, tj <= ti
  const int tj = (int)blockIdx.x - ti * (ti + 1) / 2;
  const bool diagonal = ti == tj;
  const int matrix = first_matrix + (int)blockIdx.y;
  const __nv_bfloat16* Ag = A + (int64_t)matrix * m * pitch;
  const int i0 = ti * kGtRows, j0 = tj * kGtRows;
  const int rows_i = min(kGtRows, m - i0), rows_j = min(kGtRows, m - j0);
  const int nstages = (int)(pitch / 64);

  if (tid == 0) {
    mbar_init(smem_u32(&bars[0]), 1);
    mbar_init(smem_u32(&bars[1]), 1);
    fence_mbar_init();
  }
  if (warp == 0) { tmem_alloc(smem_u32(tmem_slot), 128); tmem_relinquish(); }
  if (rows_i < kGtRows || rows_j < kGtRows)                      // rows past the matrix are never copied: they read as zero
    for (int i = tid; i < kGtStages * 2 * kGtTileBytes / 16; i += kTcThreads) reinterpret_cast<uint4*>(sA)[i] = make_uint4(0, 0, 0, 0);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_d = *tmem_slot;

  auto issue_loads = [&](int f) {
    if (f < nstages) {
      const uint32_t base_i = smem_u32(sA + (f % kGtStages) * 2 * kGtTileBytes), base_j = base_i + kGtTileBytes;
      const int64_t k0 = (int64_t)f * 64;
#pragma unroll
      for (int it = 0; it < kGtRows * 8 / kTcThreads; ++it) {    // 128 rows x 8 chunks of 16 B per operand tile
        const int idx = it * kTcThreads + tid;
        const int r = idx >> 3, c = idx & 7;
        const uint32_t off = (r >> 3) * 1024 + (r & 7) * 128 + ((c ^ (r & 7)) << 4);
        if (r < rows_i) cp_async16(base_i + off, Ag + (int64_t)(i0 + r) * pitch + k0 + c * 8);
        if (!diagonal && r < rows_j) cp_async16(base_j + off, Ag + (int64_t)(j0 + r) * pitch + k0 + c * 8);
      }
    }
    cp_async_commit();
  };

  // this thread's share of the tile: row quad * 32 + lane, columns half * 64 .. + 63
  const int quad = warp & 3, half = warp >> 2;
  double total[64];
#pragma unroll
  for (int e = 0; e < 64; ++e) total[e] = 0.0;
  bool ok = true;
  int committed = -1;
  for (int f = 0; f < kGtStages - 1; ++f) issue_loads(f);
  constexpr uint32_t idesc = instr_desc_bf16(kGtRows, kGtRows, 0, 0);
  for (int f = 0; f < nstages; ++f) {
    cp_async_wait<kGtStages - 2>();                             // this thread's copies of stage f have landed
    fence_proxy_async();
    tc_fence_before();
    ok = __syncthreads_and(ok);
    if (!ok) break;
    if (f >= 1) ok = mbar_wait(smem_u32(&bars[(f - 1) & 1]), ((f - 1) >> 1) & 1, spin_limit);
    if (ok) issue_loads(f + kGtStages - 1); else cp_async_commit();   // into the stage of f - 1, whose MMAs have completed
    if (tid == 0) {
      tc_fence_after();
      const uint32_t base_i = smem_u32(sA + (f % kGtStages) * 2 * kGtTileBytes);
      const uint32_t base_j = diagonal ? base_i : base_i + kGtTileBytes;
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) {                          // 16 coordinates (32 bytes) per MMA
        const uint64_t da = smem_desc_sw128(base_i + ks * 32, 16, 1024);
        const uint64_t db = smem_desc_sw128(base_j + ks * 32, 16, 1024);
        tc_mma(tmem_d, da, db, idesc, ((f % kGtRun) | ks) != 0);
      }
      tc_commit(smem_u32(&bars[f & 1]));
    }
    committed = f;
    if ((f + 1) % kGtRun == 0 || f == nstages - 1) {
      // end of a run: once this stage's MMAs have completed, the accumulator joins the double sums; the next run's
      // first MMA overwrites it after the next barrier, when every thread has read its part
      const bool done = mbar_wait(smem_u32(&bars[f & 1]), (f >> 1) & 1, spin_limit);
      ok = ok && done;
      tc_fence_after();
      if (ok) {
#pragma unroll
        for (int c8 = 0; c8 < 8; ++c8) {
          float v[8];
          tmem_ld8(tmem_d + ((uint32_t)(quad * 32) << 16) + (uint32_t)(half * 64 + c8 * 8), v);
#pragma unroll
          for (int e = 0; e < 8; ++e) total[c8 * 8 + e] += (double)v[e];
        }
      }
      tc_fence_before();
    }
  }
  cp_async_wait<0>();
  ok = __syncthreads_and(ok);
  if (!ok) {
    if (tid == 0) atomicExch(status, 1);
    // gave up: wait for the last commit with the full default bound, so that tensor memory is not released under an MMA
    if (committed >= 0) mbar_wait(smem_u32(&bars[committed & 1]), (committed >> 1) & 1, kSpinLimit);
  } else {
    float* G = gram + (int64_t)matrix * m * m;
    const int i = i0 + quad * 32 + lane;
    if (i < m) {
#pragma unroll
      for (int e = 0; e < 64; ++e) {
        const int j = j0 + half * 64 + e;
        if (j < m) {
          const float v = (float)total[e];
          G[(int64_t)i * m + j] = v;
          G[(int64_t)j * m + i] = v;
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_d, 128);
}

// =================================================================================================
// Gram matrix of an fp32 data matrix (short models only, see the short-model step kernel): CTA = one 64 x 64 tile
// of the lower triangle (mirrored on store), thread = 4 x 4 entries; products are summed in fp32 over 1024
// coordinates at a time and in double across those runs, in coordinate order.
// =================================================================================================
constexpr int kGramTile = 64;
constexpr int kGramK = 32;

__device__ __forceinline__ void load8_as_float(const __nv_bfloat16* p, float v[8]) {
  const uint4 raw = *reinterpret_cast<const uint4*>(p);
  const __nv_bfloat16* h = reinterpret_cast<const __nv_bfloat16*>(&raw);
#pragma unroll
  for (int e = 0; e < 8; ++e) v[e] = __bfloat162float(h[e]);
}
__device__ __forceinline__ void load8_as_float(const float* p, float v[8]) {
  const float4 lo = *reinterpret_cast<const float4*>(p), hi = *reinterpret_cast<const float4*>(p + 4);
  v[0] = lo.x; v[1] = lo.y; v[2] = lo.z; v[3] = lo.w; v[4] = hi.x; v[5] = hi.y; v[6] = hi.z; v[7] = hi.w;
}

template <typename T>
__global__ void __launch_bounds__(256)
lsq_gram_kernel(const T* __restrict__ A, int m, int64_t pitch, int first_matrix, float* __restrict__ gram) {
  __shared__ __align__(16) float sa[kGramK][kGramTile + 4];
  __shared__ __align__(16) float sb[kGramK][kGramTile + 4];
  int ti = 0;
  while ((ti + 1) * (ti + 2) / 2 <= (int)blockIdx.x) ++ti;       // tile (ti, tj) of the lower triangle, tj <= ti
  const int tj = (int)blockIdx.x - ti * (ti + 1) / 2;
  const int matrix = first_matrix + (int)blockIdx.y;
  const T* Ag = A + (int64_t)matrix * m * pitch;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int lrow = tid >> 2, c8 = (tid & 3) * 8;                 // staging: 64 rows x 4 groups of 8 coordinates
  const int ri = ti * kGramTile + lrow, rj = tj * kGramTile + lrow;
  double total[16];
  float run[16];
#pragma unroll
  for (int e = 0; e < 16; ++e) { total[e] = 0.0; run[e] = 0.0f; }
  for (int64_t k0 = 0; k0 < pitch; k0 += kGramK) {
    float va[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f}, vb[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    if (ri < m) load8_as_float(Ag + (int64_t)ri * pitch + k0 + c8, va);
    if (rj < m) load8_as_float(Ag + (int64_t)rj * pitch + k0 + c8, vb);
    __syncthreads();                                             // the previous slice's readers are done
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      sa[c8 + e][lrow] = va[e];
      sb[c8 + e][lrow] = vb[e];
    }
    __syncthreads();
#pragma unroll 8
    for (int k = 0; k < kGramK; ++k) {
      const float4 a = *reinterpret_cast<const float4*>(&sa[k][ty * 4]);
      const float4 b = *reinterpret_cast<const float4*>(&sb[k][tx * 4]);
      const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int y = 0; y < 4; ++y)
#pragma unroll
        for (int x = 0; x < 4; ++x) run[y * 4 + x] = fmaf(av[y], bv[x], run[y * 4 + x]);
    }
    if (((k0 + kGramK) & 1023) == 0) {
#pragma unroll
      for (int e = 0; e < 16; ++e) { total[e] += (double)run[e]; run[e] = 0.0f; }
    }
  }
  float* G = gram + (int64_t)matrix * m * m;
#pragma unroll
  for (int y = 0; y < 4; ++y)
#pragma unroll
    for (int x = 0; x < 4; ++x) {
      const int i = ti * kGramTile + ty * 4 + y, j = tj * kGramTile + tx * 4 + x;
      if (i < m && j < m) {
        const float v = (float)(total[y * 4 + x] + (double)run[y * 4 + x]);
        G[(int64_t)i * m + j] = v;
        G[(int64_t)j * m + i] = v;
      }
    }
}

// =================================================================================================
// Launch wrappers
// =================================================================================================
int64_t lsq_tc_chunk_coords(int64_t pitch) {
  // chunks of 8192 coordinates (a multiple of both tile sizes); short rows get a single chunk
  return pitch < 8192 ? pitch : 8192;
}
int64_t lsq_tc_chunks(int64_t pitch) {
  const int64_t c = lsq_tc_chunk_coords(pitch);
  return (pitch + c - 1) / c;
}
// Scratch of the tensor-core steps. Partials: the chunk partials of every unit, then kFinSplit second-level
// partials per unit. Residuals: bf16 hi / lo per unit and step, then one ticket counter per unit (zero between
// launches; the caller zeroes the buffer once).
static size_t chunk_partial_floats(int64_t pitch, int units) {
  return (size_t)units * lsq_tc_chunks(pitch) * kTcMaxGroup * kTcBatch * kUnitNodes;
}
static size_t resid_elems(int units) { return (size_t)units * kTcMaxGroup * 2 * kUnitNodes * kTcBatch; }
size_t lsq_tc_partial_bytes(int64_t pitch, int units) {
  return (chunk_partial_floats(pitch, units) + (size_t)units * kFinSplit * kTcMaxGroup * kTcBatch * kUnitNodes) * 4;
}
size_t lsq_tc_resid_bytes(int units) { return resid_elems(units) * 2 + (size_t)units * 4; }
size_t lsq_tc_gram_bytes(int matrices, int m) {
  const size_t bytes = (size_t)matrices * (size_t)m * (size_t)m * 4;
  return bytes <= ((size_t)256 << 20) ? bytes : 0;              // larger tables are not kept: steps go one at a time
}

uint32_t lsq_tc_default_wait_limit() { return kSpinLimit; }

namespace {

template <int G>
cudaError_t set_group_attributes() {
  cudaError_t e = cudaFuncSetAttribute(lsq_tc_scores_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, kResSmem);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(lsq_tc_update_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, upd_smem(G));
}

template <int G>
void launch_group(const StoreView& s, const LsqView& l, const LsqUnit* units_dev, int nunits, int step, float lr,
                  float* partial_dev, float* level2_dev, __nv_bfloat16* resid_dev, unsigned int* tickets_dev,
                  int* status_dev, uint32_t wait_limit, cudaStream_t st) {
  const int64_t chunk = lsq_tc_chunk_coords(s.pitch), nchunks = lsq_tc_chunks(s.pitch);
  const dim3 grid((unsigned)nchunks, nunits);
  lsq_tc_scores_kernel<G><<<grid, kTcThreads, kResSmem, st>>>(s, l, units_dev, step, partial_dev, chunk, nchunks, status_dev,
                                                              wait_limit);
  lsq_tc_finalize_kernel<<<dim3(kFinSplit, nunits), kTcBatch * kUnitNodes, 0, st>>>(
      s, l, units_dev, step, G, lr / (float)l.batch, partial_dev, nchunks, level2_dev, tickets_dev, resid_dev, status_dev);
  lsq_tc_update_kernel<G><<<grid, kTcThreads, upd_smem(G), st>>>(s, l, units_dev, step, lr, resid_dev, chunk, status_dev,
                                                                 wait_limit);
}

// Once per device: the dynamic shared-memory sizes of the tensor-core kernels.
cudaError_t ensure_attributes() {
  static bool attr_set[64] = {};
  static std::mutex attr_mutex;                   // contexts on different threads may reach this together
  std::lock_guard<std::mutex> lock(attr_mutex);
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !attr_set[dev]) {
    cudaError_t e = set_group_attributes<1>();
    if (e == cudaSuccess) e = set_group_attributes<2>();
    if (e == cudaSuccess) e = set_group_attributes<3>();
    if (e == cudaSuccess) e = set_group_attributes<4>();
    if (e == cudaSuccess) e = cudaFuncSetAttribute(lsq_gram_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kGtSmem);
    if (e != cudaSuccess) return e;
    attr_set[dev] = true;
  }
  return cudaSuccess;
}

}  // namespace

cudaError_t launch_lsq_gram(const void* A_dev, int dtype, int m, int64_t pitch, int first_matrix, int matrices,
                            float* gram_dev, int* status_dev, uint32_t wait_limit, cudaStream_t st, int* launches) {
  if (matrices == 0 || !gram_dev) return cudaSuccess;
  if (dtype == 1) {
    const cudaError_t e = ensure_attributes();
    if (e != cudaSuccess) return e;
    const int tiles = (m + kGtRows - 1) / kGtRows;
    const dim3 grid((unsigned)(tiles * (tiles + 1) / 2), (unsigned)matrices);
    lsq_gram_tc_kernel<<<grid, kTcThreads, kGtSmem, st>>>(reinterpret_cast<const __nv_bfloat16*>(A_dev), m, pitch, first_matrix,
                                                          gram_dev, status_dev, wait_limit);
  } else {
    const int tiles = (m + kGramTile - 1) / kGramTile;
    const dim3 grid((unsigned)(tiles * (tiles + 1) / 2), (unsigned)matrices);
    lsq_gram_kernel<<<grid, 256, 0, st>>>(reinterpret_cast<const float*>(A_dev), m, pitch, first_matrix, gram_dev);
  }
  ++*launches;
  return cudaGetLastError();
}

cudaError_t launch_local_lsq_tc(const StoreView& s, const LsqView& l, const LsqUnit* units_dev, int nunits, int max_units,
                                int H, float lr, float* partial_dev, void* resid_dev, int* status_dev,
                                uint32_t wait_limit, cudaStream_t st, int* launches) {
  if (nunits == 0 || H == 0) return cudaSuccess;
  if (l.batch > kTcBatch || l.dtype != 1) return cudaErrorInvalidValue;
  {
    const cudaError_t e = ensure_attributes();
    if (e != cudaSuccess) return e;
  }
  if (nunits > max_units) return cudaErrorInvalidValue;
  auto* resid = reinterpret_cast<__nv_bfloat16*>(resid_dev);
  auto* tickets = reinterpret_cast<unsigned int*>(resid + resid_elems(max_units));
  float* level2 = partial_dev + chunk_partial_floats(s.pitch, max_units);
  const int max_group = l.gram ? kTcMaxGroup : 1;
  for (int q = 0; q < H;) {
    const int G = H - q < max_group ? H - q : max_group;
    switch (G) {
      case 1: launch_group<1>(s, l, units_dev, nunits, q, lr, partial_dev, level2, resid, tickets, status_dev, wait_limit, st); break;
      case 2: launch_group<2>(s, l, units_dev, nunits, q, lr, partial_dev, level2, resid, tickets, status_dev, wait_limit, st); break;
      case 3: launch_group<3>(s, l, units_dev, nunits, q, lr, partial_dev, level2, resid, tickets, status_dev, wait_limit, st); break;
      default: launch_group<4>(s, l, units_dev, nunits, q, lr, partial_dev, level2, resid, tickets, status_dev, wait_limit, st); break;
    }
    *launches += 3;
    q += G;
  }
  return cudaGetLastError();
}

}  // namespace swarm
