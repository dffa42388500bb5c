// Least-squares local steps on bf16 data, batched over the nodes that share a data matrix and a
// minibatch, on the 5th-generation tensor cores (tcgen05.mma, accumulators in tensor memory).
//
// Section 3, "The Communication Procedure": x <- x - lr * g~(x), g~ = (1/B) sum_s (<a_s, x> - b_s) a_s
// over the B sampled rows a_s. For a unit of up to 16 nodes with the same rows this is two skinny
// contractions per step:
//   residuals  R[s][j] = sum_k A[r_s][k] * X_j[k]          (64 x 16 output, K = d)
//   update     X_j[k] -= (lr/B) * sum_s resid[s][j] A[r_s][k]   (d x 16 output, K = 64)
// Both stream the sampled rows once per unit (instead of once per node) and are HBM-bound; the
// tensor cores keep the 2*64*16 flops per coordinate off the critical path.
//
// Precision: fp32 operands are split into bf16 hi + bf16 lo (x = hi + lo up to 2^-17 relative), both
// halves multiplied against the same data tile, accumulated in fp32.
//
// Three kernels per step:
//   lsq_tc_residual_kernel  CTA = (k-chunk, unit): split-K partial R into scratch
//   lsq_tc_finalize_kernel  CTA = unit: sums the chunk partials in chunk order, subtracts labels,
//                           writes resid as bf16 hi/lo
//   lsq_tc_update_kernel    CTA = (k-chunk, unit): D = A_S^T resid per 128-coordinate tile, x -= scale * D
// Operand tiles are staged with cp.async into the 128-byte-swizzled shared-memory layouts the MMA
// descriptors name. Every wait on an mbarrier is bounded (spin_limit polls). A wait's outcome is made
// warp-uniform by a vote and CTA-uniform at the tile loop's barrier, so all threads of a CTA leave the loop
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

// =================================================================================================
// Residual partials. Tile = 128 coordinates (2 swizzle atoms of 64). Shared memory per stage:
//   A    : 2 atoms x [64 rows x 128 B]   (K-major, 128B swizzle, 8-row groups 1024 B apart)  16 KiB
// plus two operand buffers Xhi/Xlo: 2 atoms x [16 rows x 128 B] each. The fp32 models are loaded one
// tile ahead into registers (8 coordinates per thread) and converted to bf16 hi/lo straight into the
// operand buffers. Three stages of A: 65 KiB per CTA, three CTAs per SM, so that one CTA's barrier and
// operand conversion hide behind the copies of the other two (measured against five stages and two CTAs per
// SM at the 256-node workload: 5 % off the whole step).
// =================================================================================================
constexpr int kResTile = 128;
constexpr int kResAtoms = kResTile / 64;
constexpr int kResStages = 3;
constexpr int kResABytes = kResAtoms * kTcBatch * 128;         // 16384
constexpr int kResXopBytes = kResAtoms * kUnitNodes * 128;     // 4096 (one of hi / lo)
constexpr int kResSmem = kResStages * kResABytes + 2 * 2 * kResXopBytes + 1024 /*align*/ + 64;

__global__ void __launch_bounds__(kTcThreads, 3)
lsq_tc_residual_kernel(StoreView s, LsqView l, const LsqUnit* __restrict__ units, int step, float* __restrict__ partial,
                       int64_t chunk_coords, int64_t nchunks, int* __restrict__ status, uint32_t spin_limit) {
  __shared__ int poisoned;
  if (status_raised(status, &poisoned)) return;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* sA = smem;                                           // stages of A
  uint8_t* sXop = sA + kResStages * kResABytes;                 // [buf][hi|lo]
  uint64_t* bars = (uint64_t*)(sXop + 4 * kResXopBytes);        // mma_done[2]
  uint32_t* tmem_slot = (uint32_t*)(bars + 2);
  __shared__ int rows[kTcBatch];
  __shared__ int unodes[kUnitNodes];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const LsqUnit* up = units + blockIdx.y;
  struct { int group, count; } u = {up->group, up->count};
  const uint32_t event = up->event + (uint32_t)step;
  if (tid < kUnitNodes) unodes[tid] = up->nodes[tid];
  const int64_t kbase = (int64_t)blockIdx.x * chunk_coords;
  const int64_t kend = min(kbase + chunk_coords, s.pitch);
  const int ntiles = (int)((kend - kbase) / kResTile);
  const __nv_bfloat16* A = reinterpret_cast<const __nv_bfloat16*>(l.A) + (int64_t)u.group * l.m * s.pitch;

  if (tid < kTcBatch) rows[tid] = tid < l.batch ? tc_minibatch_row(tid, u.group, event, l.m, s.key0, s.key1) : 0;
  if (tid == 0) {
    mbar_init(smem_u32(&bars[0]), 1);
    mbar_init(smem_u32(&bars[1]), 1);
    fence_mbar_init();
  }
  if (warp == 0) { tmem_alloc(smem_u32(tmem_slot), 32); tmem_relinquish(); }
  // rows of the minibatch tile beyond the batch size are never copied: they must read as zero
  if (l.batch < kTcBatch)
    for (int i = tid; i < kResStages * kResABytes / 16; i += kTcThreads) reinterpret_cast<uint4*>(sA)[i] = make_uint4(0, 0, 0, 0);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_d = *tmem_slot;

  auto issue_loads = [&](int tile) {
    if (tile < ntiles) {
      const int st = tile % kResStages;
      const int64_t k0 = kbase + (int64_t)tile * kResTile;
      // A: 64 rows x 16 chunks of 16 B; thread -> (row = idx / 16, chunk = idx % 16)
      const uint32_t a_base = smem_u32(sA + st * kResABytes);
#pragma unroll
      for (int it = 0; it < kTcBatch * 16 / kTcThreads; ++it) {
        const int idx = it * kTcThreads + tid;
        const int r = idx >> 4, c = idx & 15;               // c: 16-byte chunk within the 256-byte row slice
        if (r < l.batch) {
          const int atom = c >> 3, cc = c & 7;
          const uint32_t dst = a_base + atom * (kTcBatch * 128) + (r >> 3) * 1024 + (r & 7) * 128 + ((cc ^ (r & 7)) << 4);
          cp_async16(dst, A + (int64_t)rows[r] * s.pitch + k0 + c * 8);
        }
      }
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
  int committed = -1;              // last tile whose MMAs were committed (the same in every thread)
  for (int t = 0; t < kResStages - 1; ++t) issue_loads(t);
  constexpr uint32_t idesc = instr_desc_bf16(kTcBatch, kUnitNodes, 0, 0);
  float4 xcur[2], xnext[2];
  load_x(0, xcur);
  for (int t = 0; t < ntiles; ++t) {
    const int st = t % kResStages, buf = t & 1;
    load_x(t + 1, xnext);                                   // consumed one iteration later
    cp_async_wait<kResStages - 2>();                        // this thread's copies of tile t have landed
    if (t >= 2) ok = mbar_wait(smem_u32(&bars[buf]), ((t >> 1) - 1) & 1, spin_limit) && ok;   // operand buffer free again
    // fp32 -> bf16 hi/lo into the swizzled operand layout
    {
      const int r = xr, c8 = xc8;                           // c8: group of 8 coordinates = one 16-byte bf16 chunk
      __align__(16) __nv_bfloat16 hi[8], lo[8];
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        const float4 v = xcur[q];
        split_bf16(v.x, hi[q * 4 + 0], lo[q * 4 + 0]);
        split_bf16(v.y, hi[q * 4 + 1], lo[q * 4 + 1]);
        split_bf16(v.z, hi[q * 4 + 2], lo[q * 4 + 2]);
        split_bf16(v.w, hi[q * 4 + 3], lo[q * 4 + 3]);
      }
      const int atom = c8 >> 3, cc = c8 & 7;
      const int off = atom * (kUnitNodes * 128) + (r >> 3) * 1024 + (r & 7) * 128 + ((cc ^ (r & 7)) << 4);
      *reinterpret_cast<uint4*>(sXop + (buf * 2 + 0) * kResXopBytes + off) = *reinterpret_cast<const uint4*>(hi);
      *reinterpret_cast<uint4*>(sXop + (buf * 2 + 1) * kResXopBytes + off) = *reinterpret_cast<const uint4*>(lo);
    }
    fence_proxy_async();                                    // generic-proxy writes (cp.async, st.shared) -> MMA reads
    tc_fence_before();
    ok = __syncthreads_and(ok);                             // the loop's one barrier also makes the give-up decision CTA-uniform
    if (!ok) break;
    if (tid == 0) {
      tc_fence_after();
      const uint32_t a_base = smem_u32(sA + st * kResABytes);
      const uint32_t h_base = smem_u32(sXop + (buf * 2 + 0) * kResXopBytes);
      const uint32_t l_base = smem_u32(sXop + (buf * 2 + 1) * kResXopBytes);
#pragma unroll
      for (int atom = 0; atom < kResAtoms; ++atom)
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {                    // 16 coordinates (32 bytes) per MMA
          const uint64_t da = smem_desc_sw128(a_base + atom * (kTcBatch * 128) + ks * 32, 16, 1024);
          const uint64_t dh = smem_desc_sw128(h_base + atom * (kUnitNodes * 128) + ks * 32, 16, 1024);
          const uint64_t dl = smem_desc_sw128(l_base + atom * (kUnitNodes * 128) + ks * 32, 16, 1024);
          tc_mma(tmem_d, da, dh, idesc, (t | atom | ks) != 0);
          tc_mma(tmem_d, da, dl, idesc, 1);
        }
      tc_commit(smem_u32(&bars[buf]));
    }
    committed = t;
    // refill the stage that tile t-1 used (its MMAs were committed one iteration ago); a warp whose wait
    // expired leaves that stage alone and reports at the next barrier
    if (t >= 1) ok = mbar_wait(smem_u32(&bars[(t - 1) & 1]), ((t - 1) >> 1) & 1, spin_limit);
    if (ok) issue_loads(t + kResStages - 1); else cp_async_commit();
    xcur[0] = xnext[0]; xcur[1] = xnext[1];
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
  // accumulator rows 16q..16q+15 live in lanes 32q..32q+15: warps 0..3, lanes 0..15
  if (warp < 4) {
    float v[16];
    tmem_ld8(tmem_d + ((uint32_t)(warp * 32) << 16), v);
    tmem_ld8(tmem_d + ((uint32_t)(warp * 32) << 16) + 8, v + 8);
    if (lane < 16 && ok) {
      float* dst = partial + (((int64_t)blockIdx.y * nchunks + blockIdx.x) * kTcBatch + warp * 16 + lane) * kUnitNodes;
#pragma unroll
      for (int q = 0; q < 4; ++q)
        reinterpret_cast<float4*>(dst)[q] = ntiles > 0 ? make_float4(v[q * 4], v[q * 4 + 1], v[q * 4 + 2], v[q * 4 + 3])
                                                       : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_d, 32);
}

// =================================================================================================
// Finalize: resid[s][j] = sum over chunks (in chunk order) - label, stored K-major per node as bf16
// hi / lo: R[unit][hi|lo][j][s].
// =================================================================================================
__global__ void __launch_bounds__(kTcBatch * kUnitNodes)
lsq_tc_finalize_kernel(StoreView s, LsqView l, const LsqUnit* __restrict__ units, int step, const float* __restrict__ partial,
                       int64_t nchunks, __nv_bfloat16* __restrict__ resid, const int* __restrict__ status) {
  if (*reinterpret_cast<const volatile int*>(status) != 0) return;    // the partials of a step that gave up are not complete
  const LsqUnit u = units[blockIdx.x];
  const int sidx = threadIdx.x / kUnitNodes, j = threadIdx.x % kUnitNodes;
  const float* p = partial + (int64_t)blockIdx.x * nchunks * (kTcBatch * kUnitNodes) + threadIdx.x;
  float acc = 0.0f;
#pragma unroll 8
  for (int64_t c = 0; c < nchunks; ++c) acc += p[c * (kTcBatch * kUnitNodes)];   // chunk order: fixed summation order
  float r = 0.0f;
  if (sidx < l.batch && j < u.count) {
    const int row = tc_minibatch_row(sidx, u.group, u.event + (uint32_t)step, l.m, s.key0, s.key1);
    r = row_residual(acc, l.bvec[(int64_t)u.nodes[j] * l.m + row], l.logistic);
  }
  __nv_bfloat16 hi, lo;
  split_bf16(r, hi, lo);
  __nv_bfloat16* out = resid + (int64_t)blockIdx.x * (2 * kUnitNodes * kTcBatch);
  out[j * kTcBatch + sidx] = hi;
  out[kUnitNodes * kTcBatch + j * kTcBatch + sidx] = lo;
}

// =================================================================================================
// Update. Tile = 128 coordinates. A operand = A_S^T, MN-major: per stage
//   [half h of 64 coordinates][8 groups of 8 sampled rows][8 rows x 128 B], 128B swizzle
//   (leading byte offset = 8192 between halves, stride byte offset = 1024 between row groups).
// B operand = resid hi / lo, K-major [16 nodes x 64 rows] (one swizzle atom each).
// Accumulators: 128 lanes x 16 columns, two buffers. Four stages: 70 KiB per CTA, three CTAs per SM (72 registers).
// =================================================================================================
constexpr int kUpdTile = 128;
constexpr int kUpdStages = 4;
constexpr int kUpdABytes = kTcBatch * kUpdTile * 2;             // 16384
constexpr int kUpdRBytes = kUnitNodes * 128;                   // 2048 (one of hi / lo)
constexpr int kUpdSmem = kUpdStages * kUpdABytes + 2 * kUpdRBytes + 1024 + 64;

__global__ void __launch_bounds__(kTcThreads, 3)
lsq_tc_update_kernel(StoreView s, LsqView l, const LsqUnit* __restrict__ units, int step, float lr,
                     const __nv_bfloat16* __restrict__ resid, int64_t chunk_coords, int* __restrict__ status,
                     uint32_t spin_limit) {
  __shared__ int poisoned;
  if (status_raised(status, &poisoned)) return;               // no model is touched after a step gave up
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* sA = smem;
  uint8_t* sR = sA + kUpdStages * kUpdABytes;                   // hi then lo
  uint64_t* bars = (uint64_t*)(sR + 2 * kUpdRBytes);
  uint32_t* tmem_slot = (uint32_t*)(bars + 2);
  __shared__ int rows[kTcBatch];
  __shared__ int unodes[kUnitNodes];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const LsqUnit* up = units + blockIdx.y;
  struct { int group, count; } u = {up->group, up->count};
  const uint32_t event = up->event + (uint32_t)step;
  if (tid < kUnitNodes) unodes[tid] = up->nodes[tid];
  const int64_t kbase = (int64_t)blockIdx.x * chunk_coords;
  const int64_t kend = min(kbase + chunk_coords, s.pitch);
  const int ntiles = (int)((kend - kbase) / kUpdTile);
  const __nv_bfloat16* A = reinterpret_cast<const __nv_bfloat16*>(l.A) + (int64_t)u.group * l.m * s.pitch;
  const float scale = lr / (float)l.batch;

  if (tid < kTcBatch) rows[tid] = tid < l.batch ? tc_minibatch_row(tid, u.group, event, l.m, s.key0, s.key1) : 0;
  if (tid == 0) {
    mbar_init(smem_u32(&bars[0]), 1);
    mbar_init(smem_u32(&bars[1]), 1);
    fence_mbar_init();
  }
  if (warp == 0) { tmem_alloc(smem_u32(tmem_slot), 32); tmem_relinquish(); }
  if (l.batch < kTcBatch)     // sampled-row slots beyond the batch are never copied: they must read as zero
    for (int i = tid; i < kUpdStages * kUpdABytes / 16; i += kTcThreads) reinterpret_cast<uint4*>(sA)[i] = make_uint4(0, 0, 0, 0);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_d = *tmem_slot;

  // resid hi / lo: 2 x [16 rows x 8 chunks], K-major swizzled
  if (tid < 2 * kUnitNodes * 8) {
    const int which = tid / (kUnitNodes * 8), r = (tid / 8) % kUnitNodes, c = tid & 7;
    cp_async16(smem_u32(sR + which * kUpdRBytes + (r >> 3) * 1024 + (r & 7) * 128 + ((c ^ (r & 7)) << 4)),
               resid + (int64_t)blockIdx.y * (2 * kUnitNodes * kTcBatch) + which * (kUnitNodes * kTcBatch) + r * kTcBatch + c * 8);
  }
  auto issue_loads = [&](int tile) {
    if (tile < ntiles) {
      const int st = tile % kUpdStages;
      const int64_t k0 = kbase + (int64_t)tile * kUpdTile;
      const uint32_t a_base = smem_u32(sA + st * kUpdABytes);
      // 64 rows x 16 chunks of 16 B: thread -> (row = idx / 16, chunk = idx % 16)
#pragma unroll
      for (int it = 0; it < kTcBatch * 16 / kTcThreads; ++it) {
        const int idx = it * kTcThreads + tid;
        const int r = idx >> 4, c = idx & 15;
        if (r < l.batch) {
          const int half = c >> 3, cc = c & 7;
          const uint32_t dst = a_base + half * 8192 + (r >> 3) * 1024 + (r & 7) * 128 + ((cc ^ (r & 7)) << 4);
          cp_async16(dst, A + (int64_t)rows[r] * s.pitch + k0 + c * 8);
        }
      }
    }
    cp_async_commit();
  };

  // this thread's share of the epilogue: coordinate lane of quadrant (warp % 4), nodes 8*(warp/4)..+7
  const int quad = warp & 3, jbase = (warp >> 2) * 8;
  auto epilogue = [&](int tile, const float xin[8]) {
    float dacc[8];
    tmem_ld8(tmem_d + ((uint32_t)(quad * 32) << 16) + (uint32_t)((tile & 1) * kUnitNodes + jbase), dacc);
    const int64_t k = kbase + (int64_t)tile * kUpdTile + quad * 32 + lane;
    if (k < s.d) {
#pragma unroll
      for (int q = 0; q < 8; ++q)
        if (jbase + q < u.count) s.X[(int64_t)unodes[jbase + q] * s.pitch + k] = xin[q] - scale * dacc[q];
    }
  };
  auto load_x = [&](int tile, float xin[8]) {
    const int64_t k = kbase + (int64_t)tile * kUpdTile + quad * 32 + lane;
#pragma unroll
    for (int q = 0; q < 8; ++q)
      xin[q] = (tile < ntiles && jbase + q < u.count) ? s.X[(int64_t)unodes[jbase + q] * s.pitch + k] : 0.0f;
  };

  bool ok = true;                  // this warp's waits so far
  int committed = -1;              // last tile whose MMAs were committed (the same in every thread)
  for (int t = 0; t < kUpdStages - 1; ++t) issue_loads(t);
  constexpr uint32_t idesc = instr_desc_bf16(kUpdTile, kUnitNodes, 1, 0);
  float xprev[8], xcur[8];
  for (int t = 0; t < ntiles; ++t) {
    const int st = t % kUpdStages, buf = t & 1;
    load_x(t, xcur);                                        // consumed one iteration later
    cp_async_wait<kUpdStages - 2>();
    fence_proxy_async();
    tc_fence_before();
    ok = __syncthreads_and(ok);                             // tile t landed; epilogue of tile t-2 has drained buffer `buf`;
    if (!ok) break;                                         // and the give-up decision is CTA-uniform
    if (tid == 0) {
      tc_fence_after();
      const uint32_t a_base = smem_u32(sA + st * kUpdABytes);
      const uint32_t h_base = smem_u32(sR), l_base = smem_u32(sR + kUpdRBytes);
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) {                      // 16 sampled rows per MMA = two 8-row groups
        const uint64_t da = smem_desc_sw128(a_base + ks * 2048, 8192, 1024);
        const uint64_t dh = smem_desc_sw128(h_base + ks * 32, 16, 1024);
        const uint64_t dl = smem_desc_sw128(l_base + ks * 32, 16, 1024);
        tc_mma(tmem_d + buf * kUnitNodes, da, dh, idesc, ks != 0);
        tc_mma(tmem_d + buf * kUnitNodes, da, dl, idesc, 1);
      }
      tc_commit(smem_u32(&bars[buf]));
    }
    committed = t;
    if (t >= 1) {
      ok = mbar_wait(smem_u32(&bars[(t - 1) & 1]), ((t - 1) >> 1) & 1, spin_limit);
      tc_fence_after();
      if (ok) epilogue(t - 1, xprev);
      tc_fence_before();
    }
#pragma unroll
    for (int q = 0; q < 8; ++q) xprev[q] = xcur[q];
    if (ok) issue_loads(t + kUpdStages - 1);                // stage of tile t-1: its MMAs have completed
    else cp_async_commit();
  }
  cp_async_wait<0>();
  if (ok && committed >= 0) {
    ok = mbar_wait(smem_u32(&bars[committed & 1]), (committed >> 1) & 1, spin_limit);
    tc_fence_after();
    if (ok) epilogue(committed, xprev);
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
  if (warp == 0) tmem_dealloc(tmem_d, 32);
}

// =================================================================================================
// Launch wrapper
// =================================================================================================
int64_t lsq_tc_chunk_coords(int64_t pitch) {
  // chunks of 8192 coordinates (a multiple of both tile sizes); short rows get a single chunk
  return pitch < 8192 ? pitch : 8192;
}
int64_t lsq_tc_chunks(int64_t pitch) {
  const int64_t c = lsq_tc_chunk_coords(pitch);
  return (pitch + c - 1) / c;
}
size_t lsq_tc_partial_bytes(int64_t pitch, int units) { return (size_t)units * lsq_tc_chunks(pitch) * kTcBatch * kUnitNodes * 4; }
size_t lsq_tc_resid_bytes(int units) { return (size_t)units * 2 * kUnitNodes * kTcBatch * 2; }

uint32_t lsq_tc_default_wait_limit() { return kSpinLimit; }

cudaError_t launch_local_lsq_tc(const StoreView& s, const LsqView& l, const LsqUnit* units_dev, int nunits, int H,
                                float lr, float* partial_dev, void* resid_dev, int* status_dev, uint32_t wait_limit,
                                cudaStream_t st, int* launches) {
  if (nunits == 0 || H == 0) return cudaSuccess;
  if (l.batch > kTcBatch || l.dtype != 1) return cudaErrorInvalidValue;
  static bool attr_set[64] = {};
  static std::mutex attr_mutex;                   // contexts on different threads may reach this together
  std::lock_guard<std::mutex> lock(attr_mutex);
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !attr_set[dev]) {
    cudaError_t e = cudaFuncSetAttribute(lsq_tc_residual_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kResSmem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(lsq_tc_update_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kUpdSmem);
    if (e != cudaSuccess) return e;
    attr_set[dev] = true;
  }
  const int64_t chunk = lsq_tc_chunk_coords(s.pitch), nchunks = lsq_tc_chunks(s.pitch);
  const dim3 grid((unsigned)nchunks, nunits);
  for (int q = 0; q < H; ++q) {
    lsq_tc_residual_kernel<<<grid, kTcThreads, kResSmem, st>>>(s, l, units_dev, q, partial_dev, chunk, nchunks, status_dev,
                                                               wait_limit);
    lsq_tc_finalize_kernel<<<nunits, kTcBatch * kUnitNodes, 0, st>>>(s, l, units_dev, q, partial_dev, nchunks,
                                                                     reinterpret_cast<__nv_bfloat16*>(resid_dev), status_dev);
    lsq_tc_update_kernel<<<grid, kTcThreads, kUpdSmem, st>>>(s, l, units_dev, q, lr,
                                                             reinterpret_cast<const __nv_bfloat16*>(resid_dev), chunk, status_dev,
                                                             wait_limit);
    *launches += 3;
  }
  return cudaGetLastError();
}

}  // namespace swarm
