// State generation, local SGD steps (Section 3, "The Communication Procedure": H sequential
// stochastic gradient steps, each at the running iterate) and the pair sampler (Algorithm 1,
// sampling lines).
#include <algorithm>
#include <cooperative_groups.h>
#include <cuda_bf16.h>

#include "swarm_dev.cuh"
#include "swarm_internal.h"
#include "swarm_blocks.cuh"

namespace cg = cooperative_groups;

namespace swarm {

// -----------------------------------------------------------------------------------------
// Per-node scalars: offset o_i, drift c_i (normals), label shift mu_i ~ U(-1, 1).
// scalars[i*3 + {0,1,2}].
// -----------------------------------------------------------------------------------------
__global__ void node_scalars_kernel(float* scalars, int n, float offset_std, float drift_std, uint32_t k0,
                                    uint32_t k1) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const uint4 w = philox4x32_10(0u, (uint32_t)i, 0u, kStreamNodeScalars, k0, k1);
  float z0, z1;
  normal_pair(w.x, w.y, z0, z1);
  scalars[i * 3 + 0] = __fmul_rn(offset_std, z0);
  scalars[i * 3 + 1] = __fmul_rn(drift_std, z1);
  scalars[i * 3 + 2] = __fsub_rn(__fmul_rn(2.0f, uniform_float(w.z)), 1.0f);
}

// X^i[k] = init_std * z(stream init, row i, k) + o_i ; one thread per 4 coordinates.
__global__ void init_models_kernel(StoreView s, const float* __restrict__ scalars, float init_std) {
  const int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int i = blockIdx.y;
  if (g * 4 >= s.d) return;
  float z[4];
  normal4((uint32_t)g, (uint32_t)i, 0u, kStreamInit, s.key0, s.key1, z);
  const float off = scalars[i * 3 + 0];
  float4 v;
  float* o = &v.x;
#pragma unroll
  for (int t = 0; t < 4; ++t) o[t] = (g * 4 + t < s.d) ? __fadd_rn(__fmul_rn(init_std, z[t]), off) : 0.0f;
  *reinterpret_cast<float4*>(s.X + (int64_t)i * s.pitch + g * 4) = v;
}

// -----------------------------------------------------------------------------------------
// Least-squares data: A_g[r][k] = z / sqrt(d) (rounded to bf16 when stored so), x*[k] = z,
// labels b_i[r] = <A_g(i)[r], x*> + mu_i + noise_std * z.
// -----------------------------------------------------------------------------------------
template <typename T>
__global__ void lsq_matrix_kernel(T* A, int64_t pitch, int64_t d, int m, float inv_sqrt_d, uint32_t k0, uint32_t k1) {
  const int64_t g4 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int r = blockIdx.y, grp = blockIdx.z;
  if (g4 * 4 >= pitch) return;
  float z[4];
  normal4((uint32_t)g4, (uint32_t)grp, (uint32_t)r, kStreamDataA, k0, k1, z);
  T* row = A + ((int64_t)grp * m + r) * pitch + g4 * 4;
#pragma unroll
  for (int t = 0; t < 4; ++t) {
    const float v = (g4 * 4 + t < d) ? __fmul_rn(z[t], inv_sqrt_d) : 0.0f;
    if constexpr (sizeof(T) == 2) row[t] = __float2bfloat16_rn(v); else row[t] = v;
  }
}

__global__ void xstar_kernel(float* xstar, int64_t pitch, int64_t d, uint32_t k0, uint32_t k1) {
  const int64_t g4 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (g4 * 4 >= pitch) return;
  float z[4];
  normal4((uint32_t)g4, 0u, 0u, kStreamXStar, k0, k1, z);
#pragma unroll
  for (int t = 0; t < 4; ++t) xstar[g4 * 4 + t] = (g4 * 4 + t < d) ? z[t] : 0.0f;
}

__device__ __forceinline__ float load_as_float(const float* p) { return *p; }
__device__ __forceinline__ float load_as_float(const __nv_bfloat16* p) { return __bfloat162float(*p); }

// One CTA per (row r, data matrix g): dot(A_g[r], x*) in double, then the labels of the
// nodes that own matrix g.
template <typename T>
__global__ void __launch_bounds__(256)
lsq_labels_kernel(const T* __restrict__ A, const float* __restrict__ xstar, float* bvec, const float* __restrict__ scalars,
                  int64_t pitch, int64_t d, int m, int nodes_per_group, float noise_std, uint32_t k0, uint32_t k1,
                  int logistic) {
  const int r = blockIdx.x, grp = blockIdx.y;
  const T* row = A + ((int64_t)grp * m + r) * pitch;
  double acc = 0.0;
  for (int64_t k = threadIdx.x; k < d; k += blockDim.x) acc += (double)load_as_float(row + k) * (double)xstar[k];
  __shared__ double part[8];
  acc = warp_sum(acc);
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x < nodes_per_group) {
    double dot = 0.0;
    for (int w = 0; w < 8; ++w) dot += part[w];
    const int node = grp * nodes_per_group + threadIdx.x;
    float z[4];
    normal4((uint32_t)(r / 4), (uint32_t)node, 0u, kStreamDataNoise, k0, k1, z);
    const float noise = __fmul_rn(noise_std, z[r % 4]);
    const float score = (float)(dot + (double)scalars[node * 3 + 2] + (double)noise);
    bvec[(int64_t)node * m + r] = logistic ? (score > 0.0f ? 1.0f : 0.0f) : score;   // class label = sign of the score
  }
}

// -----------------------------------------------------------------------------------------
// Synthetic-gradient local steps: x <- x - lr * (c_i + grad_std * z), H times in one memory
// pass; each step is its own sequence of rounded fp32 operations (no fusion across steps).
// -----------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
local_synth_kernel(StoreView s, const NodeList nodes, int H, float lr, float grad_std,
                   const float* __restrict__ scalars) {
  // one thread per 8 coordinates: one 256-bit load and store, two generator calls per step
  const int64_t g8 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (g8 * 8 >= s.d) return;
  const NodeDesc nd = nodes.get(blockIdx.y);
  const float c = scalars[nd.node * 3 + 1];
  float* p = s.X + (int64_t)nd.node * s.pitch + g8 * 8;
  f8 v = ld256(p);
  for (int q = 0; q < H; ++q)
    synth_step8(v, (uint32_t)g8, (uint32_t)nd.node, nd.event + (uint32_t)q, lr, grad_std, c, s.rk);
  if (g8 * 8 + 8 > s.d) {                                    // keep the row padding zero
#pragma unroll
    for (int t = 0; t < 8; ++t) if (g8 * 8 + t >= s.d) v.v[t] = 0.0f;
  }
  st256(p, v);
}

// -----------------------------------------------------------------------------------------
// Least-squares local step, general d: two kernels per step.
//   residual partials: CTA (chunk c, node t) computes for every minibatch row s the partial
//     dot product of A[r_s] and x over its chunk of kLsqChunk coordinates;
//   update: CTA (chunk c, node t) first sums the partials of each row in chunk order (a fixed
//     order, so results do not depend on scheduling), forms resid_s = <A[r_s], x> - b[r_s], then
//     x[k] -= (lr / B) * sum_s resid_s * A[r_s][k] on its chunk.
// -----------------------------------------------------------------------------------------
constexpr int kLsqThreads = 256;
constexpr int kLsqPerThread = 8;
constexpr int kLsqChunk = kLsqThreads * kLsqPerThread;   // 2048 coordinates per CTA
constexpr int kLsqMaxBatch = 256;

int64_t lsq_chunks(int64_t d) { return (d + kLsqChunk - 1) / kLsqChunk; }

__device__ __forceinline__ int minibatch_row(int s_idx, int group, uint32_t event, int m, uint32_t k0, uint32_t k1) {
  const uint4 w = philox4x32_10((uint32_t)(s_idx / 4), (uint32_t)group, event, kStreamMinibatch, k0, k1);
  const int t = s_idx & 3;
  const uint32_t word = t == 0 ? w.x : t == 1 ? w.y : t == 2 ? w.z : w.w;
  return (int)uniform_int(word, (uint32_t)m);
}

template <typename T>
__global__ void __launch_bounds__(kLsqThreads)
lsq_residual_kernel(StoreView s, LsqView l, const NodeList nodes, int step, float* __restrict__ partial,
                    int64_t nchunks) {
  const NodeDesc nd = nodes.get(blockIdx.y);
  const int group = nd.node / l.nodes_per_group;
  const uint32_t event = nd.event + (uint32_t)step;
  const int64_t k0 = (int64_t)blockIdx.x * kLsqChunk + threadIdx.x * kLsqPerThread;
  const float* xrow = s.X + (int64_t)nd.node * s.pitch;
  const T* A = reinterpret_cast<const T*>(l.A) + (int64_t)group * l.m * s.pitch;

  __shared__ int rows[kLsqMaxBatch];
  __shared__ float red[kLsqThreads / 32];
  if (threadIdx.x < l.batch) rows[threadIdx.x] = minibatch_row(threadIdx.x, group, event, l.m, s.key0, s.key1);
  float x[kLsqPerThread];
#pragma unroll
  for (int t = 0; t < kLsqPerThread; ++t) x[t] = (k0 + t < s.pitch) ? xrow[k0 + t] : 0.0f;
  __syncthreads();
  for (int si = 0; si < l.batch; ++si) {
    const T* row = A + (int64_t)rows[si] * s.pitch;
    float acc = 0.0f;
    if (k0 < s.pitch) {
#pragma unroll
      for (int t = 0; t < kLsqPerThread; ++t) acc = fmaf(load_as_float(row + k0 + t), x[t], acc);
    }
    acc = warp_sum(acc);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
      float tot = 0.0f;
#pragma unroll
      for (int w = 0; w < kLsqThreads / 32; ++w) tot += red[w];
      partial[((int64_t)blockIdx.y * l.batch + si) * nchunks + blockIdx.x] = tot;
    }
    __syncthreads();
  }
}

template <typename T>
__global__ void __launch_bounds__(kLsqThreads)
lsq_update_kernel(StoreView s, LsqView l, const NodeList nodes, int step, float lr,
                  const float* __restrict__ partial, int64_t nchunks) {
  const NodeDesc nd = nodes.get(blockIdx.y);
  const int group = nd.node / l.nodes_per_group;
  const uint32_t event = nd.event + (uint32_t)step;
  const int64_t k0 = (int64_t)blockIdx.x * kLsqChunk + threadIdx.x * kLsqPerThread;
  float* xrow = s.X + (int64_t)nd.node * s.pitch;
  const T* A = reinterpret_cast<const T*>(l.A) + (int64_t)group * l.m * s.pitch;

  __shared__ int rows[kLsqMaxBatch];
  __shared__ float resid[kLsqMaxBatch];
  // sum the chunk partials of each minibatch row in chunk order: one warp per row, lanes
  // stride the chunks, then a fixed-shape shuffle tree
  for (int si = threadIdx.x >> 5; si < l.batch; si += kLsqThreads / 32) {
    const float* p = partial + ((int64_t)blockIdx.y * l.batch + si) * nchunks;
    float acc = 0.0f;
    for (int64_t c = threadIdx.x & 31; c < nchunks; c += 32) acc += p[c];
    acc = warp_sum(acc);
    if ((threadIdx.x & 31) == 0) {
      const int r = minibatch_row(si, group, event, l.m, s.key0, s.key1);
      rows[si] = r;
      resid[si] = row_residual(acc, l.bvec[(int64_t)nd.node * l.m + r], l.logistic);
    }
  }
  __syncthreads();
  if (k0 >= s.d) return;
  float g[kLsqPerThread];
#pragma unroll
  for (int t = 0; t < kLsqPerThread; ++t) g[t] = 0.0f;
  for (int si = 0; si < l.batch; ++si) {
    const T* row = A + (int64_t)rows[si] * s.pitch + k0;
    const float rs = resid[si];
#pragma unroll
    for (int t = 0; t < kLsqPerThread; ++t) g[t] = fmaf(rs, load_as_float(row + t), g[t]);
  }
  const float scale = lr / (float)l.batch;
#pragma unroll
  for (int t = 0; t < kLsqPerThread; ++t)
    if (k0 + t < s.d) xrow[k0 + t] -= scale * g[t];
}

// -----------------------------------------------------------------------------------------
// Least-squares local steps for short models (row pitch <= 8192, batch <= 32): all H steps in one
// launch with the model in registers. A thread-block cluster of up to 8 CTAs owns one node; each CTA
// holds a 512- or 1024-coordinate slice, forms its share of the B dot products, and the CTAs exchange
// the partial sums through distributed shared memory (summed in rank order, so results do not depend
// on scheduling). The cluster barriers are hardware barriers reached by every CTA of the cluster.
// -----------------------------------------------------------------------------------------
constexpr int kSmallThreads = 128;
constexpr int kSmallMaxPitch = 8192;
constexpr int kSmallMaxBatch = 32;

template <typename T>
__device__ __forceinline__ float4 load4_as_float(const T* p);
template <>
__device__ __forceinline__ float4 load4_as_float<float>(const float* p) { return *reinterpret_cast<const float4*>(p); }
template <>
__device__ __forceinline__ float4 load4_as_float<__nv_bfloat16>(const __nv_bfloat16* p) {
  const uint2 raw = *reinterpret_cast<const uint2*>(p);
  return make_float4(__uint_as_float(raw.x << 16), __uint_as_float(raw.x & 0xFFFF0000u),
                     __uint_as_float(raw.y << 16), __uint_as_float(raw.y & 0xFFFF0000u));
}

// Shared-memory scratch of the short-model least-squares steps of one node.
constexpr int kRowsAhead = 8;            // local steps whose minibatches are drawn together
struct SmallShared {
  int rows[kRowsAhead][kSmallMaxBatch];
  float label[kRowsAhead][kSmallMaxBatch];
  float red[kSmallThreads / 32][kSmallMaxBatch];
  float part[kSmallMaxBatch];          // this CTA's partial dot products (read by the whole cluster)
  float resid[kSmallMaxBatch];
  // second step of a pair of steps taken in one round (batches of at most 16 rows)
  float red2[kSmallThreads / 32][16];
  float part2[16];
  float resid2[16];
  float gram[16][17];                  // <row s of the second step, row s' of the first>
};

// Barrier among the `count` threads that use barrier `id` (a multiple of 32 threads, whole warps).
__device__ __forceinline__ void named_barrier(int id, int count) {
  asm volatile("bar.sync %0, %1;" :: "r"(id), "r"(count) : "memory");
}

// Sums over the 32 lanes of G per-lane values at once: at each level a lane keeps one half of its values and
// hands the other half to its partner, so G rows cost G + 1 (G = 16) shuffles instead of 5 G. Lane and partner
// are paired as in the xor butterfly of warp_sum (offsets 16, 8, 4, 2, 1), so every sum has the same
// association, hence the same rounding. Lanes with an even index end up holding the sum of row `row`.
template <int G>
__device__ __forceinline__ float reduce_rows(float (&v)[G], int lane, int& row) {
  row = 0;
  int offset = 16;
#pragma unroll
  for (int width = G; width > 1; width >>= 1) {
    const int half = width >> 1;
    const bool upper = (lane & offset) != 0;
#pragma unroll
    for (int i = 0; i < half; ++i) {
      const float send = upper ? v[i] : v[i + half];
      const float keep = upper ? v[i + half] : v[i];
      v[i] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, offset);
    }
    if (upper) row += half;
    offset >>= 1;
  }
  for (; offset > 0; offset >>= 1) v[0] += __shfl_xor_sync(0xFFFFFFFFu, v[0], offset);
  return v[0];
}

// H least-squares steps of one node by kSmallThreads threads of every CTA of a cluster (ltid = 0..127 within
// the CTA; they share named barrier bar_id). Threads with active == false only take part in the cluster
// barriers, so that several thread groups of a CTA (each with its own node, scratch and named barrier) can
// run side by side. ITERS = slices of 512 coordinates per CTA. The model is read from and written back to
// global memory; the caller orders those accesses against other CTAs' work.
// Two steps per round where the data's Gram matrix is at hand and a minibatch fits the rows a thread keeps in
// flight: the second step's rows are known in advance, and <a, x_1> = <a, x_0> - (lr/B) sum_s' <a, a_s'> resid_0[s'],
// so both steps' dot products are formed against x_0 in one round of loads, warp sums and cluster exchange, the
// second step's are corrected with 16 x 16 entries of the Gram matrix (fetched alongside the rows), and the two
// updates are applied one after the other, each rounded as in a round of its own.
template <typename T, int ITERS>
__device__ __forceinline__ void lsq_small_steps(cg::cluster_group& cluster, const StoreView& s, const LsqView& l,
                                                bool active, int node, uint32_t event, int H, float lr, int csize,
                                                int ltid, int bar_id, SmallShared& sh) {
  constexpr int G = 16 / ITERS;                  // sampled rows whose loads are in flight together
  const int rank = (int)cluster.block_rank();
  const int warp = ltid >> 5, lane = ltid & 31;
  const int64_t base = (int64_t)rank * ITERS * (kSmallThreads * 4) + ltid * 4;   // first coordinate of this thread
  const int group = node / l.nodes_per_group;
  float* xrow = s.X + (int64_t)node * s.pitch + base;
  const T* A = reinterpret_cast<const T*>(l.A) + (int64_t)group * l.m * s.pitch + base;
  const float* labels = l.bvec + (int64_t)node * l.m;
  const bool one_group = l.batch <= G;           // then the rows loaded for the dot products serve the update too

  float4 x[2];
  x[0] = x[1] = make_float4(0.f, 0.f, 0.f, 0.f);
  if (active) {
    x[0] = *reinterpret_cast<const float4*>(xrow);
    if (ITERS > 1) x[1] = *reinterpret_cast<const float4*>(xrow + kSmallThreads * 4);
  }
  const float scale = lr / (float)l.batch;
  float4 a0[G], a1[G];

  const int* rows_q = sh.rows[0];
  auto load_group = [&](int s0) {
#pragma unroll
    for (int j = 0; j < G; ++j) {
      const bool on = s0 + j < l.batch;
      const T* row = A + (int64_t)rows_q[on ? s0 + j : 0] * s.pitch;
      a0[j] = on ? load4_as_float<T>(row) : make_float4(0.f, 0.f, 0.f, 0.f);
      a1[j] = (on && ITERS > 1) ? load4_as_float<T>(row + kSmallThreads * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  };

  const bool in_pairs = l.gram != nullptr && one_group;
  const float* gram = in_pairs ? l.gram + (int64_t)group * l.m * l.m : nullptr;
  float4 b0[G], b1[G];                           // the second step's rows in a round of two steps

  for (int q = 0; q < H;) {
    const int qq = q % kRowsAhead;
    if (active && qq == 0) {
      // minibatches (they depend on counters only) and their labels for the next kRowsAhead steps
      const int ahead = min(kRowsAhead, H - q) * l.batch;
      for (int idx = ltid; idx < ahead; idx += kSmallThreads) {
        const int dq = idx / l.batch, si = idx - dq * l.batch;
        const int r = minibatch_row(si, group, event + (uint32_t)(q + dq), l.m, s.key0, s.key1);
        sh.rows[dq][si] = r;
        sh.label[dq][si] = labels[r];
      }
      named_barrier(bar_id, kSmallThreads);
    }
    if (in_pairs && q + 1 < H) {
      // ---- steps q and q + 1 in one round (q is even here, so both lie in the window drawn above)
      const int* rows_p = sh.rows[qq + 1];
      if (active) {
        rows_q = sh.rows[qq];
        float gv[2];                             // this thread's entries of the 16 x 16 Gram block
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int idx = ltid + e * kSmallThreads, a = idx / l.batch, b = idx - a * l.batch;
          gv[e] = a < l.batch ? gram[(int64_t)rows_p[a] * l.m + rows_q[b]] : 0.0f;
        }
        load_group(0);
#pragma unroll
        for (int j = 0; j < G; ++j) {
          const bool on = j < l.batch;
          const T* row = A + (int64_t)rows_p[on ? j : 0] * s.pitch;
          b0[j] = on ? load4_as_float<T>(row) : make_float4(0.f, 0.f, 0.f, 0.f);
          b1[j] = (on && ITERS > 1) ? load4_as_float<T>(row + kSmallThreads * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        float acc[G], acc2[G];
#pragma unroll
        for (int j = 0; j < G; ++j) {
          acc[j] = a0[j].x * x[0].x;
          acc[j] = fmaf(a0[j].y, x[0].y, acc[j]); acc[j] = fmaf(a0[j].z, x[0].z, acc[j]); acc[j] = fmaf(a0[j].w, x[0].w, acc[j]);
          acc[j] = fmaf(a1[j].x, x[1].x, acc[j]); acc[j] = fmaf(a1[j].y, x[1].y, acc[j]);
          acc[j] = fmaf(a1[j].z, x[1].z, acc[j]); acc[j] = fmaf(a1[j].w, x[1].w, acc[j]);
          acc2[j] = b0[j].x * x[0].x;
          acc2[j] = fmaf(b0[j].y, x[0].y, acc2[j]); acc2[j] = fmaf(b0[j].z, x[0].z, acc2[j]); acc2[j] = fmaf(b0[j].w, x[0].w, acc2[j]);
          acc2[j] = fmaf(b1[j].x, x[1].x, acc2[j]); acc2[j] = fmaf(b1[j].y, x[1].y, acc2[j]);
          acc2[j] = fmaf(b1[j].z, x[1].z, acc2[j]); acc2[j] = fmaf(b1[j].w, x[1].w, acc2[j]);
        }
        int row, row2;
        const float tot = reduce_rows<G>(acc, lane, row);
        const float tot2 = reduce_rows<G>(acc2, lane, row2);
        if ((lane & 1) == 0 && row < l.batch) { sh.red[warp][row] = tot; sh.red2[warp][row2] = tot2; }
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int idx = ltid + e * kSmallThreads, a = idx / l.batch, b = idx - a * l.batch;
          if (a < l.batch) sh.gram[a][b] = gv[e];
        }
        named_barrier(bar_id, kSmallThreads);
        // warp 0 finishes the first step's sums, warp 1 the second step's
        if (ltid < l.batch) {
          float t = 0.0f;
#pragma unroll
          for (int w = 0; w < kSmallThreads / 32; ++w) t += sh.red[w][ltid];
          sh.part[ltid] = t;
        } else if (ltid >= 32 && ltid - 32 < l.batch) {
          float t = 0.0f;
#pragma unroll
          for (int w = 0; w < kSmallThreads / 32; ++w) t += sh.red2[w][ltid - 32];
          sh.part2[ltid - 32] = t;
        }
      }
      cluster.sync();                            // every CTA's partial sums of both steps are in place
      if (active) {
        float dot2 = 0.0f;
        if (ltid < l.batch) {
          float v[8];                            // remote reads issued together, summed in rank order
#pragma unroll
          for (int r = 0; r < 8; ++r) v[r] = r < csize ? *cluster.map_shared_rank(&sh.part[ltid], r) : 0.0f;
          float t = 0.0f;
#pragma unroll
          for (int r = 0; r < 8; ++r) if (r < csize) t += v[r];
          sh.resid[ltid] = row_residual(t, sh.label[qq][ltid], l.logistic);
        } else if (ltid >= 32 && ltid - 32 < l.batch) {
          float v[8];
#pragma unroll
          for (int r = 0; r < 8; ++r) v[r] = r < csize ? *cluster.map_shared_rank(&sh.part2[ltid - 32], r) : 0.0f;
#pragma unroll
          for (int r = 0; r < 8; ++r) if (r < csize) dot2 += v[r];
        }
        named_barrier(bar_id, kSmallThreads);
        if (ltid >= 32 && ltid - 32 < l.batch) {
          float corr = 0.0f;                     // <a, x_0 - x_1> / (lr/B) for the second step's row a
          for (int b = 0; b < l.batch; ++b) corr = fmaf(sh.gram[ltid - 32][b], sh.resid[b], corr);
          sh.resid2[ltid - 32] = row_residual(fmaf(-scale, corr, dot2), sh.label[qq + 1][ltid - 32], l.logistic);
        }
        named_barrier(bar_id, kSmallThreads);
        float4 g0 = make_float4(0.f, 0.f, 0.f, 0.f), g1 = g0;
#pragma unroll
        for (int j = 0; j < G; ++j) {
          const float rs = j < l.batch ? sh.resid[j] : 0.0f;
          g0.x = fmaf(rs, a0[j].x, g0.x); g0.y = fmaf(rs, a0[j].y, g0.y); g0.z = fmaf(rs, a0[j].z, g0.z); g0.w = fmaf(rs, a0[j].w, g0.w);
          g1.x = fmaf(rs, a1[j].x, g1.x); g1.y = fmaf(rs, a1[j].y, g1.y); g1.z = fmaf(rs, a1[j].z, g1.z); g1.w = fmaf(rs, a1[j].w, g1.w);
        }
        x[0].x -= scale * g0.x; x[0].y -= scale * g0.y; x[0].z -= scale * g0.z; x[0].w -= scale * g0.w;
        x[1].x -= scale * g1.x; x[1].y -= scale * g1.y; x[1].z -= scale * g1.z; x[1].w -= scale * g1.w;
        g0 = make_float4(0.f, 0.f, 0.f, 0.f); g1 = g0;
#pragma unroll
        for (int j = 0; j < G; ++j) {
          const float rs = j < l.batch ? sh.resid2[j] : 0.0f;
          g0.x = fmaf(rs, b0[j].x, g0.x); g0.y = fmaf(rs, b0[j].y, g0.y); g0.z = fmaf(rs, b0[j].z, g0.z); g0.w = fmaf(rs, b0[j].w, g0.w);
          g1.x = fmaf(rs, b1[j].x, g1.x); g1.y = fmaf(rs, b1[j].y, g1.y); g1.z = fmaf(rs, b1[j].z, g1.z); g1.w = fmaf(rs, b1[j].w, g1.w);
        }
        x[0].x -= scale * g0.x; x[0].y -= scale * g0.y; x[0].z -= scale * g0.z; x[0].w -= scale * g0.w;
        x[1].x -= scale * g1.x; x[1].y -= scale * g1.y; x[1].z -= scale * g1.z; x[1].w -= scale * g1.w;
      }
      cluster.sync();                            // all remote reads of part[] and part2[] are done before they are rewritten
      q += 2;
      continue;
    }
    rows_q = sh.rows[qq];
    if (active) {
      for (int s0 = 0; s0 < l.batch; s0 += G) {
        load_group(s0);
        float acc[G];
#pragma unroll
        for (int j = 0; j < G; ++j) {
          acc[j] = a0[j].x * x[0].x;
          acc[j] = fmaf(a0[j].y, x[0].y, acc[j]); acc[j] = fmaf(a0[j].z, x[0].z, acc[j]); acc[j] = fmaf(a0[j].w, x[0].w, acc[j]);
          acc[j] = fmaf(a1[j].x, x[1].x, acc[j]); acc[j] = fmaf(a1[j].y, x[1].y, acc[j]);
          acc[j] = fmaf(a1[j].z, x[1].z, acc[j]); acc[j] = fmaf(a1[j].w, x[1].w, acc[j]);
        }
        int row;
        const float tot = reduce_rows<G>(acc, lane, row);
        if ((lane & 1) == 0 && s0 + row < l.batch) sh.red[warp][s0 + row] = tot;
      }
      named_barrier(bar_id, kSmallThreads);
      if (ltid < l.batch) {
        float tot = 0.0f;
#pragma unroll
        for (int w = 0; w < kSmallThreads / 32; ++w) tot += sh.red[w][ltid];
        sh.part[ltid] = tot;
      }
    }
    cluster.sync();                              // every CTA's partial sums are in place
    if (active) {
      if (ltid < l.batch) {
        float v[8];                              // remote reads issued together, summed in rank order
#pragma unroll
        for (int r = 0; r < 8; ++r) v[r] = r < csize ? *cluster.map_shared_rank(&sh.part[ltid], r) : 0.0f;
        float tot = 0.0f;
#pragma unroll
        for (int r = 0; r < 8; ++r) if (r < csize) tot += v[r];
        sh.resid[ltid] = row_residual(tot, sh.label[qq][ltid], l.logistic);
      }
      named_barrier(bar_id, kSmallThreads);
      float4 g0 = make_float4(0.f, 0.f, 0.f, 0.f), g1 = g0;
      for (int s0 = 0; s0 < l.batch; s0 += G) {
        if (!one_group) load_group(s0);
#pragma unroll
        for (int j = 0; j < G; ++j) {
          const float rs = s0 + j < l.batch ? sh.resid[s0 + j] : 0.0f;
          g0.x = fmaf(rs, a0[j].x, g0.x); g0.y = fmaf(rs, a0[j].y, g0.y); g0.z = fmaf(rs, a0[j].z, g0.z); g0.w = fmaf(rs, a0[j].w, g0.w);
          g1.x = fmaf(rs, a1[j].x, g1.x); g1.y = fmaf(rs, a1[j].y, g1.y); g1.z = fmaf(rs, a1[j].z, g1.z); g1.w = fmaf(rs, a1[j].w, g1.w);
        }
      }
      x[0].x -= scale * g0.x; x[0].y -= scale * g0.y; x[0].z -= scale * g0.z; x[0].w -= scale * g0.w;
      x[1].x -= scale * g1.x; x[1].y -= scale * g1.y; x[1].z -= scale * g1.z; x[1].w -= scale * g1.w;
    }
    cluster.sync();                              // all remote reads of part[] are done before it is rewritten
    ++q;
  }
  // data rows are zero past d, so coordinates past d have stayed zero
  if (active) {
    *reinterpret_cast<float4*>(xrow) = x[0];
    if (ITERS > 1) *reinterpret_cast<float4*>(xrow + kSmallThreads * 4) = x[1];
  }
}

template <typename T, int ITERS>
__global__ void __launch_bounds__(kSmallThreads)
lsq_small_kernel(StoreView s, LsqView l, const NodeList nodes, int H, float lr, int csize) {
  cg::cluster_group cluster = cg::this_cluster();
  __shared__ SmallShared sh;
  const NodeDesc nd = nodes.get(blockIdx.x / csize);
  lsq_small_steps<T, ITERS>(cluster, s, l, true, nd.node, nd.event, H, lr, csize, threadIdx.x, 1, sh);
}

// -----------------------------------------------------------------------------------------
// Sequential gossip on short models in one launch (Section 3, "Sequential model": one interaction per
// time step). A single cluster of 256-thread CTAs walks the list of steps. In each step the two halves of
// every CTA take the H least-squares steps of the initiator and of the responder side by side (the
// cluster-wide routine above; a half idles when only the initiator steps); then CTA r < nblk performs the
// blocking interaction of block r, one sub-block per warp. Models travel between the two phases through
// global memory; the cluster barriers (release / acquire at cluster scope) order those accesses, all of
// which are made by CTAs of this one cluster. Every thread executes the same number of cluster barriers.
// -----------------------------------------------------------------------------------------
constexpr int kSeqThreads = 2 * kSmallThreads;

template <int BITS, int ITERS>
__global__ void __launch_bounds__(kSeqThreads)
lsq_sequence_kernel(StoreView s, LsqView l, const PairList steps, int H, float lr, int csize, int responders) {
  cg::cluster_group cluster = cg::this_cluster();
  __shared__ SmallShared sh[2];
  __shared__ float red[8];
  const int rank = (int)cluster.block_rank();
  const int half = threadIdx.x / kSmallThreads, ltid = threadIdx.x % kSmallThreads;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int t = 0; t < steps.n; ++t) {
    const PairDesc pd = steps.get(t);
    const int node = half == 0 ? pd.a : pd.b;
    const uint32_t event = half == 0 ? pd.lsa : pd.lsb;
    lsq_small_steps<float, ITERS>(cluster, s, l, half == 0 || responders != 0, node, event, H, lr, csize, ltid,
                                  1 + half, sh[half]);
    cluster.sync();                              // both models are complete in global memory
    if (rank < s.nblk && warp < 4) blocking_subblock<BITS>(s, pd, rank, warp, lane, red, 3);
    cluster.sync();                              // the averaged models are in place for the next step
  }
}

// -----------------------------------------------------------------------------------------
// Pair sampler: draws are generated in parallel (one per thread), accepted sequentially in
// draw order by thread 0 so that the result equals the sequential rejection procedure.
// -----------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
sample_pairs_kernel(const int32_t* __restrict__ adj, int n, int degree, int max_pairs, uint32_t launch_ctr, uint32_t k0,
                    uint32_t k1, int32_t* out_pairs, int32_t* out_count, uint8_t* used) {
  __shared__ int cand_i[256], cand_j[256];
  __shared__ int count_sh;
  for (int i = threadIdx.x; i < n; i += blockDim.x) used[i] = 0;
  if (threadIdx.x == 0) count_sh = 0;
  __syncthreads();
  const int64_t max_attempts = 16LL * max_pairs;
  for (int64_t base = 0; base < max_attempts; base += 256) {
    const int64_t attempt = base + threadIdx.x;
    if (attempt < max_attempts) {
      const uint4 w = philox4x32_10((uint32_t)attempt, 0u, launch_ctr, kStreamPairs, k0, k1);
      const int i = (int)uniform_int(w.x, (uint32_t)n);
      cand_i[threadIdx.x] = i;
      cand_j[threadIdx.x] = adj[(int64_t)i * degree + uniform_int(w.y, (uint32_t)degree)];
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      int count = count_sh;
      const int lim = (int)min((int64_t)256, max_attempts - base);
      for (int t = 0; t < lim && count < max_pairs; ++t) {
        const int i = cand_i[t], j = cand_j[t];
        if (used[i] || used[j]) continue;
        used[i] = used[j] = 1;
        out_pairs[2 * count] = i;
        out_pairs[2 * count + 1] = j;
        ++count;
      }
      count_sh = count;
    }
    __syncthreads();
    if (count_sh >= max_pairs) break;
  }
  if (threadIdx.x == 0) *out_count = count_sh;
}

// Small device-to-device row copy (queued row reads): a kernel instead of a copy-engine transfer, launched as
// a programmatic dependent, so that a row read queued between two interaction launches does not cost them
// the overlap of launch latency.
__global__ void __launch_bounds__(256)
row_copy_kernel(const uint8_t* __restrict__ src, uint8_t* __restrict__ dst, int64_t bytes) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x, stride = (int64_t)gridDim.x * blockDim.x;
  if (((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst)) & 15) == 0) {
    const int64_t vecs = bytes / 16;
    for (int64_t i = t; i < vecs; i += stride)
      reinterpret_cast<uint4*>(dst)[i] = reinterpret_cast<const uint4*>(src)[i];
    for (int64_t i = vecs * 16 + t; i < bytes; i += stride) dst[i] = src[i];
  } else {
    for (int64_t i = t; i < bytes; i += stride) dst[i] = src[i];
  }
}

__global__ void bf16_to_f32_kernel(const __nv_bfloat16* src, float* dst, int64_t count) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < count) dst[i] = __bfloat162float(src[i]);
}
__global__ void f32_to_bf16_kernel(const float* src, __nv_bfloat16* dst, int64_t count) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < count) dst[i] = __float2bfloat16_rn(src[i]);
}

// -----------------------------------------------------------------------------------------
// Launch wrappers
// -----------------------------------------------------------------------------------------
static inline unsigned cdiv(int64_t a, int64_t b) { return (unsigned)((a + b - 1) / b); }

cudaError_t launch_node_scalars(float* scalars_dev, int n, float offset_std, float drift_std, uint32_t key0,
                                uint32_t key1, cudaStream_t st, int* launches) {
  node_scalars_kernel<<<cdiv(n, 128), 128, 0, st>>>(scalars_dev, n, offset_std, drift_std, key0, key1);
  ++*launches;
  return cudaGetLastError();
}

cudaError_t launch_init_models(const StoreView& s, const float* scalars_dev, float init_std, cudaStream_t st,
                               int* launches) {
  const dim3 grid(cdiv((s.d + 3) / 4, 256), s.n);
  init_models_kernel<<<grid, 256, 0, st>>>(s, scalars_dev, init_std);
  ++*launches;
  return cudaGetLastError();
}

cudaError_t launch_lsq_data(const StoreView& s, const LsqView& l, void* A, float* xstar, float* bvec,
                            const float* scalars_dev, float noise_std, cudaStream_t st, int* launches) {
  const float inv_sqrt_d = (float)(1.0 / sqrt((double)s.d));
  const dim3 grid_a(cdiv(s.pitch / 4, 256), l.m, l.groups);
  const dim3 grid_l(l.m, l.groups);
  if (l.nodes_per_group > 256) return cudaErrorInvalidValue;
  xstar_kernel<<<cdiv(s.pitch / 4, 256), 256, 0, st>>>(xstar, s.pitch, s.d, s.key0, s.key1);
  if (l.dtype == 1) {
    auto* Ab = reinterpret_cast<__nv_bfloat16*>(A);
    lsq_matrix_kernel<<<grid_a, 256, 0, st>>>(Ab, s.pitch, s.d, l.m, inv_sqrt_d, s.key0, s.key1);
    lsq_labels_kernel<<<grid_l, 256, 0, st>>>(Ab, xstar, bvec, scalars_dev, s.pitch, s.d, l.m, l.nodes_per_group,
                                               noise_std, s.key0, s.key1, l.logistic);
  } else {
    auto* Af = reinterpret_cast<float*>(A);
    lsq_matrix_kernel<<<grid_a, 256, 0, st>>>(Af, s.pitch, s.d, l.m, inv_sqrt_d, s.key0, s.key1);
    lsq_labels_kernel<<<grid_l, 256, 0, st>>>(Af, xstar, bvec, scalars_dev, s.pitch, s.d, l.m, l.nodes_per_group,
                                               noise_std, s.key0, s.key1, l.logistic);
  }
  *launches += 3;
  return cudaGetLastError();
}

cudaError_t launch_local_synth(const StoreView& s, const NodeList& nodes, int count, int H, float lr,
                               float grad_std, const float* scalars_dev, cudaStream_t st, int* launches) {
  if (count == 0 || H == 0) return cudaSuccess;
  const dim3 grid(cdiv(s.pitch / 8, 256), count);
  local_synth_kernel<<<grid, 256, 0, st>>>(s, nodes, H, lr, grad_std, scalars_dev);
  ++*launches;
  return cudaGetLastError();
}

bool lsq_small_steps_in_pairs(int64_t pitch, int batch) {
  if (pitch > kSmallMaxPitch) return false;
  const int iters = pitch / (kSmallThreads * 4) <= 8 ? 1 : 2;
  return batch <= 16 / iters;
}

cudaError_t launch_local_lsq(const StoreView& s, const LsqView& l, const NodeList& nodes, int count, int H,
                             float lr, float* partial_dev, cudaStream_t st, int* launches) {
  if (count == 0 || H == 0) return cudaSuccess;
  if (l.batch > kLsqMaxBatch) return cudaErrorInvalidValue;
  if (s.pitch <= kSmallMaxPitch && l.batch <= kSmallMaxBatch) {
    // cluster of pitch / 512 CTAs (one 512-coordinate slice each) while that is at most 8, else pitch / 1024
    const int slices512 = (int)(s.pitch / (kSmallThreads * 4));
    const int csize = slices512 <= 8 ? slices512 : slices512 / 2;
    const int iters = slices512 <= 8 ? 1 : 2;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(count * csize));
    cfg.blockDim = dim3(kSmallThreads);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)csize;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e;
    if (l.dtype == 1) {
      e = iters == 1 ? cudaLaunchKernelEx(&cfg, lsq_small_kernel<__nv_bfloat16, 1>, s, l, nodes, H, lr, csize)
                     : cudaLaunchKernelEx(&cfg, lsq_small_kernel<__nv_bfloat16, 2>, s, l, nodes, H, lr, csize);
    } else {
      e = iters == 1 ? cudaLaunchKernelEx(&cfg, lsq_small_kernel<float, 1>, s, l, nodes, H, lr, csize)
                     : cudaLaunchKernelEx(&cfg, lsq_small_kernel<float, 2>, s, l, nodes, H, lr, csize);
    }
    ++*launches;
    return e != cudaSuccess ? e : cudaGetLastError();
  }
  const int64_t nchunks = lsq_chunks(s.d);
  const dim3 grid((unsigned)nchunks, count);
  for (int q = 0; q < H; ++q) {
    if (l.dtype == 1) {
      lsq_residual_kernel<__nv_bfloat16><<<grid, kLsqThreads, 0, st>>>(s, l, nodes, q, partial_dev, nchunks);
      lsq_update_kernel<__nv_bfloat16><<<grid, kLsqThreads, 0, st>>>(s, l, nodes, q, lr, partial_dev, nchunks);
    } else {
      lsq_residual_kernel<float><<<grid, kLsqThreads, 0, st>>>(s, l, nodes, q, partial_dev, nchunks);
      lsq_update_kernel<float><<<grid, kLsqThreads, 0, st>>>(s, l, nodes, q, lr, partial_dev, nchunks);
    }
    *launches += 2;
  }
  return cudaGetLastError();
}

bool lsq_sequence_supported(const StoreView& s, const LsqView& l) {
  return s.pitch <= kSmallMaxPitch && l.batch <= kSmallMaxBatch && l.dtype == 0;
}

cudaError_t launch_lsq_sequence(const StoreView& s, const LsqView& l, const PairList& steps, int H, float lr, int bits,
                                int responders, cudaStream_t st, int* launches) {
  if (steps.n == 0) return cudaSuccess;
  if (!lsq_sequence_supported(s, l)) return cudaErrorInvalidValue;
  const int slices512 = (int)(s.pitch / (kSmallThreads * 4));
  const int csize = slices512 <= 8 ? slices512 : slices512 / 2;
  const int iters = slices512 <= 8 ? 1 : 2;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)csize);            // one cluster walks the whole sequence
  cfg.blockDim = dim3(kSeqThreads);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)csize;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaErrorInvalidValue;
#define SWARM_SEQ_CASE(w)                                                                                      \
  case w:                                                                                                      \
    e = iters == 1 ? cudaLaunchKernelEx(&cfg, lsq_sequence_kernel<w, 1>, s, l, steps, H, lr, csize, responders) \
                   : cudaLaunchKernelEx(&cfg, lsq_sequence_kernel<w, 2>, s, l, steps, H, lr, csize, responders); \
    break;
  switch (bits) {
    SWARM_SEQ_CASE(2) SWARM_SEQ_CASE(3) SWARM_SEQ_CASE(4) SWARM_SEQ_CASE(5) SWARM_SEQ_CASE(6) SWARM_SEQ_CASE(7)
    SWARM_SEQ_CASE(8)
    default: return cudaErrorInvalidValue;
  }
#undef SWARM_SEQ_CASE
  ++*launches;
  return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_sample_pairs(const int32_t* adj_dev, int n, int degree, int max_pairs, uint32_t launch_ctr,
                                uint32_t key0, uint32_t key1, int32_t* out_pairs_dev, int32_t* out_count_dev,
                                uint8_t* used_dev, cudaStream_t st, int* launches) {
  sample_pairs_kernel<<<1, 256, 0, st>>>(adj_dev, n, degree, max_pairs, launch_ctr, key0, key1, out_pairs_dev,
                                         out_count_dev, used_dev);
  ++*launches;
  return cudaGetLastError();
}

cudaError_t launch_row_copy(const void* src_dev, void* dst_dev, int64_t bytes, cudaStream_t st, int* launches) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)std::min<int64_t>(cdiv(bytes, 16 * 256), 16));
  cfg.blockDim = dim3(256);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, row_copy_kernel, reinterpret_cast<const uint8_t*>(src_dev),
                                           reinterpret_cast<uint8_t*>(dst_dev), bytes);
  ++*launches;
  return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_bf16_to_f32(const void* src, float* dst, int64_t count, cudaStream_t st, int* launches) {
  bf16_to_f32_kernel<<<cdiv(count, 256), 256, 0, st>>>(reinterpret_cast<const __nv_bfloat16*>(src), dst, count);
  ++*launches;
  return cudaGetLastError();
}
cudaError_t launch_f32_to_bf16(const float* src, void* dst, int64_t count, cudaStream_t st, int* launches) {
  f32_to_bf16_kernel<<<cdiv(count, 256), 256, 0, st>>>(src, reinterpret_cast<__nv_bfloat16*>(dst), count);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace swarm
