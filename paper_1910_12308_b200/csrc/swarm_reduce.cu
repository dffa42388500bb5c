// Mean model mu = (1/n) sum_i X^i and potential Gamma = sum_i ||X^i - mu||^2 (Section 4).
// Both stream X[n][d] once: a thread owns 4 adjacent columns and walks down the n rows.
#include <algorithm>

#include "swarm_dev.cuh"
#include "swarm_internal.h"

namespace swarm {

constexpr int kRedThreads = 128;
constexpr int kPotentialMaxCtas = 148 * 16;   // one resident wave of 128-thread CTAs on 148 SMs
constexpr int kRowUnroll = 8;

// Programmatic dependent launch (see swarm_interact.cu): the two kernels below may become resident while their
// predecessor in the stream drains; they touch no global memory before the wait returns.
__device__ __forceinline__ void dependent_launch_prologue() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

// mu[k]: rows summed in double in row order, divided by n, rounded once.
__global__ void __launch_bounds__(kRedThreads)
mean_model_kernel(StoreView s, float* __restrict__ out) {
  dependent_launch_prologue();
  const int64_t c4 = (int64_t)blockIdx.x * kRedThreads + threadIdx.x;
  if (c4 * 4 >= s.d) return;
  const float* col = s.X + c4 * 4;
  double acc[4] = {0.0, 0.0, 0.0, 0.0};
  int i = 0;
  for (; i + kRowUnroll <= s.n; i += kRowUnroll) {
    float4 v[kRowUnroll];
#pragma unroll
    for (int u = 0; u < kRowUnroll; ++u) v[u] = *reinterpret_cast<const float4*>(col + (int64_t)(i + u) * s.pitch);
#pragma unroll
    for (int u = 0; u < kRowUnroll; ++u) {
      acc[0] += (double)v[u].x; acc[1] += (double)v[u].y; acc[2] += (double)v[u].z; acc[3] += (double)v[u].w;
    }
  }
  for (; i < s.n; ++i) {
    const float4 v = *reinterpret_cast<const float4*>(col + (int64_t)i * s.pitch);
    acc[0] += (double)v.x; acc[1] += (double)v.y; acc[2] += (double)v.z; acc[3] += (double)v.w;
  }
  const double inv = (double)s.n;
#pragma unroll
  for (int t = 0; t < 4; ++t)
    if (c4 * 4 + t < s.d) out[c4 * 4 + t] = (float)(acc[t] / inv);
}

// Per column, with the first row as shift (exact in double): s_i = x_i - x_0,
// Gamma_col = sum s_i^2 - (sum s_i)^2 / n. The shift keeps the subtraction benign when the
// models are close to each other but far from the origin. CTA partials go to scratch.
// The CTA that finishes last (a ticket counter tells) sums the partials in a fixed pattern, so the result
// does not depend on which CTA that is, writes it to out_dev and, when out_host is given (pinned host
// memory mapped into the device's address space), to the host directly, and resets the ticket.
__global__ void __launch_bounds__(kRedThreads)
potential_partial_kernel(StoreView s, double* __restrict__ partial, unsigned int* __restrict__ ticket,
                         double* __restrict__ out_dev, double* __restrict__ out_host) {
  dependent_launch_prologue();
  double gamma = 0.0;
  // a fixed number of CTAs walks the column groups, so the sum of a CTA (and with it the result) depends on
  // the grid size only, and the last CTA has few partials to add up
  for (int64_t c4 = (int64_t)blockIdx.x * kRedThreads + threadIdx.x; c4 * 4 < s.d;
       c4 += (int64_t)gridDim.x * kRedThreads) {
    const float* col = s.X + c4 * 4;
    const float4 x0 = *reinterpret_cast<const float4*>(col);
    const double b0 = x0.x, b1 = x0.y, b2 = x0.z, b3 = x0.w;
    double sm[4] = {0.0, 0.0, 0.0, 0.0}, sq[4] = {0.0, 0.0, 0.0, 0.0};
    int i = 1;
    for (; i + kRowUnroll <= s.n; i += kRowUnroll) {
      float4 v[kRowUnroll];
#pragma unroll
      for (int u = 0; u < kRowUnroll; ++u) v[u] = *reinterpret_cast<const float4*>(col + (int64_t)(i + u) * s.pitch);
#pragma unroll
      for (int u = 0; u < kRowUnroll; ++u) {
        const double d0 = (double)v[u].x - b0, d1 = (double)v[u].y - b1, d2 = (double)v[u].z - b2, d3 = (double)v[u].w - b3;
        sm[0] += d0; sm[1] += d1; sm[2] += d2; sm[3] += d3;
        sq[0] = fma(d0, d0, sq[0]); sq[1] = fma(d1, d1, sq[1]); sq[2] = fma(d2, d2, sq[2]); sq[3] = fma(d3, d3, sq[3]);
      }
    }
    for (; i < s.n; ++i) {
      const float4 v = *reinterpret_cast<const float4*>(col + (int64_t)i * s.pitch);
      const double d0 = (double)v.x - b0, d1 = (double)v.y - b1, d2 = (double)v.z - b2, d3 = (double)v.w - b3;
      sm[0] += d0; sm[1] += d1; sm[2] += d2; sm[3] += d3;
      sq[0] = fma(d0, d0, sq[0]); sq[1] = fma(d1, d1, sq[1]); sq[2] = fma(d2, d2, sq[2]); sq[3] = fma(d3, d3, sq[3]);
    }
    const double inv_n = 1.0 / (double)s.n;
#pragma unroll
    for (int t = 0; t < 4; ++t)                      // padding columns are all-zero: contribute 0
      gamma += sq[t] - sm[t] * sm[t] * inv_n;
  }
  __shared__ double red[kRedThreads / 32];
  __shared__ bool last;
  gamma = warp_sum(gamma);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = gamma;
  __syncthreads();
  if (threadIdx.x == 0) {
    double tot = 0.0;
#pragma unroll
    for (int w = 0; w < kRedThreads / 32; ++w) tot += red[w];
    partial[blockIdx.x] = tot;
    __threadfence();                                     // the partial is visible before the ticket is taken
    last = atomicAdd(ticket, 1u) == gridDim.x - 1;
  }
  __syncthreads();
  if (!last) return;
  __threadfence();
  double acc = 0.0;
  for (int64_t i = threadIdx.x; i < (int64_t)gridDim.x; i += kRedThreads) acc += __ldcg(partial + i);
  acc = warp_sum(acc);
  __syncthreads();                                       // red[] was read above
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double tot = 0.0;
#pragma unroll
    for (int w = 0; w < kRedThreads / 32; ++w) tot += red[w];
    *out_dev = tot;
    if (out_host) *out_host = tot;
    *ticket = 0u;
  }
}

// ---------------------------------------------------------------------------------------------
// Auxiliary potentials of the staleness analysis (appendix, "Notation and Auxiliary Potential
// Functions"): with X^_i = B_i the model of node i at its last initiation and m_i the mean model
// recorded then,  Gamma^_t = sum_i ||B_i - mu_t||^2,  A_t = sum_i ||B_i - m_i||^2 (each term frozen
// at the initiation),  B_t = sum_i ||mu_t - m_i||^2.  mu is the fp32 mean model of the kernel above.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float4 column_mean(const StoreView& s, const float* col) {
  double acc[4] = {0.0, 0.0, 0.0, 0.0};
  int i = 0;
  for (; i + kRowUnroll <= s.n; i += kRowUnroll) {
    float4 v[kRowUnroll];
#pragma unroll
    for (int u = 0; u < kRowUnroll; ++u) v[u] = *reinterpret_cast<const float4*>(col + (int64_t)(i + u) * s.pitch);
#pragma unroll
    for (int u = 0; u < kRowUnroll; ++u) {
      acc[0] += (double)v[u].x; acc[1] += (double)v[u].y; acc[2] += (double)v[u].z; acc[3] += (double)v[u].w;
    }
  }
  for (; i < s.n; ++i) {
    const float4 v = *reinterpret_cast<const float4*>(col + (int64_t)i * s.pitch);
    acc[0] += (double)v.x; acc[1] += (double)v.y; acc[2] += (double)v.z; acc[3] += (double)v.w;
  }
  const double inv = (double)s.n;
  return make_float4((float)(acc[0] / inv), (float)(acc[1] / inv), (float)(acc[2] / inv), (float)(acc[3] / inv));
}

__device__ __forceinline__ double sqdist4(const float4 a, const float4 b) {
  const double d0 = (double)a.x - (double)b.x, d1 = (double)a.y - (double)b.y;
  const double d2 = (double)a.z - (double)b.z, d3 = (double)a.w - (double)b.w;
  return fma(d0, d0, fma(d1, d1, fma(d2, d2, d3 * d3)));
}

// CTA-wide sum; the result is valid in thread 0. `red` holds one double per warp.
__device__ __forceinline__ double cta_sum(double v, double* red) {
  v = warp_sum(v);
  __syncthreads();                                   // red may still be read from the previous use
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  double tot = 0.0;
  if (threadIdx.x == 0) {
#pragma unroll
    for (int w = 0; w < kRedThreads / 32; ++w) tot += red[w];
  }
  return tot;
}

// The listed nodes initiated in the launch that just ran: their mean-model record becomes the current
// mean, and partial[t][cta] receives this CTA's share of ||B_node - mu||^2.
__global__ void __launch_bounds__(kRedThreads)
staleness_record_kernel(StoreView s, float* __restrict__ mu_hist, NodeList list, double* __restrict__ partial) {
  __shared__ double red[kRedThreads / 32];
  const int64_t c4 = (int64_t)blockIdx.x * kRedThreads + threadIdx.x;
  const bool live = c4 * 4 < s.d;
  float4 mu = make_float4(0.f, 0.f, 0.f, 0.f);
  if (live) mu = column_mean(s, s.X + c4 * 4);
  for (int t = 0; t < list.n; ++t) {
    const int node = list.get(t).node;
    double acc = 0.0;
    if (live) {
      const int64_t off = (int64_t)node * s.pitch + c4 * 4;
      *reinterpret_cast<float4*>(mu_hist + off) = mu;
      acc = sqdist4(*reinterpret_cast<const float4*>(s.B + off), mu);   // padding columns: 0 - 0
    }
    const double tot = cta_sum(acc, red);
    if (threadIdx.x == 0) partial[(int64_t)t * gridDim.x + blockIdx.x] = tot;
  }
}

// a_hist[node of entry t] = sum of its partials in index order; one CTA per entry.
__global__ void __launch_bounds__(kRedThreads)
staleness_record_final_kernel(const double* __restrict__ partial, int64_t parts, NodeList list,
                              double* __restrict__ a_hist) {
  __shared__ double red[kRedThreads / 32];
  const int t = blockIdx.x;
  double acc = 0.0;
  for (int64_t i = threadIdx.x; i < parts; i += kRedThreads) acc += partial[(int64_t)t * parts + i];
  const double tot = cta_sum(acc, red);
  if (threadIdx.x == 0) a_hist[list.get(t).node] = tot;
}

// partial[0][cta] = share of Gamma^, partial[1][cta] = share of B_t.
__global__ void __launch_bounds__(kRedThreads)
aux_potential_partial_kernel(StoreView s, const float* __restrict__ mu_hist, double* __restrict__ partial) {
  __shared__ double red[kRedThreads / 32];
  const int64_t c4 = (int64_t)blockIdx.x * kRedThreads + threadIdx.x;
  double gh = 0.0, bt = 0.0;
  if (c4 * 4 < s.d) {
    const float4 mu = column_mean(s, s.X + c4 * 4);
    for (int i = 0; i < s.n; ++i) {
      const int64_t off = (int64_t)i * s.pitch + c4 * 4;
      gh += sqdist4(*reinterpret_cast<const float4*>(s.B + off), mu);
      bt += sqdist4(mu, *reinterpret_cast<const float4*>(mu_hist + off));
    }
  }
  const double g = cta_sum(gh, red);
  const double b = cta_sum(bt, red);
  if (threadIdx.x == 0) { partial[blockIdx.x] = g; partial[(int64_t)gridDim.x + blockIdx.x] = b; }
}

// out[0] = Gamma^, out[1] = A_t, out[2] = B_t; CTA q sums its own series in index order.
__global__ void __launch_bounds__(kRedThreads)
aux_potential_final_kernel(const double* __restrict__ partial, int64_t parts, const double* __restrict__ a_hist,
                           int n, double* __restrict__ out) {
  __shared__ double red[kRedThreads / 32];
  const int q = blockIdx.x;
  const double* src = q == 0 ? partial : (q == 1 ? a_hist : partial + parts);
  const int64_t count = q == 1 ? (int64_t)n : parts;
  double acc = 0.0;
  for (int64_t i = threadIdx.x; i < count; i += kRedThreads) acc += src[i];
  const double tot = cta_sum(acc, red);
  if (threadIdx.x == 0) out[q] = tot;
}

cudaError_t launch_staleness_record(const StoreView& s, float* mu_hist, const NodeList& list, double* partial_dev,
                                    double* a_hist_dev, cudaStream_t st, int* launches) {
  if (list.n <= 0) return cudaSuccess;
  const int64_t parts = potential_partials(s.d);
  staleness_record_kernel<<<(unsigned)parts, kRedThreads, 0, st>>>(s, mu_hist, list, partial_dev);
  staleness_record_final_kernel<<<(unsigned)list.n, kRedThreads, 0, st>>>(partial_dev, parts, list, a_hist_dev);
  *launches += 2;
  return cudaGetLastError();
}

cudaError_t launch_aux_potentials(const StoreView& s, const float* mu_hist, const double* a_hist_dev,
                                  double* partial_dev, double* out_dev, cudaStream_t st, int* launches) {
  const int64_t parts = potential_partials(s.d);
  aux_potential_partial_kernel<<<(unsigned)parts, kRedThreads, 0, st>>>(s, mu_hist, partial_dev);
  aux_potential_final_kernel<<<3, kRedThreads, 0, st>>>(partial_dev, parts, a_hist_dev, s.n, out_dev);
  *launches += 2;
  return cudaGetLastError();
}

int64_t potential_partials(int64_t d) { return ((d + 3) / 4 + kRedThreads - 1) / kRedThreads; }

template <typename Kernel, typename... Args>
static cudaError_t launch_dependent(Kernel kernel, unsigned grid, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kRedThreads);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, args...);
  return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_mean_model(const StoreView& s, float* out_dev, cudaStream_t st, int* launches) {
  ++*launches;
  return launch_dependent(mean_model_kernel, (unsigned)potential_partials(s.d), st, s, out_dev);
}

cudaError_t launch_potential(const StoreView& s, double* partial_dev, unsigned int* ticket_dev, double* out_dev,
                             double* out_host_mapped, cudaStream_t st, int* launches) {
  const int64_t parts = std::min<int64_t>(potential_partials(s.d), kPotentialMaxCtas);
  ++*launches;
  return launch_dependent(potential_partial_kernel, (unsigned)parts, st, s, partial_dev, ticket_dev, out_dev, out_host_mapped);
}

}  // namespace swarm
