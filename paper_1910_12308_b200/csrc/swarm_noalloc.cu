// swarm_potential_static: the potential Gamma = sum_i ||X^i - mu||^2 of caller-held models, computed
// without allocating anything.
//
// Who needs this: code that holds all of its device memory up front and must not grow it afterwards --
// a serving or training process whose memory pool is sized once at start-up, a monitoring hook that runs
// inside somebody else's step and is not allowed to call cudaMalloc (which may synchronise the whole
// device and can fail late), or an embedding where the host framework owns the allocator and hands this
// library nothing but raw pointers. The regular swarm_potential needs a context, and the context
// allocates its scratch; this entry point takes the models and the result as plain device pointers and
// keeps its per-CTA partial sums in a fixed array that is part of the loaded library image.
//
// Cost of that choice: every GPU that loads the library carries the array (512 KiB) until the process
// exits, the size of the problem is capped (SWARM_STATIC_MAX_D coordinates), and all calls share the one
// array, so two calls whose kernels can overlap on the same GPU (different streams, no dependency) would
// overwrite each other's partial sums. Calls on one stream are safe. The array keeps whatever the last
// call left in it; nothing in it has to start at zero because each call first overwrites every slot it
// later reads.
//
// The address of the array is looked up once per device, on the first call made while that device is
// current. That first call should be made before any stream capture begins.
#include <mutex>

#include "../../include/swarm.h"
#include "swarm_dev.cuh"

namespace {

constexpr int kThreads = 128;             // 4 columns per thread -> 512 columns per CTA
constexpr int kRows = 8;                  // rows loaded per batch of independent loads
constexpr int64_t kMaxPartials = SWARM_STATIC_MAX_D / (kThreads * 4);   // 65,536 doubles = 512 KiB
constexpr int kMaxDevices = 64;

static __device__ __align__(256) double g_static_partials[kMaxPartials];

// Host-side record of the device address of the array, per device ordinal.
double* g_partials_addr[kMaxDevices] = {};
std::mutex g_setup_mutex;

// Same arithmetic as the context-based kernel: per column the first row is the shift (exact in double),
// Gamma_col = sum s^2 - (sum s)^2 / n with s = x_i - x_0; columns past d are skipped.
// `vec` (decided on the host): every row starts on a 16-byte boundary, so four columns travel as one 128-bit load.
__global__ void __launch_bounds__(kThreads)
static_potential_partial_kernel(const float* __restrict__ x, int n, int64_t d, int64_t pitch, int vec,
                                double* __restrict__ partial) {
  const int64_t c4 = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  double gamma = 0.0;
  if (c4 * 4 < d) {
    const float* col = x + c4 * 4;
    const bool whole = vec != 0 && c4 * 4 + 3 < d;
    double b[4], sm[4] = {0.0, 0.0, 0.0, 0.0}, sq[4] = {0.0, 0.0, 0.0, 0.0};
    auto load = [&](int64_t row, float v[4]) {
      const float* p = col + row * pitch;
      if (whole) {
        const float4 t = *reinterpret_cast<const float4*>(p);
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
      } else {
#pragma unroll
        for (int t = 0; t < 4; ++t) v[t] = (c4 * 4 + t < d) ? p[t] : 0.0f;
      }
    };
    float first[4];
    load(0, first);
#pragma unroll
    for (int t = 0; t < 4; ++t) b[t] = (double)first[t];
    int i = 1;
    for (; i + kRows <= n; i += kRows) {
      float v[kRows][4];
#pragma unroll
      for (int u = 0; u < kRows; ++u) load(i + u, v[u]);
#pragma unroll
      for (int u = 0; u < kRows; ++u)
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          const double s = (double)v[u][t] - b[t];
          sm[t] += s;
          sq[t] = fma(s, s, sq[t]);
        }
    }
    for (; i < n; ++i) {
      float v[4];
      load(i, v);
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const double s = (double)v[t] - b[t];
        sm[t] += s;
        sq[t] = fma(s, s, sq[t]);
      }
    }
    const double inv_n = 1.0 / (double)n;
#pragma unroll
    for (int t = 0; t < 4; ++t) gamma += sq[t] - sm[t] * sm[t] * inv_n;
  }
  __shared__ double red[kThreads / 32];
  gamma = swarm::warp_sum(gamma);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = gamma;
  __syncthreads();
  if (threadIdx.x == 0) {
    double tot = 0.0;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) tot += red[w];
    partial[blockIdx.x] = tot;          // every slot read by the final kernel is written here first
  }
}

__global__ void __launch_bounds__(1024)
static_potential_final_kernel(const double* __restrict__ partial, int64_t count, double* __restrict__ out) {
  double acc = 0.0;
  for (int64_t i = threadIdx.x; i < count; i += 1024) acc += partial[i];
  __shared__ double red[32];
  acc = swarm::warp_sum(acc);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x < 32) {
    double v = swarm::warp_sum(red[threadIdx.x]);
    if (threadIdx.x == 0) *out = v;
  }
}

}  // namespace

extern "C" int swarm_potential_static(const float* x_dev, int32_t n, int64_t d, int64_t pitch,
                                      double* out_gamma_dev, void* cuda_stream) {
  if (!x_dev || !out_gamma_dev || n < 2 || d < 1 || pitch < d) return SWARM_EINVAL;
  if (((uintptr_t)x_dev & 3) != 0 || ((uintptr_t)out_gamma_dev & 7) != 0) return SWARM_EINVAL;   // not a float / double address
  if (d > SWARM_STATIC_MAX_D) return SWARM_EINVAL;      // beyond the capacity of the fixed scratch array
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return SWARM_ECUDA;
  if (dev < 0 || dev >= kMaxDevices) return SWARM_EINVAL;
  double* partial = nullptr;
  {
    // first call on this device: resolve the device address of the array (the symbol's name is only a
    // host-side handle and must never be handed to a kernel as if it were a pointer)
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_partials_addr[dev]) {
      void* p = nullptr;
      if (cudaGetSymbolAddress(&p, g_static_partials) != cudaSuccess || !p) { cudaGetLastError(); return SWARM_ECUDA; }
      g_partials_addr[dev] = (double*)p;
    }
    partial = g_partials_addr[dev];
  }
  const int64_t parts = ((d + 3) / 4 + kThreads - 1) / kThreads;      // <= kMaxPartials by the check above
  cudaStream_t st = (cudaStream_t)cuda_stream;
  // 128-bit loads only when every row starts on a 16-byte boundary: base address and row pitch both count
  // (a view into a larger tensor can have an aligned pitch and a base that is off by one float)
  const int vec = (((uintptr_t)x_dev & 15) == 0 && (pitch & 3) == 0) ? 1 : 0;
  static_potential_partial_kernel<<<(unsigned)parts, kThreads, 0, st>>>(x_dev, n, d, pitch, vec, partial);
  static_potential_final_kernel<<<1, 1024, 0, st>>>(partial, parts, out_gamma_dev);
  return cudaGetLastError() == cudaSuccess ? SWARM_OK : SWARM_ECUDA;
}
