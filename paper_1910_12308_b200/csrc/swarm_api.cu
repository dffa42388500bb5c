// C ABI and host scheduler: context, device store, argument validation, counters, staging of
// pair / node descriptors and kernel launches. All arithmetic of the method runs in the kernels.
#include <algorithm>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "../../include/swarm.h"
#include "swarm_dev.cuh"
#include "swarm_internal.h"

using namespace swarm;

namespace {

// process-wide allocator hook: read by swarm_init, written by swarm_set_allocator, under g_alloc_mutex
std::mutex g_alloc_mutex;
swarm_alloc_fn g_alloc = nullptr;
swarm_free_fn g_free = nullptr;
void* g_alloc_user = nullptr;

constexpr int kStageSlots = 8;
constexpr size_t kReadQueueBytes = 1u << 20;     // device ring (and pinned mirror) of queued row reads
constexpr size_t kReadQueueMaxRow = 64u << 10;   // longer rows take the copy engine

}  // namespace

struct swarm_ctx {
  int32_t n = 0;
  int64_t d = 0, pitch = 0, nblk = 0;
  int32_t topo_kind = 0, degree = 0;
  uint64_t seed = 0;
  int device = 0;
  cudaStream_t stream = nullptr;
  swarm_config cfg{};
  int last_cuda = 0;
  int64_t launches = 0;
  bool custom_alloc = false;
  swarm_alloc_fn alloc_fn = nullptr;
  swarm_free_fn free_fn = nullptr;
  void* alloc_user = nullptr;

  // host mirrors
  std::vector<int32_t> adj;          // n * degree
  std::vector<uint32_t> w, ls;       // buffer write counters, local-step counters
  std::vector<int32_t> pbits;        // code width currently held by each buffer (0 = none)
  std::vector<uint32_t> wo, tau;     // own-register write counters, staleness clocks
  int32_t p_mode = 0;                // convention the buffers were last written in (0 none, 1 single buffer, 2 registers)
  uint32_t launch_ctr = 0;
  int32_t b_stale = 0;
  int32_t groups = 0, nodes_per_group = 0;

  // device store
  float* X = nullptr;
  float* B = nullptr;
  uint8_t* codes = nullptr;
  int8_t* exps = nullptr;
  uint8_t* own = nullptr;            // two-register protocol: own registers [n][nblk][2048] (low-byte plane, high-byte plane)
  int32_t own_prefix = 16;           // bits of a partner's own register that a reader consumes
  int8_t* oexps = nullptr;           // [n][nblk]
  int32_t* adj_dev = nullptr;
  float* scalars = nullptr;          // n * 3
  void* A = nullptr;
  float* bvec = nullptr;
  float* xstar = nullptr;
  float* lsq_partial = nullptr;      // n * batch * chunks
  float* tc_partial = nullptr;       // tensor-core path: split-K partials of the residuals
  void* tc_resid = nullptr;          // tensor-core path: residuals as bf16 hi / lo
  float* gram = nullptr;             // tensor-core path: Gram matrices of the data matrices (nullptr: not kept)
  bool sweep_backwards = false;      // direction of the next interaction launch's walk over its (pair, block) list
  std::vector<uint64_t> touched;     // per node: when an interaction kernel last visited its rows (a running count)
  uint64_t touch_seq = 0;
  int* kernel_status = nullptr;      // set by a kernel whose bounded wait expired
  int* kernel_status_host = nullptr; // pinned
  bool status_pending = false;       // kernels with bounded waits were launched since the status word was last read
  bool poisoned = false;             // a bounded wait expired: the state is undefined until swarm_configure
  uint32_t wait_limit = 0;           // polls per bounded device wait
  double* pot_partial = nullptr;
  double* pot_out = nullptr;         // 4 doubles, then the ticket counter of the potential kernel
  double* pot_host_dev = nullptr;    // device-visible address of pot_host (nullptr: not mapped)
  // auxiliary potentials of the staleness analysis (off until swarm_track_staleness)
  bool track = false;
  float* mu_hist = nullptr;          // [n][pitch] mean model at each node's last initiation
  double* a_hist = nullptr;          // n: ||snapshot - mean||^2 at each node's last initiation
  double* aux_partial = nullptr;     // max(n, 2) * potential_partials(d)
  int32_t* pairs_out_dev = nullptr;  // 2 * n/2 + 1 (sampler result, count last)
  uint8_t* used_dev = nullptr;       // n
  float* convert_tmp = nullptr;      // pitch floats (bf16 row conversion)

  // staging ring for descriptors (pinned host + device), guarded by events
  void* stage_host = nullptr;
  void* stage_dev = nullptr;
  size_t stage_slot_bytes = 0;
  cudaEvent_t stage_event[kStageSlots] = {};
  int stage_next = 0;
  double* pot_host = nullptr;        // pinned
  int32_t* pairs_out_host = nullptr; // pinned

  // queued row reads (swarm_get_tensor_async): a small kernel copies the row into a device ring, which keeps the
  // chain of programmatic dependent launches intact; the used part of the ring travels to its pinned mirror in one
  // transfer at the next synchronising call, after which the host hands the rows to their destinations
  struct QueuedRead { void* dst; size_t off, bytes; };
  uint8_t* rq_dev = nullptr;
  uint8_t* rq_host = nullptr;        // pinned
  size_t rq_used = 0;
  std::vector<QueuedRead> rq;
};

namespace {

struct DeviceGuard {
  int prev = 0;
  explicit DeviceGuard(int dev) { cudaGetDevice(&prev); if (prev != dev) cudaSetDevice(dev); else prev = -1; }
  ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

int fail_cuda(swarm_ctx* c, cudaError_t e) { c->last_cuda = (int)e; return SWARM_ECUDA; }

#define SW_CUDA(ctx, call)                                   \
  do {                                                       \
    cudaError_t e__ = (call);                                \
    if (e__ != cudaSuccess) return fail_cuda((ctx), e__);    \
  } while (0)

// Every wait on the context's stream goes through here: rows queued by swarm_get_tensor_async ride along
// (one transfer of the ring's used part) and are handed to their destinations once the stream is idle.
// The status word of the kernels with bounded waits travels the same way when such kernels ran since it was last
// read; once it has been seen set, every synchronising call reports the expired wait (cudaErrorLaunchTimeout).
int ctx_sync(swarm_ctx* c, bool report_expired_wait = true) {
  if (!c->rq.empty())
    SW_CUDA(c, cudaMemcpyAsync(c->rq_host, c->rq_dev, c->rq_used, cudaMemcpyDeviceToHost, c->stream));
  if (c->status_pending)
    SW_CUDA(c, cudaMemcpyAsync(c->kernel_status_host, c->kernel_status, sizeof(int), cudaMemcpyDeviceToHost, c->stream));
  SW_CUDA(c, cudaStreamSynchronize(c->stream));
  for (const auto& q : c->rq) std::memcpy(q.dst, c->rq_host + q.off, q.bytes);
  c->rq.clear();
  c->rq_used = 0;
  if (c->status_pending) {
    c->status_pending = false;
    if (*c->kernel_status_host != 0) c->poisoned = true;
  }
  if (c->poisoned && report_expired_wait) return fail_cuda(c, cudaErrorLaunchTimeout);
  return SWARM_OK;
}
#define SW_SYNC(ctx)                                         \
  do {                                                       \
    const int rc__ = ctx_sync(ctx);                          \
    if (rc__ != SWARM_OK) return rc__;                       \
  } while (0)

void* dev_alloc(swarm_ctx* c, size_t bytes) {
  if (bytes == 0) bytes = 256;
  void* p = nullptr;
  if (c->custom_alloc) p = c->alloc_fn(bytes, c->alloc_user);
  else if (cudaMalloc(&p, bytes) != cudaSuccess) { cudaGetLastError(); p = nullptr; }
  return p;
}
void dev_free(swarm_ctx* c, void* p) {
  if (!p) return;
  if (c->custom_alloc) c->free_fn(p, c->alloc_user); else cudaFree(p);
}

StoreView view_of(const swarm_ctx* c) {
  StoreView s;
  s.X = c->X; s.B = c->B; s.codes = c->codes; s.exps = c->exps; s.own = c->own; s.oexps = c->oexps;
  s.pitch = c->pitch; s.d = c->d; s.nblk = c->nblk; s.n = c->n;
  s.key0 = (uint32_t)c->seed; s.key1 = (uint32_t)(c->seed >> 32);
  s.rk = philox_round_keys(s.key0, s.key1);
  division_magic((uint64_t)c->nblk, &s.nblk_magic, &s.nblk_shift);
  s.backwards = 0;
  return s;
}
LsqView lsq_of(const swarm_ctx* c) {
  LsqView l;
  l.A = c->A; l.bvec = c->bvec; l.gram = c->gram; l.m = c->cfg.lsq_m; l.batch = c->cfg.lsq_batch; l.dtype = c->cfg.lsq_dtype;
  l.groups = c->groups; l.nodes_per_group = c->nodes_per_group;
  l.logistic = c->cfg.objective == SWARM_OBJ_LOGISTIC ? 1 : 0;
  return l;
}

// Communication graph (Section 2). Random k-regular graphs are unions of k/2 Hamiltonian
// cycles; a cycle comes from a Fisher-Yates shuffle driven by the topology stream, and a draw
// that would repeat an existing edge is discarded and redrawn.
bool build_graph(swarm_ctx* c) {
  const int n = c->n;
  auto& adj = c->adj;
  if (c->topo_kind == SWARM_TOPO_COMPLETE) {
    c->degree = n - 1;
    adj.clear();
    for (int i = 0; i < n; ++i)
      for (int j = 0; j < n; ++j)
        if (j != i) adj.push_back(j);
    return true;
  }
  if (c->topo_kind == SWARM_TOPO_RING) {
    if (n < 3) return false;
    c->degree = 2;
    adj.clear();
    for (int i = 0; i < n; ++i) { adj.push_back((i + n - 1) % n); adj.push_back((i + 1) % n); }
    return true;
  }
  if (c->topo_kind != SWARM_TOPO_REGULAR) return false;
  const int k = c->degree;
  if (n < 3 || k < 2 || (k & 1) || k > n - 1) return false;
  std::vector<std::vector<int>> nb(n);
  auto linked = [&](int u, int v) { return std::find(nb[u].begin(), nb[u].end(), v) != nb[u].end(); };
  const uint32_t key0 = (uint32_t)c->seed, key1 = (uint32_t)(c->seed >> 32);
  std::vector<int> order(n);
  int accepted = 0;
  for (uint32_t attempt = 0; accepted < k / 2; ++attempt) {
    if (attempt >= 4096) return false;
    for (int i = 0; i < n; ++i) order[i] = i;
    uint4 words = make_uint4(0, 0, 0, 0);
    int have = -1;
    for (int i = n - 1; i > 0; --i) {
      if (i / 4 != have) { have = i / 4; words = philox4x32_10((uint32_t)have, 0u, attempt, kStreamTopology, key0, key1); }
      const uint32_t wd = (i & 3) == 0 ? words.x : (i & 3) == 1 ? words.y : (i & 3) == 2 ? words.z : words.w;
      std::swap(order[i], order[uniform_int(wd, (uint32_t)i + 1u)]);
    }
    bool repeat = false;
    for (int t = 0; t < n; ++t)
      if (linked(order[t], order[(t + 1) % n])) { repeat = true; break; }
    if (repeat) continue;
    for (int t = 0; t < n; ++t) {
      const int u = order[t], v = order[(t + 1) % n];
      nb[u].push_back(v);
      nb[v].push_back(u);
    }
    ++accepted;
  }
  adj.clear();
  for (int i = 0; i < n; ++i) {
    std::sort(nb[i].begin(), nb[i].end());
    if ((int)nb[i].size() != k) return false;
    adj.insert(adj.end(), nb[i].begin(), nb[i].end());
  }
  return true;
}

void free_objective(swarm_ctx* c) {
  dev_free(c, c->A); c->A = nullptr;
  dev_free(c, c->bvec); c->bvec = nullptr;
  dev_free(c, c->xstar); c->xstar = nullptr;
  dev_free(c, c->lsq_partial); c->lsq_partial = nullptr;
  dev_free(c, c->tc_partial); c->tc_partial = nullptr;
  dev_free(c, c->tc_resid); c->tc_resid = nullptr;
  dev_free(c, c->gram); c->gram = nullptr;
  dev_free(c, c->convert_tmp); c->convert_tmp = nullptr;
  dev_free(c, c->B); c->B = nullptr;
  dev_free(c, c->own); c->own = nullptr;
  dev_free(c, c->oexps); c->oexps = nullptr;
  dev_free(c, c->mu_hist); c->mu_hist = nullptr;
  dev_free(c, c->a_hist); c->a_hist = nullptr;
  dev_free(c, c->aux_partial); c->aux_partial = nullptr;
  c->track = false;
  c->groups = 0; c->nodes_per_group = 0;
}

// Acquire a staging slot: returns host pointer and device pointer of the slot.
int stage_acquire(swarm_ctx* c, size_t bytes, void** host, void** dev, int* slot) {
  if (bytes > c->stage_slot_bytes) return SWARM_EINVAL;
  const int sidx = c->stage_next;
  c->stage_next = (sidx + 1) % kStageSlots;
  SW_CUDA(c, cudaEventSynchronize(c->stage_event[sidx]));
  *host = (char*)c->stage_host + (size_t)sidx * c->stage_slot_bytes;
  *dev = (char*)c->stage_dev + (size_t)sidx * c->stage_slot_bytes;
  *slot = sidx;
  return SWARM_OK;
}
int stage_commit(swarm_ctx* c, int slot, size_t bytes) {
  void* host = (char*)c->stage_host + (size_t)slot * c->stage_slot_bytes;
  void* dev = (char*)c->stage_dev + (size_t)slot * c->stage_slot_bytes;
  SW_CUDA(c, cudaMemcpyAsync(dev, host, bytes, cudaMemcpyHostToDevice, c->stream));
  return SWARM_OK;
}
int stage_release(swarm_ctx* c, int slot) {
  SW_CUDA(c, cudaEventRecord(c->stage_event[slot], c->stream));
  return SWARM_OK;
}

// Device buffers that a configuration needs beyond the ones every context has.
int alloc_objective(swarm_ctx* c, const swarm_config& cfg) {
  const int n = c->n;
  const size_t row_bytes = (size_t)c->pitch * sizeof(float);
  if (cfg.nonblocking) {
    c->B = (float*)dev_alloc(c, (size_t)n * row_bytes);
    if (!c->B) return SWARM_ENOMEM;
  }
  if (cfg.nonblocking == 2) {
    c->own = (uint8_t*)dev_alloc(c, (size_t)n * c->nblk * 2 * kBlockCoords);
    c->oexps = (int8_t*)dev_alloc(c, (size_t)n * c->nblk);
    if (!c->own || !c->oexps) return SWARM_ENOMEM;
  }
  if (cfg.objective == SWARM_OBJ_LSQ || cfg.objective == SWARM_OBJ_LOGISTIC) {
    c->groups = cfg.lsq_groups > 0 ? cfg.lsq_groups : n;
    c->nodes_per_group = n / c->groups;
    const size_t esz = cfg.lsq_dtype == SWARM_BF16 ? 2 : 4;
    c->A = dev_alloc(c, (size_t)c->groups * cfg.lsq_m * c->pitch * esz);
    c->bvec = (float*)dev_alloc(c, (size_t)n * cfg.lsq_m * sizeof(float));
    c->xstar = (float*)dev_alloc(c, row_bytes);
    c->lsq_partial = (float*)dev_alloc(c, (size_t)n * cfg.lsq_batch * lsq_chunks(c->d) * sizeof(float));
    c->convert_tmp = (float*)dev_alloc(c, row_bytes);
    if (!c->A || !c->bvec || !c->xstar || !c->lsq_partial || !c->convert_tmp) return SWARM_ENOMEM;
    const bool tensor_cores = cfg.lsq_dtype == SWARM_BF16 && cfg.lsq_batch <= 64;
    if (tensor_cores) {
      c->tc_partial = (float*)dev_alloc(c, lsq_tc_partial_bytes(c->pitch, n));
      c->tc_resid = dev_alloc(c, lsq_tc_resid_bytes(n));
      if (!c->tc_partial || !c->tc_resid) return SWARM_ENOMEM;
    }
    // Gram matrices of the data, for the kernels that take several local steps per pass
    if (tensor_cores || lsq_small_steps_in_pairs(c->pitch, cfg.lsq_batch)) {
      const size_t gram_bytes = lsq_tc_gram_bytes(c->groups, cfg.lsq_m);
      if (gram_bytes) {
        c->gram = (float*)dev_alloc(c, gram_bytes);
        if (!c->gram) return SWARM_ENOMEM;
      }
    }
  }
  return SWARM_OK;
}

swarm_config default_config() {
  swarm_config def{};
  def.objective = SWARM_OBJ_NONE; def.nonblocking = 0; def.init_std = 0.1f;
  return def;
}

// Rebuilds the whole state from the seed under `wanted`. The old objective buffers are released first (a data
// matrix can be most of the device's memory, so old and new are never held together). When an allocation
// fails, what was allocated is released again and the context is rebuilt under the default configuration (no
// objective, no snapshots: what swarm_init leaves, which needs no further memory), so that it never holds a
// configuration whose buffers are missing; the call then returns SWARM_ENOMEM.
int apply_config(swarm_ctx* c, const swarm_config& wanted) {
  free_objective(c);
  swarm_config cfg = wanted;
  int result = alloc_objective(c, cfg);
  if (result != SWARM_OK) {
    free_objective(c);
    cfg = default_config();
  }
  c->cfg = cfg;
  const int n = c->n;
  const size_t row_bytes = (size_t)c->pitch * sizeof(float);
  int nl = 0;
  StoreView s = view_of(c);
  SW_CUDA(c, cudaMemsetAsync(c->X, 0, (size_t)n * row_bytes, c->stream));
  SW_CUDA(c, cudaMemsetAsync(c->codes, 0, (size_t)n * c->nblk * kBlockCoords, c->stream));
  SW_CUDA(c, cudaMemsetAsync(c->exps, 0, (size_t)n * c->nblk, c->stream));
  SW_CUDA(c, cudaMemsetAsync(c->kernel_status, 0, sizeof(int), c->stream));
  if (c->tc_resid) SW_CUDA(c, cudaMemsetAsync(c->tc_resid, 0, lsq_tc_resid_bytes(n), c->stream));   // its ticket counters
  c->status_pending = false;
  c->poisoned = false;
  if (c->own) {
    SW_CUDA(c, cudaMemsetAsync(c->own, 0, (size_t)n * c->nblk * 2 * kBlockCoords, c->stream));
    SW_CUDA(c, cudaMemsetAsync(c->oexps, 0, (size_t)n * c->nblk, c->stream));
  }
  SW_CUDA(c, launch_node_scalars(c->scalars, n, cfg.offset_std, cfg.drift_std, s.key0, s.key1, c->stream, &nl));
  SW_CUDA(c, launch_init_models(s, c->scalars, cfg.init_std, c->stream, &nl));
  if (c->B) SW_CUDA(c, cudaMemcpyAsync(c->B, c->X, (size_t)n * row_bytes, cudaMemcpyDeviceToDevice, c->stream));
  if (cfg.objective == SWARM_OBJ_LSQ || cfg.objective == SWARM_OBJ_LOGISTIC) {
    LsqView l = lsq_of(c);
    SW_CUDA(c, launch_lsq_data(s, l, c->A, c->xstar, c->bvec, c->scalars, cfg.lsq_noise_std, c->stream, &nl));
    SW_CUDA(c, launch_lsq_gram(c->A, cfg.lsq_dtype, cfg.lsq_m, c->pitch, 0, c->groups, c->gram, c->kernel_status,
                               c->wait_limit, c->stream, &nl));
    if (c->gram && cfg.lsq_dtype == SWARM_BF16) c->status_pending = true;   // its waits are bounded too
  }
  c->launches += nl;
  std::fill(c->w.begin(), c->w.end(), 0u);
  std::fill(c->ls.begin(), c->ls.end(), 0u);
  std::fill(c->pbits.begin(), c->pbits.end(), 0);
  std::fill(c->wo.begin(), c->wo.end(), 0u);
  std::fill(c->tau.begin(), c->tau.end(), 0u);
  c->launch_ctr = 0;
  c->b_stale = 0;
  c->p_mode = 0;
  c->own_prefix = 16;
  return result;
}

int validate_config(const swarm_ctx* c, const swarm_config* cfg) {
  if (cfg->objective < SWARM_OBJ_NONE || cfg->objective > SWARM_OBJ_LOGISTIC) return SWARM_EINVAL;
  if (cfg->nonblocking < 0 || cfg->nonblocking > 2) return SWARM_EINVAL;
  if (!(cfg->init_std >= 0.0f) || !(cfg->offset_std >= 0.0f) || !(cfg->grad_std >= 0.0f) || !(cfg->drift_std >= 0.0f))
    return SWARM_EINVAL;
  if (cfg->objective == SWARM_OBJ_LSQ || cfg->objective == SWARM_OBJ_LOGISTIC) {
    if (cfg->lsq_m < 1 || cfg->lsq_batch < 1 || cfg->lsq_batch > 256) return SWARM_EINVAL;
    if (cfg->lsq_dtype != SWARM_F32 && cfg->lsq_dtype != SWARM_BF16) return SWARM_EINVAL;
    if (cfg->lsq_groups < 0 || cfg->lsq_groups > c->n) return SWARM_EINVAL;
    if (cfg->lsq_groups > 0 && (c->n % cfg->lsq_groups) != 0) return SWARM_EINVAL;
    const int npg = cfg->lsq_groups > 0 ? c->n / cfg->lsq_groups : 1;
    if (npg > 256) return SWARM_EINVAL;
    if (!(cfg->lsq_noise_std >= 0.0f)) return SWARM_EINVAL;
  }
  return SWARM_OK;
}

int validate_pairs(const swarm_ctx* c, const swarm_pair* pairs, int npairs) {
  std::vector<uint8_t> used((size_t)c->n, 0);
  for (int p = 0; p < npairs; ++p) {
    const int a = pairs[p].a, b = pairs[p].b;
    if (a < 0 || a >= c->n || b < 0 || b >= c->n) return SWARM_ERANGE;
  }
  for (int p = 0; p < npairs; ++p) {
    const int a = pairs[p].a, b = pairs[p].b;
    if (a == b || used[a] || used[b]) return SWARM_EPAIR;
    const int32_t* row = c->adj.data() + (size_t)a * c->degree;
    if (std::find(row, row + c->degree, b) == row + c->degree) return SWARM_EPAIR;
    used[a] = used[b] = 1;
  }
  return SWARM_OK;
}

int do_publish(swarm_ctx* c, int bits) {
  const size_t row_bytes = (size_t)c->pitch * sizeof(float);
  if (c->b_stale) {
    SW_CUDA(c, cudaMemcpyAsync(c->B, c->X, (size_t)c->n * row_bytes, cudaMemcpyDeviceToDevice, c->stream));
    c->b_stale = 0;
  }
  void *host, *dev;
  int slot;
  int rc = stage_acquire(c, (size_t)c->n * sizeof(uint32_t), &host, &dev, &slot);
  if (rc != SWARM_OK) return rc;
  std::memcpy(host, c->w.data(), (size_t)c->n * sizeof(uint32_t));
  rc = stage_commit(c, slot, (size_t)c->n * sizeof(uint32_t));
  if (rc != SWARM_OK) return rc;
  int nl = 0;
  SW_CUDA(c, launch_publish(view_of(c), (const uint32_t*)dev, bits, c->stream, &nl));
  c->launches += nl;
  rc = stage_release(c, slot);
  if (rc != SWARM_OK) return rc;
  for (int i = 0; i < c->n; ++i) { c->w[i] += 1; c->pbits[i] = bits; }
  c->p_mode = 1;
  return SWARM_OK;
}

int do_register_publish(swarm_ctx* c, int bits) {
  const size_t row_bytes = (size_t)c->pitch * sizeof(float);
  if (c->b_stale) {
    SW_CUDA(c, cudaMemcpyAsync(c->B, c->X, (size_t)c->n * row_bytes, cudaMemcpyDeviceToDevice, c->stream));
    c->b_stale = 0;
  }
  void *host, *dev;
  int slot;
  const size_t bytes = (size_t)2 * c->n * sizeof(uint32_t);
  int rc = stage_acquire(c, bytes, &host, &dev, &slot);
  if (rc != SWARM_OK) return rc;
  std::memcpy(host, c->w.data(), bytes / 2);
  std::memcpy((char*)host + bytes / 2, c->wo.data(), bytes / 2);
  rc = stage_commit(c, slot, bytes);
  if (rc != SWARM_OK) return rc;
  int nl = 0;
  SW_CUDA(c, launch_register_publish(view_of(c), (const uint32_t*)dev, bits, c->stream, &nl));
  c->launches += nl;
  rc = stage_release(c, slot);
  if (rc != SWARM_OK) return rc;
  for (int i = 0; i < c->n; ++i) { c->w[i] += 1; c->wo[i] += 1; c->pbits[i] = bits; }
  c->p_mode = 2;
  return SWARM_OK;
}

// The listed nodes initiated just now: store the current mean model as their record and their
// snapshot's squared distance to it (lists longer than the inline capacity go in slices).
int record_initiations(swarm_ctx* c, const int32_t* nodes, int count) {
  int nl = 0;
  for (int base = 0; base < count; base += kInlineNodes) {
    NodeList list{};
    list.n = std::min(kInlineNodes, count - base);
    for (int t = 0; t < list.n; ++t) { list.inl[t].node = nodes[base + t]; list.inl[t].event = 0; }
    SW_CUDA(c, launch_staleness_record(view_of(c), c->mu_hist, list, c->aux_partial, c->a_hist, c->stream, &nl));
  }
  c->launches += nl;
  return SWARM_OK;
}

bool buffers_need_publish(const swarm_ctx* c, int bits, int mode) {
  if (c->b_stale != 0 || c->p_mode != mode) return true;
  for (int i = 0; i < c->n; ++i)
    if (c->pbits[i] != bits) return true;
  return false;
}

}  // namespace

// =============================================================================================
extern "C" {

int swarm_set_allocator(swarm_alloc_fn alloc_fn, swarm_free_fn free_fn, void* user) {
  if ((alloc_fn == nullptr) != (free_fn == nullptr)) return SWARM_EINVAL;
  std::lock_guard<std::mutex> lock(g_alloc_mutex);
  g_alloc = alloc_fn; g_free = free_fn; g_alloc_user = user;
  return SWARM_OK;
}

const char* swarm_strerror(int code) {
  switch (code) {
    case SWARM_OK: return "ok";
    case SWARM_EINVAL: return "invalid argument";
    case SWARM_ERANGE: return "node id out of range";
    case SWARM_EPAIR: return "pairs not disjoint, self-pair, or not an edge of the graph";
    case SWARM_ESTATE: return "call not valid in the current configuration";
    case SWARM_ENOMEM: return "out of memory";
    case SWARM_ECUDA: return "CUDA error (see swarm_last_cuda_error)";
    default: return "unknown error";
  }
}

void swarm_destroy(swarm_ctx* c) {
  if (!c) return;
  DeviceGuard guard(c->device);
  cudaStreamSynchronize(c->stream);
  free_objective(c);
  dev_free(c, c->X); dev_free(c, c->codes); dev_free(c, c->exps); dev_free(c, c->adj_dev);
  dev_free(c, c->scalars); dev_free(c, c->pot_partial); dev_free(c, c->pot_out);
  dev_free(c, c->pairs_out_dev); dev_free(c, c->used_dev); dev_free(c, c->stage_dev); dev_free(c, c->kernel_status);
  dev_free(c, c->rq_dev);
  if (c->rq_host) cudaFreeHost(c->rq_host);
  if (c->kernel_status_host) cudaFreeHost(c->kernel_status_host);
  if (c->stage_host) cudaFreeHost(c->stage_host);
  if (c->pot_host) cudaFreeHost(c->pot_host);
  if (c->pairs_out_host) cudaFreeHost(c->pairs_out_host);
  for (auto& ev : c->stage_event) if (ev) cudaEventDestroy(ev);
  delete c;
}

int swarm_init(swarm_ctx** out, int32_t n, int64_t d, swarm_topology topo, uint64_t seed) {
  if (!out) return SWARM_EINVAL;
  *out = nullptr;
  if (n < 2 || d < 1 || d > ((int64_t)1 << 34)) return SWARM_EINVAL;
  swarm_ctx* c = new (std::nothrow) swarm_ctx();
  if (!c) return SWARM_ENOMEM;
  if (cudaGetDevice(&c->device) != cudaSuccess) { c->last_cuda = (int)cudaGetLastError(); delete c; return SWARM_ECUDA; }
  c->n = n; c->d = d; c->seed = seed;
  c->nblk = (d + kBlockCoords - 1) / kBlockCoords;
  c->pitch = c->nblk * kBlockCoords;
  c->topo_kind = topo.kind; c->degree = topo.degree;
  {
    std::lock_guard<std::mutex> lock(g_alloc_mutex);
    c->custom_alloc = g_alloc != nullptr;
    c->alloc_fn = g_alloc; c->free_fn = g_free; c->alloc_user = g_alloc_user;
  }
  c->wait_limit = lsq_tc_default_wait_limit();
  if (!build_graph(c)) { delete c; return SWARM_EINVAL; }
  c->w.assign(n, 0); c->ls.assign(n, 0); c->pbits.assign(n, 0); c->wo.assign(n, 0); c->tau.assign(n, 0); c->touched.assign(n, 0);

  const size_t row_bytes = (size_t)c->pitch * sizeof(float);
  const size_t max_pairs = (size_t)n / 2;
  c->stage_slot_bytes = std::max({max_pairs * sizeof(PairDesc), (size_t)n * sizeof(NodeDesc), (size_t)2 * n * sizeof(uint32_t),
                                  (size_t)n * sizeof(LsqUnit)});
  c->stage_slot_bytes = (c->stage_slot_bytes + 255) / 256 * 256;
  c->X = (float*)dev_alloc(c, (size_t)n * row_bytes);
  c->codes = (uint8_t*)dev_alloc(c, (size_t)n * c->nblk * kBlockCoords);
  c->exps = (int8_t*)dev_alloc(c, (size_t)n * c->nblk);
  c->adj_dev = (int32_t*)dev_alloc(c, c->adj.size() * sizeof(int32_t));
  c->scalars = (float*)dev_alloc(c, (size_t)n * 3 * sizeof(float));
  c->pot_partial = (double*)dev_alloc(c, (size_t)potential_partials(d) * sizeof(double));
  c->pot_out = (double*)dev_alloc(c, 5 * sizeof(double));
  c->pairs_out_dev = (int32_t*)dev_alloc(c, (2 * max_pairs + 1) * sizeof(int32_t));
  c->used_dev = (uint8_t*)dev_alloc(c, (size_t)n);
  c->kernel_status = (int*)dev_alloc(c, sizeof(int));
  c->stage_dev = dev_alloc(c, c->stage_slot_bytes * kStageSlots);
  c->rq_dev = (uint8_t*)dev_alloc(c, kReadQueueBytes);
  bool ok = c->X && c->codes && c->exps && c->adj_dev && c->scalars && c->pot_partial && c->pot_out &&
            c->pairs_out_dev && c->used_dev && c->stage_dev && c->kernel_status && c->rq_dev;
  ok = ok && cudaMallocHost((void**)&c->rq_host, kReadQueueBytes) == cudaSuccess;
  ok = ok && cudaMallocHost(&c->stage_host, c->stage_slot_bytes * kStageSlots) == cudaSuccess;
  ok = ok && cudaMallocHost((void**)&c->pot_host, 4 * sizeof(double)) == cudaSuccess;
  ok = ok && cudaMemsetAsync(c->pot_out, 0, 5 * sizeof(double), c->stream) == cudaSuccess;
  if (ok) {   // the potential kernel writes its result straight to the pinned host word when that is mapped
    void* mapped = nullptr;
    if (cudaHostGetDevicePointer(&mapped, c->pot_host, 0) == cudaSuccess) c->pot_host_dev = (double*)mapped;
    else cudaGetLastError();
  }
  ok = ok && cudaMallocHost((void**)&c->kernel_status_host, sizeof(int)) == cudaSuccess;
  ok = ok && cudaMemsetAsync(c->kernel_status, 0, sizeof(int), c->stream) == cudaSuccess;
  ok = ok && cudaMallocHost((void**)&c->pairs_out_host, (2 * max_pairs + 1) * sizeof(int32_t)) == cudaSuccess;
  for (int i = 0; ok && i < kStageSlots; ++i)
    ok = cudaEventCreateWithFlags(&c->stage_event[i], cudaEventDisableTiming) == cudaSuccess;
  if (!ok) { cudaGetLastError(); swarm_destroy(c); return SWARM_ENOMEM; }

  cudaError_t e = cudaMemcpyAsync(c->adj_dev, c->adj.data(), c->adj.size() * sizeof(int32_t), cudaMemcpyHostToDevice,
                                  c->stream);
  if (e != cudaSuccess) { swarm_destroy(c); return SWARM_ECUDA; }
  int rc = apply_config(c, default_config());
  if (rc == SWARM_OK && cudaStreamSynchronize(c->stream) != cudaSuccess) rc = SWARM_ECUDA;
  if (rc != SWARM_OK) { swarm_destroy(c); return rc; }
  *out = c;
  return SWARM_OK;
}

int swarm_configure(swarm_ctx* c, const swarm_config* cfg) {
  if (!c || !cfg) return SWARM_EINVAL;
  int rc = validate_config(c, cfg);
  if (rc != SWARM_OK) return rc;
  DeviceGuard guard(c->device);
  rc = ctx_sync(c, false);          // a context whose bounded wait expired is rebuilt here, not refused
  if (rc != SWARM_OK) return rc;
  rc = apply_config(c, *cfg);
  SW_SYNC(c);
  return rc;
}

int swarm_set_stream(swarm_ctx* c, void* cuda_stream) {
  if (!c) return SWARM_EINVAL;
  DeviceGuard guard(c->device);
  SW_SYNC(c);
  c->stream = (cudaStream_t)cuda_stream;
  return SWARM_OK;
}

int swarm_sync(swarm_ctx* c) {
  if (!c) return SWARM_EINVAL;
  DeviceGuard guard(c->device);
  SW_SYNC(c);      // also reports a bounded device wait that expired
  return SWARM_OK;
}

int swarm_set_wait_limit(swarm_ctx* c, int64_t polls) {
  if (!c || polls > (int64_t)UINT32_MAX) return SWARM_EINVAL;
  c->wait_limit = polls < 0 ? lsq_tc_default_wait_limit() : (uint32_t)polls;
  return SWARM_OK;
}

int64_t swarm_kernel_launches(swarm_ctx* c) { return c ? c->launches : 0; }
int swarm_last_cuda_error(swarm_ctx* c) { return c ? c->last_cuda : 0; }

int swarm_model_ptr(swarm_ctx* c, float** x_dev, int64_t* pitch) {
  if (!c || !x_dev || !pitch) return SWARM_EINVAL;
  *x_dev = c->X; *pitch = c->pitch;
  return SWARM_OK;
}

int swarm_local_steps(swarm_ctx* c, const int32_t* node_ids, int32_t count, int32_t H, float lr) {
  if (!c || count < 0 || H < 0 || (count > 0 && !node_ids)) return SWARM_EINVAL;
  if (c->cfg.objective == SWARM_OBJ_NONE) return SWARM_ESTATE;
  if (count > c->n) return SWARM_EINVAL;
  {
    std::vector<uint8_t> seen((size_t)c->n, 0);
    for (int t = 0; t < count; ++t)
      if (node_ids[t] < 0 || node_ids[t] >= c->n) return SWARM_ERANGE;
    for (int t = 0; t < count; ++t) {
      if (seen[node_ids[t]]) return SWARM_EINVAL;
      seen[node_ids[t]] = 1;
    }
  }
  if (count == 0 || H == 0) return SWARM_OK;
  DeviceGuard guard(c->device);
  void *host, *dev;
  int slot;
  if (c->cfg.objective >= SWARM_OBJ_LSQ && c->tc_partial) {
    // bf16 data: batch the listed nodes that share a data matrix and a step counter (hence the
    // minibatch) into units of up to 16 for the tensor-core kernels
    std::vector<LsqUnit> units;
    std::vector<int> order(node_ids, node_ids + count);
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
      const int ga = a / c->nodes_per_group, gb = b / c->nodes_per_group;
      return ga != gb ? ga < gb : c->ls[a] < c->ls[b];
    });
    for (int node : order) {
      const int g = node / c->nodes_per_group;
      if (units.empty() || units.back().group != g || units.back().event != c->ls[node] || units.back().count == 16) {
        LsqUnit u{};
        u.group = g; u.event = c->ls[node]; u.count = 0;
        units.push_back(u);
      }
      units.back().nodes[units.back().count++] = node;
    }
    const size_t bytes = units.size() * sizeof(LsqUnit);
    int rc = stage_acquire(c, bytes, &host, &dev, &slot);
    if (rc != SWARM_OK) return rc;
    std::memcpy(host, units.data(), bytes);
    rc = stage_commit(c, slot, bytes);
    if (rc != SWARM_OK) return rc;
    int nl = 0;
    SW_CUDA(c, launch_local_lsq_tc(view_of(c), lsq_of(c), (const LsqUnit*)dev, (int)units.size(), c->n, H, lr, c->tc_partial,
                                   c->tc_resid, c->kernel_status, c->wait_limit, c->stream, &nl));
    c->status_pending = true;
    c->launches += nl;
    rc = stage_release(c, slot);
    if (rc != SWARM_OK) return rc;
    for (int t = 0; t < count; ++t) c->ls[node_ids[t]] += (uint32_t)H;
    return SWARM_OK;
  }
  NodeList list{};
  list.n = count;
  int rc = SWARM_OK;
  slot = -1;
  NodeDesc* nd = list.inl;
  if (count > kInlineNodes) {
    rc = stage_acquire(c, (size_t)count * sizeof(NodeDesc), &host, &dev, &slot);
    if (rc != SWARM_OK) return rc;
    nd = (NodeDesc*)host;
    list.ptr = (const NodeDesc*)dev;
  }
  for (int t = 0; t < count; ++t) { nd[t].node = node_ids[t]; nd[t].event = c->ls[node_ids[t]]; }
  if (slot >= 0) {
    rc = stage_commit(c, slot, (size_t)count * sizeof(NodeDesc));
    if (rc != SWARM_OK) return rc;
  }
  int nl = 0;
  const StoreView s = view_of(c);
  if (c->cfg.objective == SWARM_OBJ_SYNTH) {
    SW_CUDA(c, launch_local_synth(s, list, count, H, lr, c->cfg.grad_std, c->scalars, c->stream, &nl));
  } else {
    SW_CUDA(c, launch_local_lsq(s, lsq_of(c), list, count, H, lr, c->lsq_partial, c->stream, &nl));
  }
  c->launches += nl;
  if (slot >= 0) {
    rc = stage_release(c, slot);
    if (rc != SWARM_OK) return rc;
  }
  for (int t = 0; t < count; ++t) c->ls[node_ids[t]] += (uint32_t)H;
  return SWARM_OK;
}

int swarm_local_steps_geometric(swarm_ctx* c, const int32_t* node_ids, int32_t count, int32_t mean_H, float lr,
                                int32_t* out_steps) {
  if (!c || count < 0 || mean_H < 1 || (count > 0 && !node_ids)) return SWARM_EINVAL;
  if (c->cfg.objective == SWARM_OBJ_NONE) return SWARM_ESTATE;
  if (count > c->n) return SWARM_EINVAL;
  {
    std::vector<uint8_t> seen((size_t)c->n, 0);
    for (int t = 0; t < count; ++t)
      if (node_ids[t] < 0 || node_ids[t] >= c->n) return SWARM_ERANGE;
    for (int t = 0; t < count; ++t) {
      if (seen[node_ids[t]]) return SWARM_EINVAL;
      seen[node_ids[t]] = 1;
    }
  }
  // step counts: first success among Bernoulli(1/mean_H) trials, one generator word per trial
  const uint32_t key0 = (uint32_t)c->seed, key1 = (uint32_t)(c->seed >> 32);
  std::vector<int32_t> steps((size_t)count);
  int32_t max_steps = 0;
  for (int t = 0; t < count; ++t) {
    const uint32_t node = (uint32_t)node_ids[t], event = c->ls[node_ids[t]];
    int32_t h = 1024;
    for (int trial = 0; trial < 1024; ++trial) {
      const uint4 w = philox4x32_10((uint32_t)(trial >> 2), node, event, kStreamStepCount, key0, key1);
      const uint32_t word = (trial & 3) == 0 ? w.x : (trial & 3) == 1 ? w.y : (trial & 3) == 2 ? w.z : w.w;
      if (uniform_int(word, (uint32_t)mean_H) == 0) { h = trial + 1; break; }
    }
    steps[t] = h;
    max_steps = std::max(max_steps, h);
  }
  // one launch sequence per distinct count (nodes with equal counts travel together)
  std::vector<int32_t> bucket;
  for (int32_t h = 1; h <= max_steps; ++h) {
    bucket.clear();
    for (int t = 0; t < count; ++t)
      if (steps[t] == h) bucket.push_back(node_ids[t]);
    if (bucket.empty()) continue;
    const int rc = swarm_local_steps(c, bucket.data(), (int32_t)bucket.size(), h, lr);
    if (rc != SWARM_OK) return rc;
  }
  if (out_steps) std::copy(steps.begin(), steps.end(), out_steps);
  return SWARM_OK;
}

// One interaction launch; fused_H > 0 runs that many synthetic-gradient local steps of the initiators (and of
// the responders when `responders` is set) inside the interaction kernel first.
static int interact_impl(swarm_ctx* c, const swarm_pair* pairs, int32_t npairs, int32_t bits, int32_t mode,
                         int32_t fused_H, float lr, int32_t responders, const int32_t* prefixes = nullptr) {
  if (!c || npairs < 0 || (npairs > 0 && !pairs)) return SWARM_EINVAL;
  if (mode != SWARM_BLOCKING && mode != SWARM_NONBLOCKING && mode != SWARM_REGISTERS) return SWARM_EINVAL;
  if (prefixes) {
    if (mode != SWARM_REGISTERS) return SWARM_EINVAL;
    for (int p = 0; p < npairs; ++p)
      if (prefixes[p] != 8 && prefixes[p] != 16) return SWARM_EINVAL;
  }
  const bool quant = bits >= 2 && bits <= 8;
  if (!(quant || (bits == 32 && mode == SWARM_BLOCKING))) return SWARM_EINVAL;
  if (mode == SWARM_NONBLOCKING && !c->cfg.nonblocking) return SWARM_ESTATE;
  if (mode == SWARM_REGISTERS && c->cfg.nonblocking != 2) return SWARM_ESTATE;
  if (mode == SWARM_BLOCKING && c->track) return SWARM_ESTATE;   // no outdated model to track
  if (npairs > c->n / 2) return SWARM_EPAIR;
  int rc = validate_pairs(c, pairs, npairs);
  if (rc != SWARM_OK) return rc;
  DeviceGuard guard(c->device);
  if (mode == SWARM_NONBLOCKING && buffers_need_publish(c, bits, 1)) {
    rc = do_publish(c, bits);
    if (rc != SWARM_OK) return rc;
  }
  if (mode == SWARM_REGISTERS && buffers_need_publish(c, bits, 2)) {
    rc = do_register_publish(c, bits);
    if (rc != SWARM_OK) return rc;
  }
  if (npairs == 0) return SWARM_OK;
  void *host, *dev;
  int slot = -1;
  PairList list{};
  list.n = npairs;
  PairDesc* pd = list.inl;
  if (npairs > kInlinePairs) {
    rc = stage_acquire(c, (size_t)npairs * sizeof(PairDesc), &host, &dev, &slot);
    if (rc != SWARM_OK) return rc;
    pd = (PairDesc*)host;
    list.ptr = (const PairDesc*)dev;
  }
  // The kernel may take the pairs of a launch in any order (they are disjoint; clocks and counters follow the
  // caller's list order on the host). It walks its descriptor list from one end, alternating the end from launch
  // to launch, and the descriptors are laid out so that the walk meets the pairs whose rows the previous launches
  // touched last first: a good part of those rows is still in L2.
  const bool backwards = c->sweep_backwards;
  c->sweep_backwards = !c->sweep_backwards;
  std::vector<int> walk((size_t)npairs);
  for (int p = 0; p < npairs; ++p) walk[p] = p;
  std::stable_sort(walk.begin(), walk.end(), [&](int x, int y) {
    return std::max(c->touched[pairs[x].a], c->touched[pairs[x].b]) > std::max(c->touched[pairs[y].a], c->touched[pairs[y].b]);
  });
  for (int t = 0; t < npairs; ++t) {
    const int p = walk[t], at = backwards ? npairs - 1 - t : t;
    pd[at].a = pairs[p].a; pd[at].b = pairs[p].b;
    pd[at].wa = c->w[pairs[p].a]; pd[at].wb = c->w[pairs[p].b];
    pd[at].woa = c->wo[pairs[p].a]; pd[at].prefix = (uint32_t)(prefixes ? prefixes[p] : c->own_prefix);
    pd[at].lsa = c->ls[pairs[p].a]; pd[at].lsb = c->ls[pairs[p].b];
    c->touched[pairs[p].a] = c->touched[pairs[p].b] = ++c->touch_seq;
  }
  FusedSteps fs{};
  fs.H = fused_H; fs.responders = responders ? 1 : 0; fs.lr = lr; fs.grad_std = c->cfg.grad_std; fs.scalars = c->scalars;
  if (slot >= 0) {
    rc = stage_commit(c, slot, (size_t)npairs * sizeof(PairDesc));
    if (rc != SWARM_OK) return rc;
  }
  int nl = 0;
  StoreView sv = view_of(c);
  sv.backwards = backwards ? 1u : 0u;
  if (mode == SWARM_BLOCKING) SW_CUDA(c, launch_interact_blocking(sv, list, npairs, bits, fs, c->stream, &nl));
  else if (mode == SWARM_NONBLOCKING) SW_CUDA(c, launch_interact_nonblocking(sv, list, npairs, bits, fs, c->stream, &nl));
  else SW_CUDA(c, launch_interact_registers(sv, list, npairs, bits, fs, c->stream, &nl));
  for (int p = 0; p < npairs && fused_H > 0; ++p) {
    c->ls[pairs[p].a] += (uint32_t)fused_H;
    if (responders) c->ls[pairs[p].b] += (uint32_t)fused_H;
  }
  c->launches += nl;
  if (slot >= 0) {
    rc = stage_release(c, slot);
    if (rc != SWARM_OK) return rc;
  }
  if (bits != 32) {
    for (int p = 0; p < npairs; ++p) {
      c->w[pairs[p].a] += 1; c->w[pairs[p].b] += 1;
      if (mode == SWARM_BLOCKING) { c->pbits[pairs[p].a] = bits; c->pbits[pairs[p].b] = bits; }
    }
  }
  if (mode == SWARM_REGISTERS)
    for (int p = 0; p < npairs; ++p) c->wo[pairs[p].a] += 1;
  if (mode == SWARM_BLOCKING && bits != 32) c->p_mode = 0;      // buffers now follow the blocking convention
  if (mode == SWARM_BLOCKING && c->cfg.nonblocking) c->b_stale = 1;
  // staleness clocks: interactions in list order, each resets its initiator and ages everybody else
  for (int p = 0; p < npairs; ++p) {
    for (int i = 0; i < c->n; ++i) c->tau[i] += 1;
    c->tau[pairs[p].a] = 0;
  }
  if (c->track) {
    std::vector<int32_t> init((size_t)npairs);
    for (int p = 0; p < npairs; ++p) init[p] = pairs[p].a;
    rc = record_initiations(c, init.data(), npairs);
    if (rc != SWARM_OK) return rc;
  }
  return SWARM_OK;
}

int swarm_interact(swarm_ctx* c, const swarm_pair* pairs, int32_t npairs, int32_t bits, int32_t mode) {
  return interact_impl(c, pairs, npairs, bits, mode, 0, 0.0f, 0);
}

int swarm_interact_prefixed(swarm_ctx* c, const swarm_pair* pairs, const int32_t* prefixes, int32_t npairs,
                            int32_t bits) {
  if (npairs > 0 && !prefixes) return SWARM_EINVAL;
  return interact_impl(c, pairs, npairs, bits, SWARM_REGISTERS, 0, 0.0f, 0, prefixes);
}

int swarm_step(swarm_ctx* c, const swarm_pair* pairs, int32_t npairs, int32_t H, float lr, int32_t bits, int32_t mode,
               int32_t step_responders) {
  if (!c || H < 0 || npairs < 0 || (npairs > 0 && !pairs)) return SWARM_EINVAL;
  if (H == 0) return interact_impl(c, pairs, npairs, bits, mode, 0, 0.0f, 0);
  if (c->cfg.objective == SWARM_OBJ_NONE) return SWARM_ESTATE;
  // Elementwise objective, blocking or single-buffer exchange: the steps run inside the interaction kernel. A
  // publish that the interaction triggers runs before the fused steps; that is the same as after them unless it
  // first refreshes stale snapshots from the models, so that one case takes the two-call route. So does the
  // two-register exchange, whose kernel is bound by instruction issue already (measured slower with the steps in it).
  if (c->cfg.objective == SWARM_OBJ_SYNTH && mode != SWARM_REGISTERS && !(mode != SWARM_BLOCKING && c->b_stale))
    return interact_impl(c, pairs, npairs, bits, mode, H, lr, step_responders);
  // objectives whose gradient couples all coordinates: the two calls in sequence, after the checks that
  // the interaction would make (so that a refused call leaves the models untouched)
  if (mode != SWARM_BLOCKING && mode != SWARM_NONBLOCKING && mode != SWARM_REGISTERS) return SWARM_EINVAL;
  if (!((bits >= 2 && bits <= 8) || (bits == 32 && mode == SWARM_BLOCKING))) return SWARM_EINVAL;
  if (mode == SWARM_NONBLOCKING && !c->cfg.nonblocking) return SWARM_ESTATE;
  if (mode == SWARM_REGISTERS && c->cfg.nonblocking != 2) return SWARM_ESTATE;
  if (mode == SWARM_BLOCKING && c->track) return SWARM_ESTATE;
  if (npairs > c->n / 2) return SWARM_EPAIR;
  int rc = validate_pairs(c, pairs, npairs);
  if (rc != SWARM_OK) return rc;
  std::vector<int32_t> nodes;
  nodes.reserve((size_t)npairs * 2);
  for (int p = 0; p < npairs; ++p) {
    nodes.push_back(pairs[p].a);
    if (step_responders) nodes.push_back(pairs[p].b);
  }
  rc = swarm_local_steps(c, nodes.data(), (int32_t)nodes.size(), H, lr);
  if (rc != SWARM_OK) return rc;
  return interact_impl(c, pairs, npairs, bits, mode, 0, 0.0f, 0);
}

int swarm_run_sequence(swarm_ctx* c, const swarm_pair* pairs, int32_t nsteps, int32_t H, float lr, int32_t bits,
                       int32_t step_responders) {
  if (!c || nsteps < 0 || H < 0 || (nsteps > 0 && !pairs)) return SWARM_EINVAL;
  if (!((bits >= 2 && bits <= 8) || bits == 32)) return SWARM_EINVAL;
  if (H > 0 && c->cfg.objective == SWARM_OBJ_NONE) return SWARM_ESTATE;
  if (c->track) return SWARM_ESTATE;
  for (int t = 0; t < nsteps; ++t) {
    const int rc = validate_pairs(c, pairs + t, 1);
    if (rc != SWARM_OK) return rc;
  }
  if (nsteps == 0) return SWARM_OK;
  DeviceGuard guard(c->device);
  const StoreView s = view_of(c);
  const LsqView l = lsq_of(c);
  const bool lsq = c->cfg.objective == SWARM_OBJ_LSQ || c->cfg.objective == SWARM_OBJ_LOGISTIC;
  if (!(lsq && bits != 32 && !c->tc_partial && lsq_sequence_supported(s, l))) {
    // no single-launch form for this configuration: the steps one by one
    for (int t = 0; t < nsteps; ++t) {
      const int rc = swarm_step(c, pairs + t, 1, H, lr, bits, SWARM_BLOCKING, step_responders);
      if (rc != SWARM_OK) return rc;
    }
    return SWARM_OK;
  }
  // One launch per slice of the sequence. The host knows how every counter evolves (each step advances the
  // two buffers' write counters by one and the stepping nodes' local-step counters by H), so the descriptors
  // of all steps are written up front and the kernel needs no counters of its own.
  const int max_slice = (int)std::max<size_t>(kInlinePairs, c->stage_slot_bytes / sizeof(PairDesc));
  for (int base = 0; base < nsteps; base += max_slice) {
    const int count = std::min(max_slice, nsteps - base);
    void *host = nullptr, *dev = nullptr;
    int slot = -1;
    PairList list{};
    list.n = count;
    PairDesc* pd = list.inl;
    if (count > kInlinePairs) {
      const int rc = stage_acquire(c, (size_t)count * sizeof(PairDesc), &host, &dev, &slot);
      if (rc != SWARM_OK) return rc;
      pd = (PairDesc*)host;
      list.ptr = (const PairDesc*)dev;
    }
    for (int t = 0; t < count; ++t) {
      const int a = pairs[base + t].a, b = pairs[base + t].b;
      pd[t].a = a; pd[t].b = b;
      pd[t].wa = c->w[a]; pd[t].wb = c->w[b]; pd[t].woa = c->wo[a];
      pd[t].lsa = c->ls[a]; pd[t].lsb = c->ls[b]; pd[t].prefix = 16;
      c->w[a] += 1; c->w[b] += 1;
      c->pbits[a] = bits; c->pbits[b] = bits;
      c->ls[a] += (uint32_t)H;
      if (step_responders) c->ls[b] += (uint32_t)H;
      for (int i = 0; i < c->n; ++i) c->tau[i] += 1;
      c->tau[a] = 0;
    }
    if (slot >= 0) {
      const int rc = stage_commit(c, slot, (size_t)count * sizeof(PairDesc));
      if (rc != SWARM_OK) return rc;
    }
    int nl = 0;
    SW_CUDA(c, launch_lsq_sequence(s, l, list, H, lr, bits, step_responders ? 1 : 0, c->stream, &nl));
    c->launches += nl;
    if (slot >= 0) {
      const int rc = stage_release(c, slot);
      if (rc != SWARM_OK) return rc;
    }
  }
  c->p_mode = 0;
  if (c->cfg.nonblocking) c->b_stale = 1;
  return SWARM_OK;
}

int swarm_track_staleness(swarm_ctx* c, int32_t enable) {
  if (!c) return SWARM_EINVAL;
  DeviceGuard guard(c->device);
  if (!enable) {
    SW_SYNC(c);
    dev_free(c, c->mu_hist); c->mu_hist = nullptr;
    dev_free(c, c->a_hist); c->a_hist = nullptr;
    dev_free(c, c->aux_partial); c->aux_partial = nullptr;
    c->track = false;
    return SWARM_OK;
  }
  if (!c->cfg.nonblocking || c->b_stale) return SWARM_ESTATE;
  if (!c->track) {
    const size_t parts = (size_t)potential_partials(c->d);
    c->mu_hist = (float*)dev_alloc(c, (size_t)c->n * c->pitch * sizeof(float));
    c->a_hist = (double*)dev_alloc(c, (size_t)c->n * sizeof(double));
    c->aux_partial = (double*)dev_alloc(c, (size_t)std::max(kInlineNodes, 2) * parts * sizeof(double));
    if (!c->mu_hist || !c->a_hist || !c->aux_partial) {
      dev_free(c, c->mu_hist); c->mu_hist = nullptr;
      dev_free(c, c->a_hist); c->a_hist = nullptr;
      dev_free(c, c->aux_partial); c->aux_partial = nullptr;
      return SWARM_ENOMEM;
    }
    SW_CUDA(c, cudaMemsetAsync(c->mu_hist, 0, (size_t)c->n * c->pitch * sizeof(float), c->stream));
    c->track = true;
  }
  std::vector<int32_t> all((size_t)c->n);
  for (int i = 0; i < c->n; ++i) all[i] = i;
  const int rc = record_initiations(c, all.data(), c->n);
  if (rc != SWARM_OK) return rc;
  std::fill(c->tau.begin(), c->tau.end(), 0u);
  return SWARM_OK;
}

int swarm_aux_potentials(swarm_ctx* c, double* out3) {
  if (!c || !out3) return SWARM_EINVAL;
  if (!c->track) return SWARM_ESTATE;
  DeviceGuard guard(c->device);
  int nl = 0;
  SW_CUDA(c, launch_aux_potentials(view_of(c), c->mu_hist, c->a_hist, c->aux_partial, c->pot_out, c->stream, &nl));
  c->launches += nl;
  SW_CUDA(c, cudaMemcpyAsync(c->pot_host, c->pot_out, 3 * sizeof(double), cudaMemcpyDeviceToHost, c->stream));
  SW_SYNC(c);
  out3[0] = c->pot_host[0]; out3[1] = c->pot_host[1]; out3[2] = c->pot_host[2];
  return SWARM_OK;
}

int swarm_register_publish(swarm_ctx* c, int32_t bits) {
  if (!c || (bits < 2 || bits > 8)) return SWARM_EINVAL;
  if (c->cfg.nonblocking != 2) return SWARM_ESTATE;
  DeviceGuard guard(c->device);
  return do_register_publish(c, bits);
}

int swarm_set_own_prefix(swarm_ctx* c, int32_t bits) {
  if (!c || (bits != 8 && bits != 16)) return SWARM_EINVAL;
  if (c->cfg.nonblocking != 2) return SWARM_ESTATE;
  c->own_prefix = bits;
  return SWARM_OK;
}
int swarm_get_own_prefix(swarm_ctx* c, int32_t* bits) {
  if (!c || !bits) return SWARM_EINVAL;
  *bits = c->own_prefix;
  return SWARM_OK;
}

int swarm_get_buffer_mode(swarm_ctx* c, int32_t* mode) {
  if (!c || !mode) return SWARM_EINVAL;
  *mode = c->p_mode;
  return SWARM_OK;
}
int swarm_set_buffer_mode(swarm_ctx* c, int32_t mode) {
  if (!c || mode < 0 || mode > 2) return SWARM_EINVAL;
  c->p_mode = mode;
  return SWARM_OK;
}

int swarm_publish(swarm_ctx* c, int32_t bits) {
  if (!c || (bits < 2 || bits > 8)) return SWARM_EINVAL;
  if (!c->cfg.nonblocking) return SWARM_ESTATE;
  DeviceGuard guard(c->device);
  return do_publish(c, bits);
}

int swarm_mean_model(swarm_ctx* c, float* out_dev) {
  if (!c || !out_dev) return SWARM_EINVAL;
  DeviceGuard guard(c->device);
  int nl = 0;
  SW_CUDA(c, launch_mean_model(view_of(c), out_dev, c->stream, &nl));
  c->launches += nl;
  return SWARM_OK;
}

int swarm_potential(swarm_ctx* c, double* out_gamma) {
  if (!c || !out_gamma) return SWARM_EINVAL;
  DeviceGuard guard(c->device);
  int nl = 0;
  SW_CUDA(c, launch_potential(view_of(c), c->pot_partial, (unsigned int*)(c->pot_out + 4), c->pot_out, c->pot_host_dev,
                              c->stream, &nl));
  c->launches += nl;
  if (!c->pot_host_dev)
    SW_CUDA(c, cudaMemcpyAsync(c->pot_host, c->pot_out, sizeof(double), cudaMemcpyDeviceToHost, c->stream));
  SW_SYNC(c);
  *out_gamma = *c->pot_host;
  return SWARM_OK;
}

int swarm_sample_pairs(swarm_ctx* c, int32_t max_pairs, swarm_pair* out_pairs, int32_t* out_count) {
  if (!c || !out_pairs || !out_count || max_pairs < 1) return SWARM_EINVAL;
  DeviceGuard guard(c->device);
  const size_t max_slots = (size_t)(c->n / 2);
  int nl = 0;
  // the draw budget is 16 * max_pairs even when max_pairs exceeds n/2; acceptance stops at n/2 anyway
  SW_CUDA(c, launch_sample_pairs(c->adj_dev, c->n, c->degree, max_pairs, c->launch_ctr, (uint32_t)c->seed,
                                 (uint32_t)(c->seed >> 32), c->pairs_out_dev, c->pairs_out_dev + 2 * max_slots,
                                 c->used_dev, c->stream, &nl));
  c->launches += nl;
  SW_CUDA(c, cudaMemcpyAsync(c->pairs_out_host, c->pairs_out_dev, (2 * max_slots + 1) * sizeof(int32_t),
                             cudaMemcpyDeviceToHost, c->stream));
  SW_SYNC(c);
  const int count = c->pairs_out_host[2 * max_slots];
  for (int p = 0; p < count; ++p) { out_pairs[p].a = c->pairs_out_host[2 * p]; out_pairs[p].b = c->pairs_out_host[2 * p + 1]; }
  *out_count = count;
  c->launch_ctr += 1;
  return SWARM_OK;
}

int swarm_get_state(swarm_ctx* c, uint32_t* launch, int32_t* b_stale) {
  if (!c || !launch || !b_stale) return SWARM_EINVAL;
  *launch = c->launch_ctr; *b_stale = c->b_stale;
  return SWARM_OK;
}
int swarm_set_state(swarm_ctx* c, uint32_t launch, int32_t b_stale) {
  if (!c || (b_stale != 0 && b_stale != 1)) return SWARM_EINVAL;
  if (b_stale && !c->cfg.nonblocking) return SWARM_ESTATE;
  c->launch_ctr = launch; c->b_stale = b_stale;
  return SWARM_OK;
}

static int tensor_access(swarm_ctx* c, int32_t which, int32_t node, void* host, size_t bytes, bool write,
                         bool wait = true) {
  if (!c || !host) return SWARM_EINVAL;
  // rows that live in host mirrors or need a conversion pass have no asynchronous form
  if (!wait && (which == SWARM_T_ADJ || which == SWARM_T_COUNTERS || which == SWARM_T_CLOCKS || which == SWARM_T_A))
    return SWARM_EINVAL;
  const bool per_node = which != SWARM_T_XSTAR && which != SWARM_T_A && which != SWARM_T_GRAM;
  if (per_node && (node < 0 || node >= c->n)) return SWARM_ERANGE;
  DeviceGuard guard(c->device);
  const size_t d = (size_t)c->d;
  void* dev = nullptr;
  size_t want = 0;
  switch (which) {
    case SWARM_T_X: dev = c->X + (size_t)node * c->pitch; want = d * 4; break;
    case SWARM_T_B:
      if (!c->B) return SWARM_ESTATE;
      dev = c->B + (size_t)node * c->pitch; want = d * 4; break;
    case SWARM_T_CODES: dev = c->codes + (size_t)node * c->nblk * kBlockCoords; want = (size_t)c->nblk * kBlockCoords; break;
    case SWARM_T_EXPS: dev = c->exps + (size_t)node * c->nblk; want = (size_t)c->nblk; break;
    case SWARM_T_ADJ:
      if (write) return SWARM_EINVAL;
      if (bytes != (size_t)c->degree * 4) return SWARM_EINVAL;
      std::memcpy(host, c->adj.data() + (size_t)node * c->degree, bytes);
      return SWARM_OK;
    case SWARM_T_BVEC:
      if (!c->bvec) return SWARM_ESTATE;
      dev = c->bvec + (size_t)node * c->cfg.lsq_m; want = (size_t)c->cfg.lsq_m * 4; break;
    case SWARM_T_XSTAR:
      if (!c->xstar) return SWARM_ESTATE;
      dev = c->xstar; want = d * 4; break;
    case SWARM_T_SCALARS: dev = c->scalars + (size_t)node * 3; want = 12; break;
    case SWARM_T_OWN:
      if (!c->own) return SWARM_ESTATE;
      dev = c->own + (size_t)node * c->nblk * 2 * kBlockCoords; want = (size_t)c->nblk * 2 * kBlockCoords; break;
    case SWARM_T_OEXPS:
      if (!c->oexps) return SWARM_ESTATE;
      dev = c->oexps + (size_t)node * c->nblk; want = (size_t)c->nblk; break;
    case SWARM_T_MU_RECORD:
      if (!c->track) return SWARM_ESTATE;
      dev = c->mu_hist + (size_t)node * c->pitch; want = d * 4; break;
    case SWARM_T_A_RECORD:
      if (!c->track) return SWARM_ESTATE;
      dev = c->a_hist + node; want = 8; break;
    case SWARM_T_GRAM: {
      if (!c->gram) return SWARM_ESTATE;
      if (write) return SWARM_EINVAL;
      if (node < 0 || node >= c->groups) return SWARM_ERANGE;
      const size_t m = (size_t)c->cfg.lsq_m;
      dev = c->gram + (size_t)node * m * m; want = m * m * 4; break;
    }
    case SWARM_T_CLOCKS: {
      if (bytes != 8) return SWARM_EINVAL;
      uint32_t* v = (uint32_t*)host;
      if (write) { c->wo[node] = v[0]; c->tau[node] = v[1]; }
      else { v[0] = c->wo[node]; v[1] = c->tau[node]; }
      return SWARM_OK;
    }
    case SWARM_T_COUNTERS: {
      if (bytes != 12) return SWARM_EINVAL;
      uint32_t* v = (uint32_t*)host;
      if (write) {
        if (v[2] == 1 || v[2] > 8) return SWARM_EINVAL;
        c->w[node] = v[0]; c->ls[node] = v[1]; c->pbits[node] = (int32_t)v[2];
      } else {
        v[0] = c->w[node]; v[1] = c->ls[node]; v[2] = (uint32_t)c->pbits[node];
      }
      return SWARM_OK;
    }
    case SWARM_T_A: {
      if (!c->A) return SWARM_ESTATE;
      if (node < 0 || node >= c->groups) return SWARM_ERANGE;
      const size_t m = (size_t)c->cfg.lsq_m;
      if (bytes != m * d * 4) return SWARM_EINVAL;
      SW_SYNC(c);
      int nl = 0;
      for (size_t r = 0; r < m; ++r) {
        char* hrow = (char*)host + r * d * 4;
        if (c->cfg.lsq_dtype == SWARM_F32) {
          float* drow = (float*)c->A + ((size_t)node * m + r) * c->pitch;
          if (write) SW_CUDA(c, cudaMemcpyAsync(drow, hrow, d * 4, cudaMemcpyHostToDevice, c->stream));
          else SW_CUDA(c, cudaMemcpyAsync(hrow, drow, d * 4, cudaMemcpyDeviceToHost, c->stream));
        } else {
          uint16_t* drow = (uint16_t*)c->A + ((size_t)node * m + r) * c->pitch;
          if (write) {
            SW_CUDA(c, cudaMemcpyAsync(c->convert_tmp, hrow, d * 4, cudaMemcpyHostToDevice, c->stream));
            SW_CUDA(c, launch_f32_to_bf16(c->convert_tmp, drow, (int64_t)d, c->stream, &nl));
          } else {
            SW_CUDA(c, launch_bf16_to_f32(drow, c->convert_tmp, (int64_t)d, c->stream, &nl));
            SW_CUDA(c, cudaMemcpyAsync(hrow, c->convert_tmp, d * 4, cudaMemcpyDeviceToHost, c->stream));
          }
          SW_SYNC(c);   // convert_tmp and pageable host memory are reused per row
        }
      }
      // rewritten rows change the matrix's Gram matrix, which the grouped local steps read
      if (write)
        SW_CUDA(c, launch_lsq_gram(c->A, c->cfg.lsq_dtype, c->cfg.lsq_m, c->pitch, node, 1, c->gram, c->kernel_status,
                                   c->wait_limit, c->stream, &nl));
      if (write && c->gram && c->cfg.lsq_dtype == SWARM_BF16) c->status_pending = true;
      c->launches += nl;
      SW_SYNC(c);
      return SWARM_OK;
    }
    default: return SWARM_EINVAL;
  }
  if (bytes != want) return SWARM_EINVAL;
  // the copy is ordered after earlier work by the stream; one synchronisation at the end is enough
  if (!write && !wait && bytes <= kReadQueueMaxRow) {
    // short queued read: into the ring now (a small dependent kernel, no copy engine between two launches),
    // to `host` at the next synchronising call
    const size_t need = (bytes + 15) / 16 * 16;
    if (c->rq_used + need > kReadQueueBytes) SW_SYNC(c);          // ring full: deliver what is queued first
    int nl = 0;
    SW_CUDA(c, launch_row_copy(dev, c->rq_dev + c->rq_used, (int64_t)bytes, c->stream, &nl));
    c->launches += nl;
    c->rq.push_back({host, c->rq_used, bytes});
    c->rq_used += need;
    return SWARM_OK;
  }
  if (write) SW_CUDA(c, cudaMemcpyAsync(dev, host, bytes, cudaMemcpyHostToDevice, c->stream));
  else SW_CUDA(c, cudaMemcpyAsync(host, dev, bytes, cudaMemcpyDeviceToHost, c->stream));
  if (wait) SW_SYNC(c);
  return SWARM_OK;
}

int swarm_get_data_rows(swarm_ctx* c, int32_t matrix, int32_t row0, int32_t nrows, float* dst, size_t bytes) {
  if (!c || !dst || nrows < 0) return SWARM_EINVAL;
  if (!c->A) return SWARM_ESTATE;
  if (matrix < 0 || matrix >= c->groups) return SWARM_ERANGE;
  if (row0 < 0 || (int64_t)row0 + nrows > c->cfg.lsq_m) return SWARM_ERANGE;
  const size_t d = (size_t)c->d;
  if (bytes != (size_t)nrows * d * 4) return SWARM_EINVAL;
  DeviceGuard guard(c->device);
  SW_SYNC(c);
  int nl = 0;
  for (int32_t r = 0; r < nrows; ++r) {
    char* hrow = (char*)dst + (size_t)r * d * 4;
    const size_t row = (size_t)matrix * c->cfg.lsq_m + (size_t)(row0 + r);
    if (c->cfg.lsq_dtype == SWARM_F32) {
      SW_CUDA(c, cudaMemcpyAsync(hrow, (const float*)c->A + row * c->pitch, d * 4, cudaMemcpyDeviceToHost, c->stream));
    } else {
      SW_CUDA(c, launch_bf16_to_f32((const uint16_t*)c->A + row * c->pitch, c->convert_tmp, (int64_t)d, c->stream, &nl));
      SW_CUDA(c, cudaMemcpyAsync(hrow, c->convert_tmp, d * 4, cudaMemcpyDeviceToHost, c->stream));
      SW_SYNC(c);   // convert_tmp is reused per row
    }
  }
  c->launches += nl;
  SW_SYNC(c);
  return SWARM_OK;
}

int swarm_get_tensor(swarm_ctx* c, int32_t which, int32_t node, void* dst, size_t bytes) {
  return tensor_access(c, which, node, dst, bytes, false);
}
int swarm_get_tensor_async(swarm_ctx* c, int32_t which, int32_t node, void* dst, size_t bytes) {
  return tensor_access(c, which, node, dst, bytes, false, false);
}
int swarm_set_tensor(swarm_ctx* c, int32_t which, int32_t node, const void* src, size_t bytes) {
  return tensor_access(c, which, node, const_cast<void*>(src), bytes, true);
}

}  // extern "C"
