// SwarmSGD pairwise-gossip oracle: a plain, slow, single-purpose CPU implementation.
//
// THIS IS TEST INFRASTRUCTURE. It exists so that the CUDA library can be checked
// element by element against something a reader can verify against the paper by
// eye. Nothing in the product path may include, link, import or call it. It shares
// no code, header, table or helper with the CUDA sources.
//
// What it follows (Alistarh et al., "Asynchronous Decentralized SGD with Quantized
// and Local Updates"):
//   * schedule: Section 2 "The Distributed System Model" and Algorithm 1 (initiator
//     uniform over nodes, responder uniform over its neighbours);
//   * local steps: Section 3 "The Communication Procedure" and the appendix section
//     "Notation and Auxiliary Potential Functions" (H sequential stochastic
//     gradient steps, each evaluated at the running iterate);
//   * interaction: Section 3 (both nodes receive Q(X^i)/2 + Q(X^j)/2, the initiator
//     additionally subtracts its pending local update) and Algorithm 1;
//   * quantizer: Corollary 1 (unbiased, error independent of the model norm,
//     decoded against a key that only needs to be close to the encoded vector).
//     The corollary is an existence statement; the construction used here is a
//     cubic lattice of power-of-two step 2^e whose points are coloured with their
//     index mod 2^b, decoded to the lattice point of that colour nearest the key;
//   * mean model and potential: Section 4 (mu_t, Gamma_t).
//
// Parity status of the parts (what each is pinned to in the CPU test-suite):
//   Philox4x32-10 ........ published known-answer vectors of the generator
//   integer/float maps ... moments and chi-square
//   topology ............. degree/symmetry/connectivity, lambda_2 closed forms
//   pair sampler ......... disjointness, adjacency, edge law 1/(n*rho_i)
//   exponent rule ........ exact rational brute force
//   Enc/Dec .............. exhaustive enumeration of the 2^16 rounding uniforms,
//                          lattice fixed points, decode-window theorem, far keys
//   packing .............. numpy bit-order routine
//   interactions ......... mean preservation, exact Gamma-change identity,
//                          unbiasedness over write counters
//   local steps .......... finite differences / convergence on consistent systems,
//                          sample moments
//   mu, Gamma ............ complete-graph identity and n = 2 closed form
//   steady-state level of Gamma over long runs: parity unpinned (statistical only)
//
// Build: g++ -O2 -std=c++17 -ffp-contract=off -fPIC -shared (see build.py).
// All floating point that decides an integer (codes, exponents) is done in fp32
// with one IEEE operation per step, exactly as written; accumulations that the
// method defines over the reals (dot products, mu, Gamma) are done in double.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <thread>
#include <vector>

namespace {

// ---------------------------------------------------------------------------
// Counter-based generator: Philox-4x32 with 10 rounds (Salmon et al., SC'11).
// ---------------------------------------------------------------------------
constexpr uint32_t kMul0 = 0xD2511F53u, kMul1 = 0xCD9E8D57u;
constexpr uint32_t kWeyl0 = 0x9E3779B9u, kWeyl1 = 0xBB67AE85u;

enum Stream : uint32_t {
  kStreamInit = 1, kStreamDataA = 2, kStreamDataNoise = 3, kStreamXStar = 4,
  kStreamNodeScalars = 5, kStreamTopology = 6, kStreamPairs = 7,
  kStreamMinibatch = 8, kStreamSynthGrad = 9, kStreamRounding = 10, kStreamStepCount = 11, kStreamOwnRounding = 12
};

void philox(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    if (round > 0) { k0 += kWeyl0; k1 += kWeyl1; }
    const uint64_t p0 = (uint64_t)kMul0 * c0;
    const uint64_t p1 = (uint64_t)kMul1 * c2;
    const uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
    const uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
    const uint32_t n0 = hi1 ^ c1 ^ k0;
    const uint32_t n1 = lo1;
    const uint32_t n2 = hi0 ^ c3 ^ k1;
    const uint32_t n3 = lo0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

struct Rng {
  uint32_t key[2];
  explicit Rng(uint64_t seed) { key[0] = (uint32_t)seed; key[1] = (uint32_t)(seed >> 32); }
  void words(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t out[4]) const {
    const uint32_t ctr[4] = {c0, c1, c2, c3};
    philox(ctr, key, out);
  }
};

// Uniform integer in [0, m): high half of the 32x32 product.
uint32_t uniform_int(uint32_t word, uint32_t m) { return (uint32_t)(((uint64_t)word * m) >> 32); }

// Uniform float in [0, 1): top 24 bits.
float uniform_float(uint32_t word) { return (float)(word >> 8) * 0x1p-24f; }

// Box-Muller: two words -> two standard normals, evaluated in double, rounded once.
void normal_pair(uint32_t w0, uint32_t w1, float out[2]) {
  const double u1 = ((double)(w0 >> 8) + 1.0) * 0x1p-24;  // (0, 1]
  const double u2 = (double)(w1 >> 8) * 0x1p-24;          // [0, 1)
  const double r = std::sqrt(-2.0 * std::log(u1));
  const double two_pi = 6.283185307179586476925286766559;
  out[0] = (float)(r * std::cos(two_pi * u2));
  out[1] = (float)(r * std::sin(two_pi * u2));
}

// Element k of the normal vector attached to (row, event, stream): four normals per
// generator call, call index k div 4.
float normal_at(const Rng& rng, uint32_t stream, uint32_t row, uint32_t event, int64_t k) {
  uint32_t w[4];
  rng.words((uint32_t)(k / 4), row, event, stream, w);
  float z[2];
  const int j = (int)(k % 4);
  if (j < 2) normal_pair(w[0], w[1], z); else normal_pair(w[2], w[3], z);
  return z[j & 1];
}

// ---------------------------------------------------------------------------
// Quantizer (constructive reading of Corollary 1): lattice 2^e * Z per coordinate,
// 2^b colours, L = 2^(b-1) - 1 the largest key distance (in lattice steps) that is
// always decoded correctly.
// ---------------------------------------------------------------------------
constexpr int kBlock = 1024;   // coordinates that share one exponent
constexpr int kExpMin = -126, kExpMax = 119;

int lattice_L(int bits) { return (1 << (bits - 1)) - 1; }

// Least e with L * 2^e >= rho, then raised so that M * 2^-e stays below 2^23
// (the scaled coordinates remain exactly representable integers plus fraction),
// and clamped to [-126, 119] so that both 2^e and 2^-e are normal floats.
int exponent_rule(float rho, float M, int bits) {
  const float L = (float)lattice_L(bits);
  int e;
  if (rho == 0.0f) {
    e = kExpMin;
  } else {
    int fe;
    std::frexp(rho, &fe);        // rho = m * 2^fe, m in [0.5, 1)
    e = fe - bits;               // L * 2^e < 2^(fe-1) <= rho: strictly too small
    while ((double)L * std::ldexp(1.0, e) < (double)rho) ++e;   // exact in double
  }
  if (M > 0.0f) {
    int fm;
    std::frexp(M, &fm);
    e = std::max(e, fm - 23);
  }
  e = std::max(e, kExpMin);
  e = std::min(e, kExpMax);
  return e;
}

float pow2f(int e) { return std::ldexp(1.0f, e); }   // e in [-126, 126]: exact, normal

// Saturating float -> int32 (round toward -inf already applied by the caller).
int32_t saturate_i32(float f) {
  if (std::isnan(f)) return 0;
  if (f >= 2147483648.0f) return std::numeric_limits<int32_t>::max();
  if (f <= -2147483648.0f) return std::numeric_limits<int32_t>::min();
  return (int32_t)f;
}

// Stochastic rounding of x onto the lattice of step 2^e with a 16-bit uniform u:
// rounds up with probability floor(frac * 2^16) / 2^16.
int32_t enc_q(float x, int e, uint32_t u16) {
  const float t = x * pow2f(-e);
  const float f = std::floor(t);
  const float frac = t - f;
  const uint32_t thr = (uint32_t)std::floor(frac * 65536.0f);
  const int32_t base = saturate_i32(f);
  return (int32_t)((uint32_t)base + (u16 < thr ? 1u : 0u));
}

uint32_t code_of(int32_t q, int bits) { return (uint32_t)q & ((1u << bits) - 1u); }

// Decode colour c against key y: the lattice index congruent to c (mod 2^b) inside
// the window [q_y - L, q_y + L + 1] around the key's own cell q_y.
float dec(float y, uint32_t c, int e, int bits) {
  const float ty = y * pow2f(-e);
  const int32_t qy = saturate_i32(std::floor(ty));
  const uint32_t mask = (1u << bits) - 1u;
  int32_t delta = (int32_t)((c - (uint32_t)qy) & mask);
  if (delta > (1 << (bits - 1))) delta -= (1 << bits);
  const int32_t q = (int32_t)((uint32_t)qy + (uint32_t)delta);
  return (float)q * pow2f(e);
}

// The 16-bit rounding uniforms of a buffer owner at write counter w: one generator
// call per 8 consecutive coordinates; coordinate k takes word (k mod 8) div 2, low
// half when k is even, high half when k is odd.
uint32_t sr_uniform(const Rng& rng, uint32_t owner, uint32_t w, int64_t k) {
  uint32_t words[4];
  rng.words((uint32_t)(k / 8), owner, w, kStreamRounding, words);
  const uint32_t word = words[(k % 8) / 2];
  return (k % 2 == 0) ? (word & 0xFFFFu) : (word >> 16);
}

// Packing inside a block: a little-endian bit stream, the code of local coordinate k occupies bits
// [k*b, (k+1)*b) of the block's 128*b bytes (bit t of the stream is bit t mod 8 of byte t div 8).
void put_code(uint8_t* block_bytes, int k, uint32_t c, int bits) {
  for (int t = 0; t < bits; ++t) {
    const int pos = k * bits + t;
    if ((c >> t) & 1u) block_bytes[pos / 8] = (uint8_t)(block_bytes[pos / 8] | (1u << (pos % 8)));
  }
}
uint32_t get_code(const uint8_t* block_bytes, int k, int bits) {
  uint32_t c = 0;
  for (int t = 0; t < bits; ++t) {
    const int pos = k * bits + t;
    c |= (uint32_t)((block_bytes[pos / 8] >> (pos % 8)) & 1u) << t;
  }
  return c;
}

// ---------------------------------------------------------------------------
// Swarm state
// ---------------------------------------------------------------------------
struct Config {
  int32_t objective;      // 0 none, 1 synthetic gradient, 2 least squares, 3 logistic regression (labels in {0, 1})
  int32_t nonblocking;    // 1: base snapshots exist; 2: also the nodes' own registers (two-register protocol)
  float init_std, offset_std;
  float grad_std, drift_std;
  int32_t lsq_m, lsq_batch, lsq_dtype, lsq_groups;
  float lsq_noise_std;
};

float round_to_bf16(float v) {   // round to nearest even onto 8 significant bits
  uint32_t u;
  std::memcpy(&u, &v, 4);
  const uint32_t lsb = (u >> 16) & 1u;
  u += 0x7FFFu + lsb;
  u &= 0xFFFF0000u;
  float r;
  std::memcpy(&r, &u, 4);
  return r;
}

struct Swarm {
  int32_t n = 0;
  int64_t d = 0;
  int64_t nblk = 0;
  int32_t kind = 0, degree = 0;
  Rng rng;
  Config cfg{};
  std::vector<int32_t> adj;          // n * degree
  std::vector<float> X, B;           // n * d
  std::vector<uint8_t> codes;        // n * nblk * 1024 (layout depends on pbits)
  std::vector<int8_t> exps;          // n * nblk
  std::vector<int32_t> pbits;        // n
  std::vector<uint32_t> w, ls;       // write counters, local-step counters
  uint32_t launch = 0;
  int32_t b_stale = 0;
  // two-register protocol (Section 3, "The Communication Registers"): the register a node writes
  // itself holds a 16-bit encoding of its snapshot; `codes` is then the register others write.
  std::vector<uint8_t> own;          // n * nblk * 2048: per block 1024 low bytes, then 1024 high bytes
  int32_t own_prefix = 16;           // bits of a partner's own register that a reader consumes (8 or 16)
  std::vector<int8_t> oexps;         // n * nblk
  std::vector<uint32_t> wo;          // write counters of the own registers
  std::vector<uint32_t> tau;         // interactions since the node last initiated
  // auxiliary potentials of the staleness analysis (appendix, "Potential Functions"): per node the mean
  // model at its last initiation and the squared distance of its snapshot to that mean
  int32_t track = 0;
  std::vector<float> mu_hist;        // n * d
  std::vector<double> a_hist;        // n
  int32_t p_mode = 0;                // convention the buffers were last written in: 0 none/blocking, 1 single buffer, 2 registers
  // objective data
  std::vector<float> offset, drift, shift;   // per-node scalars
  std::vector<float> A;              // groups * m * d
  std::vector<float> bvec;           // n * m
  std::vector<float> xstar;          // d
  int32_t groups = 0;

  Swarm(int32_t n_, int64_t d_, uint64_t seed) : n(n_), d(d_), rng(seed) {}
  float* x(int i) { return X.data() + (int64_t)i * d; }
  float* base(int i) { return B.data() + (int64_t)i * d; }
  uint8_t* code_row(int i) { return codes.data() + (int64_t)i * nblk * kBlock; }
  // own register: the 16-bit colour of coordinate k is split over two byte planes of its block, so that
  // a reader which needs only the 8-bit prefix (the low byte) touches half of the register
  uint8_t* own_lo(int i, int64_t k) { return own.data() + ((int64_t)i * nblk + k / kBlock) * 2 * kBlock + k % kBlock; }
  uint32_t own_get(int i, int64_t k) { const uint8_t* p = own_lo(i, k); return (uint32_t)p[0] | ((uint32_t)p[kBlock] << 8); }
  void own_put(int i, int64_t k, uint32_t c) { uint8_t* p = own_lo(i, k); p[0] = (uint8_t)c; p[kBlock] = (uint8_t)(c >> 8); }
  int8_t* exp_row(int i) { return exps.data() + (int64_t)i * nblk; }
  int group_of(int i) const { return groups == n ? i : i / (n / groups); }
};

bool build_topology(Swarm& s) {
  const int n = s.n;
  if (s.kind == 0) {
    s.degree = n - 1;
    s.adj.resize((size_t)n * s.degree);
    for (int i = 0; i < n; ++i) {
      int t = 0;
      for (int j = 0; j < n; ++j) if (j != i) s.adj[(size_t)i * s.degree + t++] = j;
    }
    return true;
  }
  if (s.kind == 1) {
    if (n < 3) return false;
    s.degree = 2;
    s.adj.resize((size_t)n * 2);
    for (int i = 0; i < n; ++i) {
      s.adj[(size_t)i * 2 + 0] = (i + n - 1) % n;
      s.adj[(size_t)i * 2 + 1] = (i + 1) % n;
    }
    return true;
  }
  if (s.kind == 2) {
    const int k = s.degree;
    if (k < 2 || (k % 2) != 0 || k > n - 1 || n < 3) return false;
    std::vector<uint8_t> edge((size_t)n * n, 0);
    std::vector<int> perm(n);
    int cycles = 0;
    for (uint32_t attempt = 0; attempt < 4096 && cycles < k / 2; ++attempt) {
      for (int i = 0; i < n; ++i) perm[i] = i;
      for (int i = n - 1; i >= 1; --i) {         // Fisher-Yates, word i of this attempt
        uint32_t wd[4];
        s.rng.words((uint32_t)(i / 4), 0, attempt, kStreamTopology, wd);
        const int j = (int)uniform_int(wd[i % 4], (uint32_t)(i + 1));
        std::swap(perm[i], perm[j]);
      }
      bool clash = false;
      for (int t = 0; t < n && !clash; ++t) {
        const int u = perm[t], v = perm[(t + 1) % n];
        if (edge[(size_t)u * n + v]) clash = true;
      }
      if (clash) continue;
      for (int t = 0; t < n; ++t) {
        const int u = perm[t], v = perm[(t + 1) % n];
        edge[(size_t)u * n + v] = edge[(size_t)v * n + u] = 1;
      }
      ++cycles;
    }
    if (cycles < k / 2) return false;
    s.adj.resize((size_t)n * k);
    for (int i = 0; i < n; ++i) {
      int t = 0;
      for (int j = 0; j < n; ++j) if (edge[(size_t)i * n + j]) s.adj[(size_t)i * k + t++] = j;
      if (t != k) return false;
    }
    return true;
  }
  return false;
}

void init_state(Swarm& s) {
  const int n = s.n;
  const int64_t d = s.d;
  const Config& c = s.cfg;
  s.offset.assign(n, 0.0f); s.drift.assign(n, 0.0f); s.shift.assign(n, 0.0f);
  s.track = 0; s.mu_hist.clear(); s.a_hist.clear();
  for (int i = 0; i < n; ++i) {
    uint32_t wd[4];
    s.rng.words(0, (uint32_t)i, 0, kStreamNodeScalars, wd);
    float z[2];
    normal_pair(wd[0], wd[1], z);
    s.offset[i] = c.offset_std * z[0];
    s.drift[i] = c.drift_std * z[1];
    s.shift[i] = 2.0f * uniform_float(wd[2]) - 1.0f;
  }
  s.X.assign((size_t)n * d, 0.0f);
  for (int i = 0; i < n; ++i) {
    float* xi = s.x(i);
    for (int64_t k = 0; k < d; ++k) {
      const float p = c.init_std * normal_at(s.rng, kStreamInit, (uint32_t)i, 0, k);
      xi[k] = p + s.offset[i];
    }
  }
  if (c.nonblocking) s.B = s.X; else s.B.clear();
  s.codes.assign((size_t)n * s.nblk * kBlock, 0);
  s.exps.assign((size_t)n * s.nblk, 0);
  s.pbits.assign(n, 0);
  s.w.assign(n, 0); s.ls.assign(n, 0);
  s.launch = 0; s.b_stale = 0; s.p_mode = 0;
  s.tau.assign(n, 0); s.wo.assign(n, 0);
  s.own_prefix = 16;
  if (c.nonblocking == 2) { s.own.assign((size_t)n * s.nblk * 2 * kBlock, 0); s.oexps.assign((size_t)n * s.nblk, 0); }
  else { s.own.clear(); s.oexps.clear(); }

  s.A.clear(); s.bvec.clear(); s.xstar.clear(); s.groups = 0;
  if (c.objective == 2 || c.objective == 3) {
    const int m = c.lsq_m;
    s.groups = c.lsq_groups > 0 ? c.lsq_groups : n;
    const float inv_sqrt_d = (float)(1.0 / std::sqrt((double)d));
    s.A.resize((size_t)s.groups * m * d);
    for (int g = 0; g < s.groups; ++g)
      for (int r = 0; r < m; ++r) {
        float* row = s.A.data() + ((size_t)g * m + r) * d;
        for (int64_t k = 0; k < d; ++k) {
          float v = normal_at(s.rng, kStreamDataA, (uint32_t)g, (uint32_t)r, k) * inv_sqrt_d;
          if (c.lsq_dtype == 1) v = round_to_bf16(v);
          row[k] = v;
        }
      }
    s.xstar.resize(d);
    for (int64_t k = 0; k < d; ++k) s.xstar[k] = normal_at(s.rng, kStreamXStar, 0, 0, k);
    s.bvec.resize((size_t)n * m);
    for (int i = 0; i < n; ++i) {
      const int g = s.group_of(i);
      for (int r = 0; r < m; ++r) {
        const float* row = s.A.data() + ((size_t)g * m + r) * d;
        double acc = 0.0;
        for (int64_t k = 0; k < d; ++k) acc += (double)row[k] * (double)s.xstar[k];
        const float noise = c.lsq_noise_std * normal_at(s.rng, kStreamDataNoise, (uint32_t)i, 0, r);
        const float score = (float)(acc + (double)s.shift[i] + (double)noise);
        // least squares: real-valued label; logistic regression: its sign as a {0, 1} class
        s.bvec[(size_t)i * m + r] = c.objective == 3 ? (score > 0.0f ? 1.0f : 0.0f) : score;
      }
    }
  }
}

// ---------------------------------------------------------------------------
// Local steps
// ---------------------------------------------------------------------------
void minibatch_rows(const Swarm& s, int node, uint32_t event, int32_t* rows) {
  const int g = s.group_of(node);
  for (int t = 0; t < s.cfg.lsq_batch; ++t) {
    uint32_t wd[4];
    s.rng.words((uint32_t)(t / 4), (uint32_t)g, event, kStreamMinibatch, wd);
    rows[t] = (int32_t)uniform_int(wd[t % 4], (uint32_t)s.cfg.lsq_m);
  }
}

void local_step_synth(Swarm& s, int i, float lr) {
  float* xi = s.x(i);
  const uint32_t event = s.ls[i];
  for (int64_t k = 0; k < s.d; ++k) {
    const float z = normal_at(s.rng, kStreamSynthGrad, (uint32_t)i, event, k);
    const float p = s.cfg.grad_std * z;
    const float g = s.drift[i] + p;
    const float st = lr * g;
    xi[k] = xi[k] - st;
  }
}

// One minibatch step of node i on the given rows of its data matrix (Section 3, "The Communication
// Procedure": x <- x - lr * g~(x), g~ the gradient of the minibatch objective at the running iterate).
void lsq_step_on_rows(Swarm& s, int i, const int32_t* rows, int bsz, float lr) {
  const int m = s.cfg.lsq_m;
  const int64_t d = s.d;
  const float* Ag = s.A.data() + (size_t)s.group_of(i) * m * d;
  float* xi = s.x(i);
  std::vector<double> resid(bsz);
  for (int t = 0; t < bsz; ++t) {
    const float* row = Ag + (size_t)rows[t] * d;
    double acc = 0.0;
    for (int64_t k = 0; k < d; ++k) acc += (double)row[k] * (double)xi[k];
    // least squares: f = (1/2m) sum (a.x - b)^2; logistic: f = (1/m) sum log(1 + e^{a.x}) - y a.x.
    // Either way the stochastic gradient is (1/B) sum_s resid_s a_s with the residual below.
    const double pred = s.cfg.objective == 3 ? 1.0 / (1.0 + std::exp(-acc)) : acc;
    resid[t] = pred - (double)s.bvec[(size_t)i * m + rows[t]];
  }
  for (int64_t k = 0; k < d; ++k) {
    double g = 0.0;
    for (int t = 0; t < bsz; ++t) g += resid[t] * (double)Ag[(size_t)rows[t] * d + k];
    g /= (double)bsz;
    xi[k] = (float)((double)xi[k] - (double)lr * g);
  }
}

void local_step_lsq(Swarm& s, int i, float lr) {
  std::vector<int32_t> rows(s.cfg.lsq_batch);
  minibatch_rows(s, i, s.ls[i], rows.data());
  lsq_step_on_rows(s, i, rows.data(), s.cfg.lsq_batch, lr);
}

// Number of local steps of a node as a geometric random variable of mean H (Section 3, "Sequential
// model"): Bernoulli trials with success probability 1/H, the count is the index of the first
// success. Trial t of node i at step counter e uses word t of stream 11; capped at 1024 trials.
constexpr int kMaxGeometricTrials = 1024;
int geometric_steps(const Swarm& s, int node, uint32_t event, int mean_h) {
  for (int t = 0; t < kMaxGeometricTrials; ++t) {
    uint32_t wd[4];
    s.rng.words((uint32_t)(t / 4), (uint32_t)node, event, kStreamStepCount, wd);
    if (uniform_int(wd[t % 4], (uint32_t)mean_h) == 0) return t + 1;
  }
  return kMaxGeometricTrials;
}

// ---------------------------------------------------------------------------
// Interactions
// ---------------------------------------------------------------------------
void encode_block(const Swarm& s, const float* x, int64_t k0, int len, int e, int bits,
                  uint32_t owner, uint32_t wctr, uint8_t* block_bytes) {
  std::memset(block_bytes, 0, (size_t)kBlock * bits / 8);
  for (int k = 0; k < len; ++k) {
    const uint32_t u = sr_uniform(s.rng, owner, wctr, k0 + k);
    put_code(block_bytes, k, code_of(enc_q(x[k0 + k], e, u), bits), bits);
  }
}

void interact_blocking(Swarm& s, int a, int b, int bits) {
  float* xa = s.x(a); float* xb = s.x(b);
  const int64_t d = s.d;
  if (bits == 32) {
    for (int64_t k = 0; k < d; ++k) { const float v = 0.5f * (xa[k] + xb[k]); xa[k] = v; xb[k] = v; }
    return;
  }
  const size_t block_bytes = (size_t)kBlock * bits / 8;
  for (int64_t blk = 0; blk < s.nblk; ++blk) {
    const int64_t k0 = blk * kBlock;
    const int len = (int)std::min<int64_t>(kBlock, d - k0);
    float rho = 0.0f, M = 0.0f;
    for (int k = 0; k < len; ++k) {
      const float va = xa[k0 + k], vb = xb[k0 + k];
      rho = std::max(rho, std::fabs(va - vb));
      M = std::max(M, std::max(std::fabs(va), std::fabs(vb)));
    }
    const int e = exponent_rule(rho, M, bits);
    uint8_t* ca = s.code_row(a) + blk * block_bytes;
    uint8_t* cb = s.code_row(b) + blk * block_bytes;
    encode_block(s, xa, k0, len, e, bits, (uint32_t)a, s.w[a], ca);
    encode_block(s, xb, k0, len, e, bits, (uint32_t)b, s.w[b], cb);
    s.exp_row(a)[blk] = (int8_t)e;
    s.exp_row(b)[blk] = (int8_t)e;
    for (int k = 0; k < len; ++k) {
      // each side decodes the partner's buffer with its own model as the key
      const float Qa = dec(xb[k0 + k], get_code(ca, k, bits), e, bits);
      const float Qb = dec(xa[k0 + k], get_code(cb, k, bits), e, bits);
      const float v = 0.5f * (Qa + Qb);
      xa[k0 + k] = v; xb[k0 + k] = v;
    }
  }
  s.w[a] += 1; s.w[b] += 1;
  s.pbits[a] = bits; s.pbits[b] = bits;
}

// Fill every communication buffer with an encoding of the node's base snapshot,
// scaled per block by the spread of all base snapshots in that block.
void publish(Swarm& s, int bits) {
  const int n = s.n; const int64_t d = s.d;
  if (s.b_stale) { s.B = s.X; s.b_stale = 0; }
  const size_t block_bytes = (size_t)kBlock * bits / 8;
  for (int64_t blk = 0; blk < s.nblk; ++blk) {
    const int64_t k0 = blk * kBlock;
    const int len = (int)std::min<int64_t>(kBlock, d - k0);
    float rho = 0.0f, M = 0.0f;
    for (int k = 0; k < len; ++k) {
      float lo = s.base(0)[k0 + k], hi = lo;
      for (int i = 0; i < n; ++i) {
        const float v = s.base(i)[k0 + k];
        lo = std::min(lo, v); hi = std::max(hi, v);
        M = std::max(M, std::fabs(v));
      }
      rho = std::max(rho, hi - lo);
    }
    const int e = exponent_rule(rho, M, bits);
    for (int i = 0; i < n; ++i) {
      encode_block(s, s.base(i), k0, len, e, bits, (uint32_t)i, s.w[i],
                   s.code_row(i) + blk * block_bytes);
      s.exp_row(i)[blk] = (int8_t)e;
    }
  }
  for (int i = 0; i < n; ++i) { s.w[i] += 1; s.pbits[i] = bits; }
  s.p_mode = 1;
}

bool needs_publish(const Swarm& s, int bits, int mode) {
  if (s.b_stale || s.p_mode != mode) return true;
  for (int i = 0; i < s.n; ++i) if (s.pbits[i] != bits) return true;
  return false;
}

void interact_nonblocking(Swarm& s, int a, int b, int bits) {
  const int64_t d = s.d;
  float* xa = s.x(a); float* ba = s.base(a);
  const size_t block_bytes = (size_t)kBlock * bits / 8;
  std::vector<float> new_x(kBlock), avg(kBlock);
  for (int64_t blk = 0; blk < s.nblk; ++blk) {
    const int64_t k0 = blk * kBlock;
    const int len = (int)std::min<int64_t>(kBlock, d - k0);
    uint8_t* ca = s.code_row(a) + blk * block_bytes;
    uint8_t* cb = s.code_row(b) + blk * block_bytes;
    const int ea = s.exp_row(a)[blk], eb = s.exp_row(b)[blk];
    float spread = 0.0f, dmax = 0.0f, M = 0.0f;
    for (int k = 0; k < len; ++k) {
      const float key = ba[k0 + k];                 // the initiator's own model is the key
      const float own = dec(key, get_code(ca, k, bits), ea, bits);
      const float oth = dec(key, get_code(cb, k, bits), eb, bits);
      const float av = 0.5f * (own + oth);
      const float D = key - xa[k0 + k];             // pending local update (eta * h)
      const float nx = av - D;
      avg[k] = av; new_x[k] = nx;
      spread = std::max(spread, std::fabs(own - oth));
      dmax = std::max(dmax, std::fabs(D));
      M = std::max(M, std::max(std::fabs(nx), std::fabs(av)));
    }
    const float rho = 2.0f * spread + dmax;
    const int e = exponent_rule(rho, M, bits);
    std::memset(ca, 0, block_bytes);
    std::memset(cb, 0, block_bytes);
    for (int k = 0; k < len; ++k) {
      const uint32_t ua = sr_uniform(s.rng, (uint32_t)a, s.w[a], k0 + k);
      const uint32_t ub = sr_uniform(s.rng, (uint32_t)b, s.w[b], k0 + k);
      put_code(ca, k, code_of(enc_q(new_x[k], e, ua), bits), bits);
      put_code(cb, k, code_of(enc_q(avg[k], e, ub), bits), bits);
    }
    s.exp_row(a)[blk] = (int8_t)e;
    s.exp_row(b)[blk] = (int8_t)e;
    for (int k = 0; k < len; ++k) { xa[k0 + k] = new_x[k]; ba[k0 + k] = new_x[k]; }
  }
  s.w[a] += 1; s.w[b] += 1;
}

// ---------------------------------------------------------------------------
// Two-register protocol: Algorithm 1 with its chain of three decodes.
//   own register of node k      O_k = Enc16(X^_k)    written only by k, 16 bits per coordinate,
//                                                    step of an 8-bit code of the guard distance
//                                                    (the writer does not know its readers' keys)
//   current register of node k  P_k = Enc_b(X_k)     written by whoever last interacted with k,
//                                                    scaled by the exact distance to its decoding
//                                                    key Q(X^_k) (the writer knows that key)
// Variable rate (Corollary 1, second case, and "Counting Communication Cost"): the long code sits in
// the writer's own register and a reader consumes only a prefix sized by its distance. The b-bit colour
// of a lattice point is the low b bits of its 16-bit colour, so the prefix is the low-order part; the
// register stores the low bytes of a block before the high bytes, and a reader that trusts its key to be
// within 127 steps reads the first half only (prefix = 8). The prefix is the reader's: every interaction
// states how many bits of its responder's own register its initiator consumes (own_prefix is the default for
// launches that state none). A node decoding its own register (key = the very snapshot that was encoded,
// less than one step away) always uses the 8-bit prefix.
// ---------------------------------------------------------------------------
constexpr int kOwnBits = 16;
constexpr int kOwnResolutionBits = 8;

uint32_t own_uniform(const Rng& rng, uint32_t owner, uint32_t w, int64_t k) {
  uint32_t words[4];
  rng.words((uint32_t)(k / 8), owner, w, kStreamOwnRounding, words);
  const uint32_t word = words[(k % 8) / 2];
  return (k % 2 == 0) ? (word & 0xFFFFu) : (word >> 16);
}

// Write O_i = Enc16(v) for one block with exponent eo, return the written lattice points in qhat.
void write_own_block(Swarm& s, int i, int64_t blk, const float* v, int len, int eo, float* qhat) {
  const int64_t k0 = blk * kBlock;
  for (int k = 0; k < len; ++k) {
    const int32_t q = enc_q(v[k], eo, own_uniform(s.rng, (uint32_t)i, s.wo[i], k0 + k));
    s.own_put(i, k0 + k, code_of(q, kOwnBits));
    qhat[k] = (float)q * pow2f(eo);
  }
  s.oexps[(int64_t)i * s.nblk + blk] = (int8_t)eo;
}

// Write P_i = Enc_b(v) for one block, scaled by the exact distance to the key `key`.
void write_current_block(Swarm& s, int i, int64_t blk, const float* v, const float* key, int len, int bits) {
  const int64_t k0 = blk * kBlock;
  float rho = 0.0f, M = 0.0f;
  for (int k = 0; k < len; ++k) {
    rho = std::max(rho, std::fabs(v[k] - key[k]));
    M = std::max(M, std::max(std::fabs(v[k]), std::fabs(key[k])));
  }
  const int e = exponent_rule(rho, M, bits);
  const size_t block_bytes = (size_t)kBlock * bits / 8;
  uint8_t* c = s.code_row(i) + blk * block_bytes;
  std::memset(c, 0, block_bytes);
  for (int k = 0; k < len; ++k)
    put_code(c, k, code_of(enc_q(v[k], e, sr_uniform(s.rng, (uint32_t)i, s.w[i], k0 + k)), bits), bits);
  s.exp_row(i)[blk] = (int8_t)e;
}

// Initial register contents: every node's registers hold encodings of its snapshot.
void register_publish(Swarm& s, int bits) {
  const int n = s.n; const int64_t d = s.d;
  if (s.b_stale) { s.B = s.X; s.b_stale = 0; }
  std::vector<float> qhat(kBlock);
  for (int64_t blk = 0; blk < s.nblk; ++blk) {
    const int64_t k0 = blk * kBlock;
    const int len = (int)std::min<int64_t>(kBlock, d - k0);
    float rho = 0.0f, M = 0.0f;
    for (int k = 0; k < len; ++k) {
      float lo = s.base(0)[k0 + k], hi = lo;
      for (int i = 0; i < n; ++i) {
        const float v = s.base(i)[k0 + k];
        lo = std::min(lo, v); hi = std::max(hi, v);
        M = std::max(M, std::fabs(v));
      }
      rho = std::max(rho, hi - lo);
    }
    const int eo = exponent_rule(rho, M, kOwnResolutionBits);
    for (int i = 0; i < n; ++i) {
      write_own_block(s, i, blk, s.base(i) + k0, len, eo, qhat.data());
      write_current_block(s, i, blk, s.base(i) + k0, qhat.data(), len, bits);
    }
  }
  for (int i = 0; i < n; ++i) { s.wo[i] += 1; s.w[i] += 1; s.pbits[i] = bits; }
  s.p_mode = 2;
}

void interact_registers(Swarm& s, int a, int b, int bits, int pfx) {
  const int64_t d = s.d;
  float* xa = s.x(a); float* ba = s.base(a);
  const size_t block_bytes = (size_t)kBlock * bits / 8;
  std::vector<float> new_x(kBlock), avg(kBlock), qhat_b(kBlock), qhat_new(kBlock);
  for (int64_t blk = 0; blk < s.nblk; ++blk) {
    const int64_t k0 = blk * kBlock;
    const int len = (int)std::min<int64_t>(kBlock, d - k0);
    const uint8_t* ca = s.code_row(a) + blk * block_bytes;
    const uint8_t* cb = s.code_row(b) + blk * block_bytes;
    const uint32_t pmask = (1u << pfx) - 1u;
    const int eoa = s.oexps[(int64_t)a * s.nblk + blk], eob = s.oexps[(int64_t)b * s.nblk + blk];
    const int epa = s.exp_row(a)[blk], epb = s.exp_row(b)[blk];
    float spread = 0.0f, dmax = 0.0f, M = 0.0f;
    for (int k = 0; k < len; ++k) {
      const float snap = ba[k0 + k];
      const float qhat_a = dec(snap, s.own_get(a, k0 + k) & 0xFFu, eoa, 8);   // Q(X^_a): local, key = own snapshot
      const float Qa = dec(qhat_a, get_code(ca, k, bits), epa, bits);         // Q(X_a)  <- Dec(Q(X^_a), Enc(X_a))
      qhat_b[k] = dec(snap, s.own_get(b, k0 + k) & pmask, eob, pfx);          // Q(X^_b) <- Dec(X^_a, prefix of Enc(X^_b))
      const float Qb = dec(qhat_b[k], get_code(cb, k, bits), epb, bits);      // Q(X_b)  <- Dec(Q(X^_b), Enc(X_b))
      const float av = 0.5f * (Qa + Qb);
      const float D = snap - xa[k0 + k];                                      // pending local update (eta * h)
      const float nx = av - D;
      avg[k] = av; new_x[k] = nx;
      spread = std::max(spread, std::fabs(Qa - Qb));
      dmax = std::max(dmax, std::fabs(D));
      M = std::max(M, std::max(std::fabs(nx), std::fabs(av)));
    }
    const float rho = 2.0f * spread + dmax;
    const int eo = exponent_rule(rho, M, kOwnResolutionBits);
    write_own_block(s, a, blk, new_x.data(), len, eo, qhat_new.data());       // own register of a
    write_current_block(s, a, blk, new_x.data(), qhat_new.data(), len, bits); // current register of a
    write_current_block(s, b, blk, avg.data(), qhat_b.data(), len, bits);     // current register of b
    for (int k = 0; k < len; ++k) { xa[k0 + k] = new_x[k]; ba[k0 + k] = new_x[k]; }
  }
  s.wo[a] += 1; s.w[a] += 1; s.w[b] += 1;
}

// mu = (1/n) sum_i X^i, accumulated in double in node order, rounded once.
void mean_model(const Swarm& s, float* out) {
  for (int64_t k = 0; k < s.d; ++k) {
    double acc = 0.0;
    for (int i = 0; i < s.n; ++i) acc += (double)s.X[(int64_t)i * s.d + k];
    out[k] = (float)(acc / (double)s.n);
  }
}

// Node i initiated: remember the mean model of that moment and ||X^_i - mu||^2 (one term of A_t).
void record_initiation(Swarm& s, int i, const float* mu) {
  double a = 0.0;
  for (int64_t k = 0; k < s.d; ++k) {
    s.mu_hist[(int64_t)i * s.d + k] = mu[k];
    const double t = (double)s.base(i)[k] - (double)mu[k];
    a += t * t;
  }
  s.a_hist[i] = a;
}

int validate_pairs(const Swarm& s, const int32_t* pairs, int npairs) {
  std::vector<uint8_t> used(s.n, 0);
  for (int p = 0; p < npairs; ++p) {
    const int a = pairs[2 * p], b = pairs[2 * p + 1];
    if (a < 0 || a >= s.n || b < 0 || b >= s.n) return -2;
    if (a == b || used[a] || used[b]) return -3;
    bool adjacent = false;
    for (int t = 0; t < s.degree; ++t) if (s.adj[(size_t)a * s.degree + t] == b) adjacent = true;
    if (!adjacent) return -3;
    used[a] = used[b] = 1;
  }
  return 0;
}

}  // namespace

// ---------------------------------------------------------------------------
// C interface for the tests (ctypes)
// ---------------------------------------------------------------------------
extern "C" {

void orc_philox(const uint32_t* ctr, const uint32_t* key, uint32_t* out) { philox(ctr, key, out); }
uint32_t orc_uniform_int(uint32_t word, uint32_t m) { return uniform_int(word, m); }
float orc_uniform_float(uint32_t word) { return uniform_float(word); }
void orc_normal_pair(uint32_t w0, uint32_t w1, float* out) { normal_pair(w0, w1, out); }
int orc_exponent(float rho, float M, int bits) { return exponent_rule(rho, M, bits); }
int32_t orc_enc_q(float x, int e, uint32_t u16) { return enc_q(x, e, u16); }
uint32_t orc_code(int32_t q, int bits) { return code_of(q, bits); }
float orc_dec(float y, uint32_t c, int e, int bits) { return dec(y, c, e, bits); }
float orc_round_bf16(float v) { return round_to_bf16(v); }

void orc_sr_uniforms(uint64_t seed, uint32_t owner, uint32_t w, int64_t k0, int64_t count, uint16_t* out) {
  Rng rng(seed);
  for (int64_t k = 0; k < count; ++k) out[k] = (uint16_t)sr_uniform(rng, owner, w, k0 + k);
}

// codes: one per byte, count <= 1024; out: 1024*bits/8 bytes
void orc_pack_block(const uint8_t* codes, int count, int bits, uint8_t* out) {
  std::memset(out, 0, (size_t)kBlock * bits / 8);
  for (int k = 0; k < count; ++k) put_code(out, k, codes[k], bits);
}
void orc_unpack_block(const uint8_t* packed, int count, int bits, uint8_t* codes) {
  for (int k = 0; k < count; ++k) codes[k] = (uint8_t)get_code(packed, k, bits);
}

void* orc_create(int32_t n, int64_t d, int32_t kind, int32_t degree, uint64_t seed) {
  if (n < 2 || d < 1) return nullptr;
  Swarm* s = new Swarm(n, d, seed);
  s->kind = kind; s->degree = degree;
  s->nblk = (d + kBlock - 1) / kBlock;
  if (!build_topology(*s)) { delete s; return nullptr; }
  s->cfg = Config{0, 0, 0.1f, 0.0f, 0.0f, 0.0f, 0, 0, 0, 0, 0.0f};
  init_state(*s);
  return s;
}
void orc_destroy(void* h) { delete (Swarm*)h; }

int orc_configure(void* h, const Config* c) {
  Swarm& s = *(Swarm*)h;
  if (c->objective < 0 || c->objective > 3 || c->nonblocking < 0 || c->nonblocking > 2) return -1;
  if (c->objective >= 2) {
    if (c->lsq_m < 1 || c->lsq_batch < 1 || c->lsq_dtype < 0 || c->lsq_dtype > 1) return -1;
    if (c->lsq_groups < 0 || (c->lsq_groups > 0 && s.n % c->lsq_groups != 0)) return -1;
  }
  s.cfg = *c;
  init_state(s);
  return 0;
}

int32_t orc_degree(void* h) { return ((Swarm*)h)->degree; }
int64_t orc_nblk(void* h) { return ((Swarm*)h)->nblk; }
int32_t* orc_adj(void* h) { return ((Swarm*)h)->adj.data(); }
float* orc_X(void* h) { return ((Swarm*)h)->X.data(); }
float* orc_B(void* h) { Swarm& s = *(Swarm*)h; return s.B.empty() ? nullptr : s.B.data(); }
uint8_t* orc_codes(void* h) { return ((Swarm*)h)->codes.data(); }
int8_t* orc_exps(void* h) { return ((Swarm*)h)->exps.data(); }
int32_t* orc_pbits(void* h) { return ((Swarm*)h)->pbits.data(); }
uint32_t* orc_w(void* h) { return ((Swarm*)h)->w.data(); }
uint32_t* orc_ls(void* h) { return ((Swarm*)h)->ls.data(); }
uint32_t* orc_launch(void* h) { return &((Swarm*)h)->launch; }
int32_t* orc_b_stale(void* h) { return &((Swarm*)h)->b_stale; }
float* orc_A(void* h) { Swarm& s = *(Swarm*)h; return s.A.empty() ? nullptr : s.A.data(); }
float* orc_bvec(void* h) { Swarm& s = *(Swarm*)h; return s.bvec.empty() ? nullptr : s.bvec.data(); }
float* orc_xstar(void* h) { Swarm& s = *(Swarm*)h; return s.xstar.empty() ? nullptr : s.xstar.data(); }
float* orc_offset(void* h) { return ((Swarm*)h)->offset.data(); }
float* orc_drift(void* h) { return ((Swarm*)h)->drift.data(); }
float* orc_shift(void* h) { return ((Swarm*)h)->shift.data(); }
int32_t orc_groups(void* h) { return ((Swarm*)h)->groups; }

int orc_minibatch_rows(void* h, int32_t node, uint32_t event, int32_t* rows) {
  Swarm& s = *(Swarm*)h;
  if (s.cfg.objective < 2 || node < 0 || node >= s.n) return -1;
  minibatch_rows(s, node, event, rows);
  return 0;
}

// Algorithm 1, sampling lines: initiator uniform over the nodes, responder uniform
// over the initiator's neighbours; draws touching a node already paired in this
// launch are rejected so that the accepted pairs are disjoint.
int orc_sample_pairs(void* h, int32_t max_pairs, int32_t* out_pairs, int32_t* out_count) {
  Swarm& s = *(Swarm*)h;
  if (max_pairs < 1) return -1;
  std::vector<uint8_t> used(s.n, 0);
  int count = 0;
  for (int64_t attempt = 0; attempt < 16LL * max_pairs && count < max_pairs; ++attempt) {
    uint32_t wd[4];
    s.rng.words((uint32_t)attempt, 0, s.launch, kStreamPairs, wd);
    const int i = (int)uniform_int(wd[0], (uint32_t)s.n);
    const int j = s.adj[(size_t)i * s.degree + uniform_int(wd[1], (uint32_t)s.degree)];
    if (used[i] || used[j]) continue;
    used[i] = used[j] = 1;
    out_pairs[2 * count] = i; out_pairs[2 * count + 1] = j;
    ++count;
  }
  *out_count = count;
  s.launch += 1;
  return 0;
}

int orc_local_steps(void* h, const int32_t* nodes, int32_t count, int32_t H, float lr) {
  Swarm& s = *(Swarm*)h;
  if (s.cfg.objective == 0 || H < 0 || count < 0) return -1;
  std::vector<uint8_t> seen(s.n, 0);
  for (int t = 0; t < count; ++t) {
    if (nodes[t] < 0 || nodes[t] >= s.n) return -2;
    if (seen[nodes[t]]) return -1;
    seen[nodes[t]] = 1;
  }
  for (int t = 0; t < count; ++t) {
    const int i = nodes[t];
    for (int q = 0; q < H; ++q) {
      if (s.cfg.objective == 1) local_step_synth(s, i, lr); else local_step_lsq(s, i, lr);
      s.ls[i] += 1;
    }
  }
  return 0;
}

// One least-squares (or logistic) step of `node` on an explicit list of rows of its data matrix instead of
// the rows its counter would draw; the step counter advances as for a drawn minibatch. For checks of a
// single step of a large swarm on a small copy of the rows it touched.
int orc_local_step_on_rows(void* h, int32_t node, const int32_t* rows, int32_t count, float lr) {
  Swarm& s = *(Swarm*)h;
  if (s.cfg.objective < 2 || node < 0 || node >= s.n || count < 1) return -1;
  for (int t = 0; t < count; ++t) if (rows[t] < 0 || rows[t] >= s.cfg.lsq_m) return -2;
  lsq_step_on_rows(s, node, rows, count, lr);
  s.ls[node] += 1;
  return 0;
}

// Local steps with a geometric number of steps per node (mean mean_h); out_steps receives the counts.
int orc_local_steps_geometric(void* h, const int32_t* nodes, int32_t count, int32_t mean_h, float lr, int32_t* out_steps) {
  Swarm& s = *(Swarm*)h;
  if (s.cfg.objective == 0 || mean_h < 1 || count < 0) return -1;
  std::vector<uint8_t> seen(s.n, 0);
  for (int t = 0; t < count; ++t) {
    if (nodes[t] < 0 || nodes[t] >= s.n) return -2;
    if (seen[nodes[t]]) return -1;
    seen[nodes[t]] = 1;
  }
  for (int t = 0; t < count; ++t) {
    const int i = nodes[t];
    const int steps = geometric_steps(s, i, s.ls[i], mean_h);
    if (out_steps) out_steps[t] = steps;
    for (int q = 0; q < steps; ++q) {
      if (s.cfg.objective == 1) local_step_synth(s, i, lr); else local_step_lsq(s, i, lr);
      s.ls[i] += 1;
    }
  }
  return 0;
}

// pairs: npairs x (initiator, responder). threads > 1 splits the (disjoint, hence
// independent) pairs over plain std::thread workers.
// prefixes (may be null: the context's default for every pair): per pair the number of bits, 8 or 16, of the
// responder's own register that the initiator reads (two-register mode only).
int orc_interact_prefixed(void* h, const int32_t* pairs, const int32_t* prefixes, int32_t npairs, int32_t bits,
                          int32_t mode, int32_t threads) {
  Swarm& s = *(Swarm*)h;
  if (npairs < 0 || mode < 0 || mode > 2) return -1;
  if (prefixes) {
    if (mode != 2) return -1;
    for (int p = 0; p < npairs; ++p) if (prefixes[p] != 8 && prefixes[p] != 16) return -1;
  }
  if (!((bits >= 2 && bits <= 8) || (bits == 32 && mode == 0))) return -1;
  if (mode == 1 && !s.cfg.nonblocking) return -4;
  if (mode == 2 && s.cfg.nonblocking != 2) return -4;
  if (mode == 0 && s.track) return -4;   // a blocking exchange has no outdated model to track
  const int v = validate_pairs(s, pairs, npairs);
  if (v != 0) return v;
  if (mode == 1 && needs_publish(s, bits, 1)) publish(s, bits);
  if (mode == 2 && needs_publish(s, bits, 2)) register_publish(s, bits);
  auto run = [&](int p) {
    if (mode == 0) interact_blocking(s, pairs[2 * p], pairs[2 * p + 1], bits);
    else if (mode == 1) interact_nonblocking(s, pairs[2 * p], pairs[2 * p + 1], bits);
    else interact_registers(s, pairs[2 * p], pairs[2 * p + 1], bits, prefixes ? prefixes[p] : s.own_prefix);
  };
  if (threads <= 1 || npairs <= 1) {
    for (int p = 0; p < npairs; ++p) run(p);
  } else {
    const int T = std::min(threads, npairs);
    std::vector<std::thread> pool;
    for (int t = 0; t < T; ++t)
      pool.emplace_back([&, t]() { for (int p = t; p < npairs; p += T) run(p); });
    for (auto& th : pool) th.join();
  }
  // a blocking exchange moves X without refreshing the base snapshots and leaves the buffers in its
  // own convention (keys = partner models)
  if (mode == 0 && npairs > 0 && bits != 32) s.p_mode = 0;
  if (mode == 0 && s.cfg.nonblocking && npairs > 0) s.b_stale = 1;
  // staleness clocks (appendix, "Notation and Auxiliary Potential Functions"): the interactions of a
  // launch are taken in list order; an interaction resets its initiator and ages everybody else
  for (int p = 0; p < npairs; ++p) {
    for (int i = 0; i < s.n; ++i) s.tau[i] += 1;
    s.tau[pairs[2 * p]] = 0;
  }
  // the interactions of one launch count as simultaneous for the auxiliary potentials: every initiator
  // of the launch records the mean model after the launch
  if (s.track && npairs > 0) {
    std::vector<float> mu(s.d);
    mean_model(s, mu.data());
    for (int p = 0; p < npairs; ++p) record_initiation(s, pairs[2 * p], mu.data());
  }
  return 0;
}

int orc_interact(void* h, const int32_t* pairs, int32_t npairs, int32_t bits, int32_t mode, int32_t threads) {
  return orc_interact_prefixed(h, pairs, nullptr, npairs, bits, mode, threads);
}

// Start (or stop) tracking the auxiliary potentials: every node counts as having initiated just now.
int orc_track_staleness(void* h, int32_t enable) {
  Swarm& s = *(Swarm*)h;
  if (!enable) { s.track = 0; s.mu_hist.clear(); s.a_hist.clear(); return 0; }
  if (!s.cfg.nonblocking || s.b_stale) return -4;
  s.track = 1;
  s.mu_hist.assign((size_t)s.n * s.d, 0.0f);
  s.a_hist.assign(s.n, 0.0);
  std::vector<float> mu(s.d);
  mean_model(s, mu.data());
  for (int i = 0; i < s.n; ++i) { record_initiation(s, i, mu.data()); s.tau[i] = 0; }
  return 0;
}
float* orc_mu_hist(void* h) { Swarm& s = *(Swarm*)h; return s.mu_hist.empty() ? nullptr : s.mu_hist.data(); }
double* orc_a_hist(void* h) { Swarm& s = *(Swarm*)h; return s.a_hist.empty() ? nullptr : s.a_hist.data(); }

// out = { Gamma^_t = sum_i ||X^_i - mu_t||^2,  A_t = sum_i ||X_{t-tau_i} - mu_{t-tau_i}||^2,
//         B_t = sum_i ||mu_t - mu_{t-tau_i}||^2 }  with X^_i = X_{t-tau_i} the snapshot of node i.
int orc_aux_potentials(void* h, double* out) {
  Swarm& s = *(Swarm*)h;
  if (!s.track) return -4;
  std::vector<float> mu(s.d);
  mean_model(s, mu.data());
  double gh = 0.0, A = 0.0, Bt = 0.0;
  for (int i = 0; i < s.n; ++i) {
    for (int64_t k = 0; k < s.d; ++k) {
      const double t = (double)s.base(i)[k] - (double)mu[k];
      gh += t * t;
      const double u = (double)mu[k] - (double)s.mu_hist[(int64_t)i * s.d + k];
      Bt += u * u;
    }
    A += s.a_hist[i];
  }
  out[0] = gh; out[1] = A; out[2] = Bt;
  return 0;
}

int orc_register_publish(void* h, int32_t bits) {
  Swarm& s = *(Swarm*)h;
  if (s.cfg.nonblocking != 2 || (bits < 2 || bits > 8)) return -1;
  register_publish(s, bits);
  return 0;
}

uint8_t* orc_own(void* h) { Swarm& s = *(Swarm*)h; return s.own.empty() ? nullptr : s.own.data(); }
int orc_set_own_prefix(void* h, int32_t bits) {
  Swarm& s = *(Swarm*)h;
  if (bits != 8 && bits != 16) return -1;
  if (s.cfg.nonblocking != 2) return -4;
  s.own_prefix = bits;
  return 0;
}
int32_t orc_get_own_prefix(void* h) { return ((Swarm*)h)->own_prefix; }
int8_t* orc_oexps(void* h) { Swarm& s = *(Swarm*)h; return s.oexps.empty() ? nullptr : s.oexps.data(); }
uint32_t* orc_wo(void* h) { return ((Swarm*)h)->wo.data(); }
uint32_t* orc_tau(void* h) { return ((Swarm*)h)->tau.data(); }
int32_t* orc_p_mode(void* h) { return &((Swarm*)h)->p_mode; }

int orc_publish(void* h, int32_t bits) {
  Swarm& s = *(Swarm*)h;
  if (!s.cfg.nonblocking || (bits < 2 || bits > 8)) return -1;
  publish(s, bits);
  return 0;
}

// mu = (1/n) sum_i X^i, accumulated in double, rounded once.
void orc_mean_model(void* h, float* out) { mean_model(*(Swarm*)h, out); }

// Gamma = sum_i ||X^i - mu||^2, two passes in double.
double orc_potential(void* h) {
  Swarm& s = *(Swarm*)h;
  double gamma = 0.0;
  for (int64_t k = 0; k < s.d; ++k) {
    double mu = 0.0;
    for (int i = 0; i < s.n; ++i) mu += (double)s.x(i)[k];
    mu /= (double)s.n;
    for (int i = 0; i < s.n; ++i) { const double t = (double)s.x(i)[k] - mu; gamma += t * t; }
  }
  return gamma;
}

}  // extern "C"
