// Host-side view of the kernels: launch wrappers implemented in the .cu files and the
// plain-data descriptors they take. No CUDA types beyond cudaStream_t cross this header.
#pragma once
#include <cstddef>
#include <cstdint>
#include <cuda_runtime.h>

namespace swarm {

// One interaction of a launch, with the write counters that index the rounding uniforms.
struct PairDesc {
  int32_t a, b;        // initiator, responder
  uint32_t wa, wb;     // write counters of the two buffers before this interaction
  uint32_t woa;        // write counter of the initiator's own register (two-register protocol)
  uint32_t lsa, lsb;   // local-step counters of the two nodes (steps fused into the interaction)
  uint32_t prefix;     // two-register protocol: bits (8 or 16) of the responder's own register that the initiator reads
};

// Synthetic-gradient local steps taken inside an interaction kernel before the exchange (H = 0: none).
struct FusedSteps {
  int32_t H;
  int32_t responders;  // 1: the responder of each pair steps too; 0: initiators only
  float lr, grad_std;
  const float* scalars; // [n][3] per-node offset, drift, shift
};

// One node of a local-step launch.
struct NodeDesc {
  int32_t node;
  uint32_t event;      // local-step counter before this call
};

// Descriptor lists travel either inline in the kernel parameters (short lists: no copy engine
// involved, which matters when a launch is only a few microseconds long) or through device memory.
constexpr int kInlinePairs = 64;
constexpr int kInlineNodes = 64;
struct PairList {
  const PairDesc* ptr;
  int32_t n;
  PairDesc inl[kInlinePairs];
#ifdef __CUDACC__
  __device__ __forceinline__ PairDesc get(int64_t i) const { return n <= kInlinePairs ? inl[i] : ptr[i]; }
#endif
};
struct NodeList {
  const NodeDesc* ptr;
  int32_t n;
  NodeDesc inl[kInlineNodes];
#ifdef __CUDACC__
  __device__ __forceinline__ NodeDesc get(int i) const { return n <= kInlineNodes ? inl[i] : ptr[i]; }
#endif
};

// Up to 16 nodes that share a data matrix and a local-step counter (hence a minibatch): one batched
// tensor-core least-squares step.
struct LsqUnit {
  int32_t group;
  uint32_t event;      // local-step counter of these nodes before this call
  int32_t count;       // nodes in use (1..16)
  int32_t nodes[16];
  int32_t pad;
};

// The ten round keys of the generator key (round r uses key + r * Weyl constant): computed once on the host and
// carried in the kernel parameters, where the generator reads them as constants.
struct PhiloxRoundKeys { uint32_t k0[10], k1[10]; };

struct StoreView {
  float* X;            // [n][pitch]
  float* B;            // [n][pitch] or nullptr
  uint8_t* codes;      // [n][nblk * 1024]
  int8_t* exps;        // [n][nblk]
  uint8_t* own;        // [n][nblk][2048] own registers (two-register protocol) or nullptr: per block the low
                       // bytes of the 1024 16-bit colours, then their high bytes
  int8_t* oexps;       // [n][nblk] exponents of the own registers
  int64_t pitch;       // elements per row, multiple of 1024
  int64_t d;
  int64_t nblk;
  int32_t n;
  uint32_t key0, key1; // generator key (seed low / high word)
  PhiloxRoundKeys rk;  // its round keys
  // warp index -> (pair, block) without a division: for w < 2^31, w / nblk = umulhi(w, nblk_magic) >> nblk_shift
  // (nblk_magic = 0: nblk is 1 and the quotient is w itself)
  uint32_t nblk_magic, nblk_shift;
  // 1: an interaction launch walks its (pair, block) list from the end. Launches alternate, so that a launch starts
  // with the rows its predecessor touched last, a good part of which is still in L2.
  uint32_t backwards;
};

// Multiplier and shift with floor(w / divisor) = umulhi(w, magic) >> shift for every w < 2^31 (divisor >= 2):
// with L = ceil(log2 divisor) and magic = floor(2^(31 + L) / divisor) + 1 the product w * magic / 2^(31 + L) exceeds
// w / divisor by less than 2^-L <= 1 / divisor, which cannot reach the next integer.
inline void division_magic(uint64_t divisor, uint32_t* magic, uint32_t* shift) {
  if (divisor < 2) { *magic = 0; *shift = 0; return; }
  uint32_t L = 0;
  while (((uint64_t)1 << L) < divisor) ++L;
  *magic = (uint32_t)((((uint64_t)1 << (31 + L)) / divisor) + 1);
  *shift = L - 1;
}

struct LsqView {
  const void* A;       // [groups][m][pitch] fp32 or bf16
  const float* bvec;   // [n][m]
  const float* gram;   // [groups][m][m] Gram matrices A A^T of the data matrices, or nullptr when not kept
  int32_t m, batch, dtype, groups, nodes_per_group;
  int32_t logistic;    // 1: residual = sigmoid(<a, x>) - y with labels in {0, 1}; 0: residual = <a, x> - b
};

// --- swarm_interact.cu -------------------------------------------------------------------
cudaError_t launch_interact_blocking(const StoreView& s, const PairList& pairs, int npairs, int bits,
                                     const FusedSteps& fs, cudaStream_t st, int* launches);
cudaError_t launch_interact_nonblocking(const StoreView& s, const PairList& pairs, int npairs, int bits,
                                        const FusedSteps& fs, cudaStream_t st, int* launches);
// wctr_dev: n write counters (uint32) used for the rounding uniforms of each node's buffer.
cudaError_t launch_publish(const StoreView& s, const uint32_t* wctr_dev, int bits, cudaStream_t st, int* launches);
// Two-register protocol. wctr_dev: n write counters of the current registers followed by n of the own registers.
cudaError_t launch_interact_registers(const StoreView& s, const PairList& pairs, int npairs, int bits,
                                      const FusedSteps& fs, cudaStream_t st, int* launches);
cudaError_t launch_register_publish(const StoreView& s, const uint32_t* wctr_dev, int bits, cudaStream_t st,
                                    int* launches);

// --- swarm_local.cu ----------------------------------------------------------------------
cudaError_t launch_init_models(const StoreView& s, const float* scalars_dev, float init_std, cudaStream_t st,
                               int* launches);
cudaError_t launch_node_scalars(float* scalars_dev, int n, float offset_std, float drift_std, uint32_t key0,
                                uint32_t key1, cudaStream_t st, int* launches);
cudaError_t launch_lsq_data(const StoreView& s, const LsqView& l, void* A, float* xstar, float* bvec,
                            const float* scalars_dev, float noise_std, cudaStream_t st, int* launches);
cudaError_t launch_local_synth(const StoreView& s, const NodeList& nodes, int count, int H, float lr,
                               float grad_std, const float* scalars_dev, cudaStream_t st, int* launches);
// partial_dev: scratch of count * batch * lsq_chunks(d) floats.
cudaError_t launch_local_lsq(const StoreView& s, const LsqView& l, const NodeList& nodes, int count, int H,
                             float lr, float* partial_dev, cudaStream_t st, int* launches);
int64_t lsq_chunks(int64_t d);
// True when the short-model kernels take two steps per round given the data's Gram matrix (row pitch and batch
// size small enough that both minibatches stay in registers).
bool lsq_small_steps_in_pairs(int64_t pitch, int batch);
// Sequential gossip in one launch (short models, fp32 least-squares data, batch <= 32): steps.n steps of one
// pair each; per step the pair's nodes (the initiator only if responders == 0) take H local steps, then the
// pair interacts in blocking mode at `bits` bits. The descriptors carry the counters of every step.
bool lsq_sequence_supported(const StoreView& s, const LsqView& l);
cudaError_t launch_lsq_sequence(const StoreView& s, const LsqView& l, const PairList& steps, int H, float lr, int bits,
                                int responders, cudaStream_t st, int* launches);

// --- swarm_lsq_tc.cu (bf16 data, batch <= 64) ----------------------------------------------
size_t lsq_tc_partial_bytes(int64_t pitch, int units);
size_t lsq_tc_resid_bytes(int units);
// Bytes of the Gram matrices of `matrices` data matrices of m rows; 0 when they are too large to keep (local steps
// then go one at a time instead of in groups).
size_t lsq_tc_gram_bytes(int matrices, int m);
// gram_dev[first_matrix .. first_matrix + matrices) = A A^T of those data matrices (dtype 1: bf16, on the tensor
// cores, with bounded waits that raise *status_dev like the step kernels'; else fp32; row padding must be zero).
cudaError_t launch_lsq_gram(const void* A_dev, int dtype, int m, int64_t pitch, int first_matrix, int matrices,
                            float* gram_dev, int* status_dev, uint32_t wait_limit, cudaStream_t st, int* launches);
// H steps of every unit, in groups of up to four steps per pair of passes when l.gram is set (one step otherwise).
// status_dev: one int, set to 1 if a bounded wait inside a kernel expired (kernels that find it set return at
// once); wait_limit: polls after which a wait on a tensor-core commit gives up.
// partial_dev and resid_dev: lsq_tc_partial_bytes / lsq_tc_resid_bytes for max_units units, the latter zeroed once.
cudaError_t launch_local_lsq_tc(const StoreView& s, const LsqView& l, const LsqUnit* units_dev, int nunits, int max_units,
                                int H, float lr, float* partial_dev, void* resid_dev, int* status_dev,
                                uint32_t wait_limit, cudaStream_t st, int* launches);
uint32_t lsq_tc_default_wait_limit();
cudaError_t launch_sample_pairs(const int32_t* adj_dev, int n, int degree, int max_pairs, uint32_t launch_ctr,
                                uint32_t key0, uint32_t key1, int32_t* out_pairs_dev, int32_t* out_count_dev,
                                uint8_t* used_dev, cudaStream_t st, int* launches);

// --- swarm_reduce.cu ---------------------------------------------------------------------
cudaError_t launch_mean_model(const StoreView& s, float* out_dev, cudaStream_t st, int* launches);
// partial_dev: potential_partials(d) doubles of scratch; ticket_dev: one zero-initialised counter (left at
// zero); out_dev: one double; out_host_mapped: device-visible address of a pinned host double, or nullptr.
cudaError_t launch_potential(const StoreView& s, double* partial_dev, unsigned int* ticket_dev, double* out_dev,
                             double* out_host_mapped, cudaStream_t st, int* launches);
int64_t potential_partials(int64_t d);
// Staleness tracking. mu_hist_dev: [n][pitch] mean-model records; a_hist_dev: n doubles;
// partial_dev: list.n * potential_partials(d) doubles (record) or 2 * potential_partials(d) (query).
cudaError_t launch_staleness_record(const StoreView& s, float* mu_hist_dev, const NodeList& list,
                                    double* partial_dev, double* a_hist_dev, cudaStream_t st, int* launches);
// out_dev: three doubles (Gamma-hat, A_t, B_t).
cudaError_t launch_aux_potentials(const StoreView& s, const float* mu_hist_dev, const double* a_hist_dev,
                                  double* partial_dev, double* out_dev, cudaStream_t st, int* launches);

// Device-to-device copy of a short row by a small dependent kernel (keeps the launch pipeline of programmatic
// dependents intact, which a copy-engine transfer between two launches would not).
cudaError_t launch_row_copy(const void* src_dev, void* dst_dev, int64_t bytes, cudaStream_t st, int* launches);

// Row conversion helpers for get/set of bf16 data.
cudaError_t launch_bf16_to_f32(const void* src, float* dst, int64_t count, cudaStream_t st, int* launches);
cudaError_t launch_f32_to_bf16(const float* src, void* dst, int64_t count, cudaStream_t st, int* launches);

}  // namespace swarm
