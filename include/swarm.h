/*
 * swarm.h -- C ABI of the B200 SwarmSGD gossip-interaction library.
 *
 * Paper: Alistarh et al., "Asynchronous Decentralized SGD with Quantized and Local
 * Updates" (SwarmSGD). n node models X^1..X^n in R^d live side by side in one GPU's
 * memory; time is counted in pairwise interactions over the edges of a graph G
 * (Section 2, "The Distributed System Model").
 *
 * General conventions
 *   - Every call returns SWARM_OK (0) or a negative SWARM_E* code; nothing aborts or
 *     throws across this boundary. swarm_strerror() names a code; for SWARM_ECUDA
 *     swarm_last_cuda_error() returns the CUDA error of the failing call.
 *   - The context owns every device buffer. Pointers named *_host are host memory,
 *     *_dev device memory; both stay owned by the caller and are only read or
 *     written during the call unless stated otherwise.
 *   - Arguments are validated on the host before anything is launched: a rejected
 *     call changes no state and no counter.
 *   - Device work is asynchronous on the context's stream and ordered by call order.
 *     swarm_potential, swarm_get_tensor, swarm_sample_pairs and swarm_sync wait for it.
 *   - Device-side waits are bounded (only the tensor-core local-step kernels have any). A kernel whose wait
 *     runs out raises a status word, writes no result and returns; later kernels of the context that would
 *     build on its result return at once. Every synchronising call checks that word: from then on each of them
 *     returns SWARM_ECUDA with swarm_last_cuda_error() == cudaErrorLaunchTimeout (the models are in an
 *     undefined state) until swarm_configure rebuilds the context from its seed.
 *   - One context is bound to the CUDA device that was current at swarm_init and is
 *     not thread-safe.
 *   - All kernels are compiled for sm_100a only; there is no CPU path.
 *   - Models and snapshots are expected to be finite. Magnitudes up to the largest float, subnormals and
 *     decode keys arbitrarily far from the encoded value are defined behaviour (saturating conversions,
 *     aliased lattice points); a 1024-coordinate block that holds a NaN or an infinity yields unspecified
 *     values for that block (never a fault: no address depends on model data).
 *
 * Memory layout (row-major, every row padded to a multiple of 1024 elements)
 *   X[n][pitch]   fp32 live models
 *   B[n][pitch]   fp32 base snapshots (non-blocking mode only): the model a node
 *                 adopted at its last initiation (Algorithm 1: \hat X^i)
 *   codes[n][nblk*1024] bytes: the node's communication buffer; at b bits per
 *                 coordinate the first nblk*128*b bytes are meaningful. Within a
 *                 1024-coordinate block the codes form a little-endian bit stream: the code of
 *                 local coordinate k occupies bits [k*b, (k+1)*b) of the block's 128*b bytes
 *                 (stream bit t = bit t mod 8 of byte t div 8); codes past d are zero.
 *   exps[n][nblk] int8 lattice exponents e (step 2^e) of each block of the buffer
 *   nblk = ceil(d / 1024)
 */
#ifndef SWARM_B200_H
#define SWARM_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct swarm_ctx swarm_ctx;

/* A directed interaction: a = initiator, b = responder (Section 2; Algorithm 1, sampling lines). */
typedef struct { int32_t a, b; } swarm_pair;

/* Communication graph G (Section 2). degree is read for SWARM_TOPO_REGULAR only (even, 2..n-1). */
typedef struct { int32_t kind, degree; } swarm_topology;
enum { SWARM_TOPO_COMPLETE = 0, SWARM_TOPO_RING = 1, SWARM_TOPO_REGULAR = 2 };

enum { SWARM_BLOCKING = 0, SWARM_NONBLOCKING = 1, SWARM_REGISTERS = 2 };
enum { SWARM_OBJ_NONE = 0, SWARM_OBJ_SYNTH = 1, SWARM_OBJ_LSQ = 2, SWARM_OBJ_LOGISTIC = 3 };
enum { SWARM_F32 = 0, SWARM_BF16 = 1 };

enum {
  SWARM_OK = 0,
  SWARM_EINVAL = -1,  /* bad n, d, bits, mode, H, count, NULL pointer, size mismatch          */
  SWARM_ERANGE = -2,  /* node id outside [0, n)                                                */
  SWARM_EPAIR  = -3,  /* pairs not disjoint, a == b, or (a, b) not an edge of G                */
  SWARM_ESTATE = -4,  /* e.g. non-blocking mode without base snapshots, local steps without an objective */
  SWARM_ENOMEM = -5,  /* device or host allocation failed                                      */
  SWARM_ECUDA  = -6   /* a CUDA call failed                                                    */
};

/* Workload description (everything the paper leaves to the experiment). Standard deviations,
 * not variances. Applying it re-creates the whole state from the seed. */
typedef struct {
  int32_t objective;     /* SWARM_OBJ_*                                                           */
  int32_t nonblocking;   /* 1: keep base snapshots B and allow SWARM_NONBLOCKING; 2: also keep the nodes'
                            own registers (16 bits per coordinate) and allow SWARM_REGISTERS       */
  float   init_std;      /* X^i[k] = init_std * z + o_i                                           */
  float   offset_std;    /* per-node scalar o_i ~ N(0, offset_std^2)                              */
  float   grad_std;      /* SYNTH: stochastic gradient = c_i + grad_std * z                       */
  float   drift_std;     /* SYNTH: per-node scalar c_i ~ N(0, drift_std^2) (non-IID term)         */
  int32_t lsq_m;         /* LSQ: rows of each data matrix                                         */
  int32_t lsq_batch;     /* LSQ: minibatch size (rows drawn uniformly with replacement)           */
  int32_t lsq_dtype;     /* LSQ: SWARM_F32 or SWARM_BF16 storage of the data matrices             */
  int32_t lsq_groups;    /* LSQ: number of data matrices; 0 = one per node, else must divide n    */
  float   lsq_noise_std; /* LSQ: label noise; labels = A x* + mu_i + noise, mu_i ~ U(-1, 1).
                            SWARM_OBJ_LOGISTIC uses the same lsq_* fields: logistic regression on the same data
                            with class labels 1[A x* + mu_i + noise > 0], gradient (sigmoid(a.x) - y) a      */
} swarm_config;

/* Optional device allocator (e.g. a framework's caching allocator). Must be installed before
 * swarm_init; applies to contexts created afterwards. alloc returns NULL on failure. */
typedef void *(*swarm_alloc_fn)(size_t bytes, void *user);
typedef void (*swarm_free_fn)(void *ptr, void *user);
int swarm_set_allocator(swarm_alloc_fn alloc_fn, swarm_free_fn free_fn, void *user);

/* ------------------------------------------------------------------------------------------
 * The five core calls
 * ---------------------------------------------------------------------------------------- */

/* Section 2 / Section 3: create n >= 2 node models of dimension d >= 1 on graph `topo`, with
 * the counter-based generator keyed by `seed`. Defaults: init_std = 0.1, no objective, no base
 * snapshots (see swarm_configure). *out receives the context (caller destroys it).
 * Errors: EINVAL (n, d, topology; regular graph not constructible), ENOMEM, ECUDA. */
int swarm_init(swarm_ctx **out, int32_t n, int64_t d, swarm_topology topo, uint64_t seed);

/* Section 3, "The Communication Procedure": each listed node takes H sequential stochastic
 * gradient steps of size lr on its own objective, every gradient evaluated at the running
 * iterate (\tilde h^q = \tilde g_i(X - sum_{s<q} lr \tilde h^s)); the steps are applied in
 * place to X^i. node_ids_host: `count` distinct ids (host). H >= 0.
 * Least squares and logistic regression on bf16 data with minibatches of at most 64 rows: the rows of a
 * node's next steps are known in advance and a step moves the model along its sampled rows only, so up to
 * four consecutive steps are evaluated from one pass over the model (their scores <a, x> against the model
 * before the first of them, corrected step by step with inner products of data rows, which the library keeps
 * as the data matrices' Gram matrices when these take at most 256 MiB) and applied in one pass. The iterates
 * are the same sequential ones; the model is rounded to fp32 once per group instead of once per step.
 * Errors: ESTATE (no objective), EINVAL (H < 0, count < 0, duplicate id), ERANGE. */
int swarm_local_steps(swarm_ctx *ctx, const int32_t *node_ids_host, int32_t count, int32_t H, float lr);

/* Section 3, "Sequential model": as swarm_local_steps, but every listed node takes a geometric number
 * of steps with mean mean_H (the analysis' stand-in for Poisson-clock activation; E[H_i^2] = 2H^2 - H).
 * The count of node i is the index of the first success in Bernoulli(1/mean_H) trials drawn from the
 * counter-based generator (stream 11, row i, event = the node's step counter), capped at 1024.
 * out_steps_host (may be NULL) receives the `count` step counts.
 * Errors: as swarm_local_steps; EINVAL for mean_H < 1. */
int swarm_local_steps_geometric(swarm_ctx *ctx, const int32_t *node_ids_host, int32_t count, int32_t mean_H, float lr,
                                int32_t *out_steps_host);

/* Algorithm 1, interaction lines; Corollary 1 for Enc/Dec. `pairs_host` holds npairs disjoint
 * directed edges of G. bits in {2, ..., 8}: lattice quantizer with that many bits per
 * coordinate (one bit leaves no decoding window: L = 2^(b-1) - 1 = 0); bits = 32 (blocking only):
 * identity quantizer (Corollary 2).
 *   SWARM_BLOCKING: per 1024-block the common exponent e is taken from the exact range of
 *     X^a - X^b; both models are encoded into their own buffers, each side decodes the
 *     partner's buffer with its own model as key, and both adopt Q(X^a)/2 + Q(X^b)/2.
 *   SWARM_NONBLOCKING: the initiator decodes its own and the responder's buffer with its base
 *     snapshot as key, averages, subtracts its pending local update B^a - X^a, adopts the
 *     result as model and snapshot, and writes Enc(new model) to its own buffer and Enc(average)
 *     to the responder's; the responder's model is not touched. Buffers are (re)published from
 *     the snapshots first if they do not hold `bits`-bit codes or a blocking call intervened.
 *   SWARM_REGISTERS: the two-register protocol of Section 3 ("The Communication Registers") with
 *     Algorithm 1's chain of three decodes. Each node has an own register (16-bit encoding of its
 *     snapshot, written only by the node, with the step of an 8-bit code of the guard distance) and a
 *     current register (b-bit, written by its last interaction partner, scaled by the exact distance to
 *     its decoding key). The initiator a computes Q(X^a) = Dec(B^a, own_a), Q(X_a) = Dec(Q(X^a), cur_a),
 *     Q(X^b) = Dec(B^a, own_b), Q(X_b) = Dec(Q(X^b), cur_b), adopts Q(X_a)/2 + Q(X_b)/2 - (B^a - X^a) as
 *     model and snapshot, rewrites both of its registers and writes Enc(average) to cur_b. Registers are
 *     (re)initialised from the snapshots first when they are not in this convention at `bits` bits.
 * Every call advances the staleness clocks: interactions of a launch are taken in list order, each
 * resets its initiator's clock and ages all other nodes by one. The pairs of a launch are disjoint, so the order
 * in which the device works through them does not show in any result; the library chooses it (launches walk
 * their pairs from alternating ends, most recently visited rows first, for the sake of the L2 cache).
 * Errors: EINVAL (bits, mode, npairs < 0, NULL), ERANGE, EPAIR, ESTATE. */
int swarm_interact(swarm_ctx *ctx, const swarm_pair *pairs_host, int32_t npairs, int32_t bits, int32_t mode);

/* Algorithm 1, one whole step of a launch: the initiator of every pair (and its responder when
 * step_responders != 0) takes H local steps with learning rate lr, then the pairs interact. Same
 * results, bit for bit, as swarm_local_steps on those nodes followed by swarm_interact(pairs, bits, mode).
 * With SWARM_OBJ_SYNTH and a blocking or single-buffer exchange the steps run inside the interaction kernel, so
 * the models make one trip through HBM instead of two and the launch is one kernel; with the two-register
 * exchange, and with the least-squares objectives, whose gradient couples all coordinates of a model, the
 * library runs the two calls in sequence. H = 0 is swarm_interact.
 * Errors: those of the two calls; a refused call leaves the models untouched. */
int swarm_step(swarm_ctx *ctx, const swarm_pair *pairs_host, int32_t npairs, int32_t H, float lr, int32_t bits,
               int32_t mode, int32_t step_responders);

/* Section 3, "Sequential model": nsteps interactions one after the other, pairs_host[t] being the pair of
 * time step t (consecutive pairs may share nodes). Same results, bit for bit, as
 *     for t: swarm_step(ctx, &pairs_host[t], 1, H, lr, bits, SWARM_BLOCKING, step_responders).
 * For short models (row pitch <= 8192) with fp32 least-squares or logistic data and a minibatch of at most
 * 32 rows the whole sequence runs in ONE kernel launch (a thread-block cluster walks the steps; launch
 * latency, which dominates such steps, is paid once per 64 steps or more); otherwise the library issues the
 * steps one by one. Refused (ESTATE) while staleness tracking is on, like every blocking exchange.
 * Errors: EINVAL (nsteps < 0, H < 0, bits, NULL), ERANGE, EPAIR (a pair that is not an edge), ESTATE; all pairs
 * are checked before anything runs. */
int swarm_run_sequence(swarm_ctx *ctx, const swarm_pair *pairs_host, int32_t nsteps, int32_t H, float lr,
                       int32_t bits, int32_t step_responders);

/* Section 4: mu = (1/n) sum_i X^i, written to out_dev (d floats, device memory). */
int swarm_mean_model(swarm_ctx *ctx, float *out_dev);

/* Section 4: Gamma = sum_i ||X^i - mu||^2, written to *out_gamma_host. Synchronises. */
int swarm_potential(swarm_ctx *ctx, double *out_gamma_host);

/* Appendix, "Notation and Auxiliary Potential Functions": the potentials that the analysis uses to
 * control outdated models. With X^_i = X_{t - tau_i} the snapshot B_i of node i (its model right after
 * its last initiation) and m_i the mean model recorded at that moment,
 *     Gamma^_t = sum_i ||X^_i - mu_t||^2,   A_t = sum_i ||X^_i - m_i||^2,   B_t = sum_i ||mu_t - m_i||^2,
 * and Gamma^_t <= 2 A_t + 2 B_t. mu is the fp32 mean model that swarm_mean_model produces; sums in fp64.
 * swarm_track_staleness(ctx, 1) allocates the records (n * pitch floats of device memory), treats every
 * node as having initiated just now (records = current mean, clocks tau = 0) and makes every later
 * non-blocking or register interaction update the records of its initiators; the interactions of one
 * launch count as simultaneous: all its initiators record the mean model after the launch (one extra
 * pass over the n models per launch). enable = 0 frees the records.
 * Errors: ESTATE (configuration without snapshots, snapshots stale after a blocking exchange), ENOMEM.
 * While tracking is on, swarm_interact in SWARM_BLOCKING mode returns ESTATE. */
int swarm_track_staleness(swarm_ctx *ctx, int32_t enable);
/* out3_host receives Gamma^_t, A_t, B_t. Synchronises. ESTATE unless tracking is on. */
int swarm_aux_potentials(swarm_ctx *ctx, double *out3_host);

/* ------------------------------------------------------------------------------------------
 * Auxiliary calls
 * ---------------------------------------------------------------------------------------- */

/* Apply a workload description and rebuild the state from the seed (models, per-node scalars,
 * data, counters). The buffers of the previous configuration are released first. If the new ones cannot be
 * allocated the call returns ENOMEM and leaves the context in the default configuration of swarm_init (no
 * objective, no snapshots, init_std = 0.1, state rebuilt from the seed), never with a configuration whose
 * buffers are missing. Errors: EINVAL (nothing changed), ENOMEM, ECUDA. */
int swarm_configure(swarm_ctx *ctx, const swarm_config *cfg_host);

/* Algorithm 1, sampling lines: draw up to max_pairs disjoint pairs for the next launch
 * (initiator uniform over nodes, responder uniform over its neighbours, draws that touch an
 * already paired node rejected, at most 16*max_pairs draws). Runs on the device, synchronises,
 * advances the launch counter. out_pairs_host has room for max_pairs entries. */
int swarm_sample_pairs(swarm_ctx *ctx, int32_t max_pairs, swarm_pair *out_pairs_host, int32_t *out_count_host);

/* Fill all communication buffers with `bits`-bit encodings of the base snapshots (see
 * swarm_interact, SWARM_NONBLOCKING). Errors: ESTATE without base snapshots, EINVAL. */
int swarm_publish(swarm_ctx *ctx, int32_t bits);

/* Initialise both registers of every node from the snapshots (see swarm_interact, SWARM_REGISTERS).
 * Errors: ESTATE unless configured with nonblocking = 2, EINVAL. */
int swarm_register_publish(swarm_ctx *ctx, int32_t bits);

/* Corollary 1, second case, and "Counting Communication Cost": the long code lives in the writer's own
 * register and a reader consumes only a prefix sized by its distance to the encoded vector. The b-bit
 * colour of a lattice point is the low b bits of its 16-bit colour, and the register keeps the low bytes of
 * a block before the high bytes, so a reader with `bits` = 8 reads the first half of its partner's own
 * register only; correct while its snapshot is within 127 register steps of the partner's (partners that
 * keep meeting are; a distant third node needs 16). Beyond that the decode aliases by multiples of 256
 * steps (defined behaviour, as for every decode outside its window). Default 16; every swarm_configure
 * resets it. A node decoding its own register always uses the 8-bit prefix (its key is the encoded
 * snapshot itself). Errors: EINVAL (bits not 8 or 16), ESTATE (configuration without own registers). */
int swarm_set_own_prefix(swarm_ctx *ctx, int32_t bits);
int swarm_get_own_prefix(swarm_ctx *ctx, int32_t *bits_host);

/* The same passages, per reader: swarm_interact in SWARM_REGISTERS mode in which the initiator of
 * pairs_host[p] reads prefixes_host[p] bits (8 or 16) of its responder's own register, whatever
 * swarm_set_own_prefix says (that setting is the prefix of every pair of a plain swarm_interact). A launch can
 * thus mix partners that keep meeting (8 bits: half of the partner's own register crosses the memory system)
 * with a reader whose snapshot is far from its partner's (16 bits). The prefix is the reader's statement about
 * its distance; the construction has no check value, so a prefix that is too short aliases (defined
 * behaviour, see swarm_set_own_prefix). prefixes_host: npairs int32 values, host memory, read during the call.
 * Errors: those of swarm_interact; EINVAL for a prefix other than 8 or 16 or a NULL list with npairs > 0. */
int swarm_interact_prefixed(swarm_ctx *ctx, const swarm_pair *pairs_host, const int32_t *prefixes_host,
                            int32_t npairs, int32_t bits);

/* State access (checkpointing, test injection). `which` selects the array, `node` the row
 * (ignored for whole-context arrays). bytes must equal the row size exactly. Both synchronise. */
enum {
  SWARM_T_X = 0,        /* d floats                                  */
  SWARM_T_B = 1,        /* d floats (ESTATE without snapshots)       */
  SWARM_T_CODES = 2,    /* nblk*1024 bytes                           */
  SWARM_T_EXPS = 3,     /* nblk int8                                 */
  SWARM_T_ADJ = 4,      /* degree int32 (read-only)                  */
  SWARM_T_A = 5,        /* node = data-matrix id; lsq_m*d floats (bf16 storage is widened/rounded) */
  SWARM_T_BVEC = 6,     /* lsq_m floats                              */
  SWARM_T_XSTAR = 7,    /* d floats, node ignored                    */
  SWARM_T_SCALARS = 8,  /* 3 floats: offset o_i, drift c_i, shift mu_i */
  SWARM_T_COUNTERS = 9, /* 3 uint32: buffer write counter, local-step counter, code width of the buffer */
  SWARM_T_OWN = 10,     /* nblk*2048 bytes: own register, per block 1024 low bytes then 1024 high bytes of
                           the 16-bit colours (ESTATE unless nonblocking = 2)                               */
  SWARM_T_OEXPS = 11,   /* nblk int8: exponents of the own register                                         */
  SWARM_T_CLOCKS = 12,  /* 2 uint32: write counter of the own register, staleness clock tau                 */
  SWARM_T_MU_RECORD = 13, /* d floats: mean model at the node's last initiation (ESTATE unless tracking)    */
  SWARM_T_A_RECORD = 14,  /* 1 double: ||snapshot - mean||^2 at the node's last initiation                  */
  SWARM_T_GRAM = 15       /* node = data-matrix id; lsq_m*lsq_m floats: the matrix's Gram matrix A A^T, kept for the
                             local steps that are evaluated several at a time (read-only; ESTATE when not kept) */
};
int swarm_get_tensor(swarm_ctx *ctx, int32_t which, int32_t node, void *dst_host, size_t bytes);
/* The same read queued on the context's stream without waiting: dst_host (any host memory, which must stay
 * valid until then) holds the row once swarm_sync, or any other synchronising call issued later (swarm_potential,
 * swarm_get_tensor, swarm_sample_pairs, ...), returns. For callers that consume a result of every step without
 * stalling the launch pipeline. Only rows kept in device memory: EINVAL for SWARM_T_ADJ, SWARM_T_COUNTERS,
 * SWARM_T_CLOCKS, SWARM_T_A. Rows of up to 64 KiB are copied at once, by a small kernel, into a 1 MiB ring inside
 * the context (the row's value is the one at this point of the stream) and travel to the host in one transfer
 * at that later call; when the ring is full the call itself synchronises first. Longer rows are copied by the
 * copy engine straight to dst_host (pinned memory, or that copy is not asynchronous). */
int swarm_get_tensor_async(swarm_ctx *ctx, int32_t which, int32_t node, void *dst_host, size_t bytes);
int swarm_set_tensor(swarm_ctx *ctx, int32_t which, int32_t node, const void *src_host, size_t bytes);
/* Rows row0 .. row0 + nrows - 1 of least-squares data matrix `matrix` as floats (bf16 storage is widened), nrows * d
 * floats into dst_host; a whole matrix (SWARM_T_A) can be gigabytes. bytes must equal nrows * d * 4. Synchronises.
 * Errors: ESTATE (no least-squares data), ERANGE (matrix, rows), EINVAL. */
int swarm_get_data_rows(swarm_ctx *ctx, int32_t matrix, int32_t row0, int32_t nrows, float *dst_host, size_t bytes);

/* Whole-context counters: launch counter of the pair sampler and the "snapshots stale" flag. */
int swarm_get_state(swarm_ctx *ctx, uint32_t *launch_host, int32_t *b_stale_host);
int swarm_set_state(swarm_ctx *ctx, uint32_t launch, int32_t b_stale);
/* Convention the communication buffers were last written in: 0 none / blocking, 1 single buffer
 * (SWARM_NONBLOCKING), 2 registers (SWARM_REGISTERS). */
int swarm_get_buffer_mode(swarm_ctx *ctx, int32_t *mode_host);
int swarm_set_buffer_mode(swarm_ctx *ctx, int32_t mode);

/* Device pointer and row pitch (in elements) of X, for callers that consume models in place.
 * Valid until the next swarm_configure / swarm_destroy. */
int swarm_model_ptr(swarm_ctx *ctx, float **x_dev, int64_t *pitch);

/* Potential of caller-held models with no allocation of any kind (the paper has no counterpart: this
 * exists for callers that are not allowed to allocate). Meant for code that owns all its device memory
 * up front -- a process with a fixed memory pool, a hook running inside another component's step, a host
 * framework that passes only raw pointers -- and therefore cannot create a context (contexts allocate
 * their scratch) or tolerate cudaMalloc's device-wide synchronisation and late failure.
 *   x_dev          n rows of d floats, row i at x_dev + i*pitch (device memory, read only; pitch >= d,
 *                  in elements; when x_dev is 16-byte aligned and pitch a multiple of 4 every row is, and the
 *                  rows are read with 128-bit loads; any other float-aligned base or pitch is read element by element)
 *   out_gamma_dev  one double in device memory, written asynchronously on cuda_stream
 *   cuda_stream    cudaStream_t (NULL = default stream) on the current device
 * Gamma = sum_i ||X^i - mu||^2 as in swarm_potential, same arithmetic. The per-CTA partial sums live in a
 * fixed 512 KiB array inside the library image (every GPU that loads the library holds it until the
 * process exits), which caps the size: d <= SWARM_STATIC_MAX_D, otherwise SWARM_EINVAL and nothing is
 * launched. All calls share that array: calls on one stream are ordered and safe, calls that may overlap
 * on the same GPU race on it. The first call made with a given device current looks up the array's
 * device address (no allocation); make that first call before starting any stream capture.
 * Errors: EINVAL (NULL pointer, x_dev not 4-byte or out_gamma_dev not 8-byte aligned, n < 2, d < 1, pitch < d,
 * d > SWARM_STATIC_MAX_D), ECUDA. */
#define SWARM_STATIC_MAX_D 33554432
int swarm_potential_static(const float *x_dev, int32_t n, int64_t d, int64_t pitch, double *out_gamma_dev,
                           void *cuda_stream);

int swarm_set_stream(swarm_ctx *ctx, void *cuda_stream);   /* cudaStream_t; NULL = default stream */
int swarm_sync(swarm_ctx *ctx);
/* Failure detection (the paper has no counterpart): the number of polls after which a device-side wait gives
 * up (see "Device-side waits are bounded" above). polls < 0 restores the default (2^22 polls; one poll may
 * itself block for a hardware-defined time, so this is seconds). polls = 0 makes every such wait give up at
 * once, which is how the error path is exercised on a healthy GPU without faulting or hanging it: the
 * kernel still waits, bounded by the default, for its own tensor-core work before it releases tensor memory.
 * Errors: EINVAL (NULL, polls >= 2^32). */
int swarm_set_wait_limit(swarm_ctx *ctx, int64_t polls);
int64_t swarm_kernel_launches(swarm_ctx *ctx);             /* kernels launched so far by this context */
int swarm_last_cuda_error(swarm_ctx *ctx);                 /* cudaError_t of the last SWARM_ECUDA       */
const char *swarm_strerror(int code);
void swarm_destroy(swarm_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* SWARM_B200_H */
