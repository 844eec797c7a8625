/*
 * signmuon.h - C ABI of the SignMuon optimizer step for NVIDIA B200 (sm_100a).
 *
 * One object computes, for M data-parallel workers held on one GPU as a batch
 * axis, the step of Alg. 2 / Alg. 3 of the SignMuon paper:
 *
 *   per worker m:   G~ = G_m + lambda W                      (weight decay)
 *                   Mom_m <- beta Mom_m + (1 - beta) G~       (momentum)
 *                   U_m = PolarNS(Mom_m; K, eps, fro)         (Alg. 4)
 *                   B_m = PackBits(sign(U_m))                 (>= 0 -> 1, < 0 -> 0)
 *   shared:         S = sign(sum_m S_m) = sign(2 c - M)       (majority vote, ties -> +1;
 *                                                              c = popcount over workers)
 *                   D = S, or S / sqrt(rows cols) (Eq. 2), or PolarNS(S) (local polar step)
 *                   W <- W - eta D
 *
 * The sum all-reduce / all-gather of the paper is replaced by an on-device
 * reduction over the worker axis; there is no collective.
 *
 * Conventions
 *   - Every pointer is tagged HOST or DEVICE below.  Device pointers must be
 *     16-byte aligned.  All matrices are row-major and contiguous.
 *   - The library allocates no device memory: the caller provides the state
 *     buffer (momenta; persistent across steps) and the workspace (scratch;
 *     contents meaningful only between a step and the next one).
 *   - signmuon_step only enqueues work on the given stream and never
 *     synchronises.  One context must not be used from two streams at once.
 *   - Every function returns SIGNMUON_OK (0) or a negative error code; nothing
 *     throws, aborts or prints.
 *
 * Packed payload format (App. B, "Packed 1-bit representation"; Alg. 3 note):
 *   parameters are concatenated in creation order, each padded to a 32-bit
 *   word; entry i of a parameter (flat row-major index) is bit (i & 31) of word
 *   (i >> 5), i.e. bit (i & 7) of byte (i >> 3); 1 <-> +1, 0 <-> -1; pad bits
 *   are 0.  One worker's payload is 4 * sum_p ceil(d_p / 32) bytes
 *   (= ceil(d / 8) when every d_p is a multiple of 32): one bit per entry,
 *   1/32 of a float32 gradient.
 */
#ifndef SIGNMUON_H_
#define SIGNMUON_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct signmuon_ctx signmuon_ctx;   /* opaque host object */

enum {
  SIGNMUON_OK = 0,
  SIGNMUON_ERR_INVALID_ARG = -1,      /* null pointer, out-of-range scalar */
  SIGNMUON_ERR_BAD_SHAPE = -2,        /* rows/cols < 1 or too large */
  SIGNMUON_ERR_NOT_BOUND = -3,        /* step/payload before signmuon_bind */
  SIGNMUON_ERR_BUFFER_TOO_SMALL = -4, /* state/workspace smaller than signmuon_state_bytes says */
  SIGNMUON_ERR_CUDA = -5,             /* a CUDA call or launch failed (sticky) */
  SIGNMUON_ERR_TIMEOUT = -6,          /* a bounded device-side wait ran out (see signmuon_status) */
  SIGNMUON_ERR_UNSUPPORTED_ARCH = -7, /* current device is not compute capability 10.x */
  SIGNMUON_ERR_MISALIGNED = -8,       /* a device pointer is not 16-byte aligned */
  SIGNMUON_ERR_TOO_LARGE = -9,        /* problem exceeds a fixed capacity (signmuon_momentum_norm_noalloc) */
  SIGNMUON_ERR_NO_MEMORY = -10        /* a host allocation (context, pinned table mirror) failed */
};

typedef enum { SIGNMUON_F32 = 0, SIGNMUON_BF16 = 1 } signmuon_dtype;

typedef enum {
  SIGNMUON_PARAM_MATRIX = 0, /* Newton-Schulz path (Alg. 2 with Alg. 4) */
  SIGNMUON_PARAM_PLAIN = 1   /* vector-like parameter: sign of the momentum, no Newton-Schulz
                                (App. B treats vectors as m x n with one dimension 1, for which
                                PolarNS keeps every sign) */
} signmuon_kind;

typedef struct {
  int64_t rows, cols;          /* conv weights arrive reshaped to out x (in*kh*kw) */
  int32_t kind;                /* signmuon_kind */
  int32_t weight_dtype;        /* signmuon_dtype of W */
  int32_t grad_dtype;          /* signmuon_dtype of G */
} signmuon_param;

typedef struct {
  int32_t num_params;
  const signmuon_param* params; /* HOST, copied by signmuon_create */
  int32_t num_workers;          /* M >= 1 (at most 255): the workers that vote */
  float momentum;               /* beta in [0, 1)                       (Alg. 1 input) */
  float lr;                     /* eta; signmuon_step may override it per call */
  int32_t ns_steps;             /* K >= 0; K = 0 gives the sign of the momentum */
  int32_t local_polar;          /* 0/1: D = PolarNS(S) after the vote (Sec. 3, "Sign-Muon update") */
  float weight_decay;           /* lambda >= 0, coupled: G~ = G + lambda W */
  float eps;                    /* Alg. 4 stability constant; <= 0 selects 1e-12 */
  int32_t update_scale;         /* 0: W -= eta S (Alg. 2)   1: W -= eta S / sqrt(rows cols) (Eq. 2) */
  int32_t flags;                /* SIGNMUON_FLAG_* */
  int32_t ns_scale;             /* Alg. 4 "scale" of the workers' PolarNS: SIGNMUON_SCALE_FRO (sigma = ||Mom||_F) or
                                   SIGNMUON_SCALE_SPECTRAL (sigma = PowerIter(Mom, power_iters, eps), Alg. 5).  The
                                   local polar step always uses ||S||_F = sqrt(rows cols). */
  int32_t power_iters;          /* P of Alg. 5, 0..64 (the paper's experiments use 2); ignored for SCALE_FRO */
  /* Worker sharding (Alg. 2 / Alg. 3 with the workers spread over several GPUs).  local_workers == 0: this
   * context computes all num_workers workers (one GPU simulates them all).  local_workers > 0: it computes
   * workers [worker_offset, worker_offset + local_workers) only - state, gradients and Newton-Schulz buffers
   * cover those workers, gradients arrive as [local_workers][rows][cols] - while the payload buffer still has
   * one row per worker of the job; the rows of the other workers are filled by the exchange (all-gather of the
   * packed words, Alg. 3) before the vote stage. */
  int32_t worker_offset;
  int32_t local_workers;
  int32_t update_rule;          /* SIGNMUON_RULE_* */
} signmuon_config;

/* Update rules.  SIGNMUON: Alg. 2 / Alg. 3.  MUON: the full-precision comparison optimizer of Sec. 5.1 on the same
 * kernels - Alg. 1 without the sign line, data-parallel with float gradient averaging: matrix parameters keep ONE
 * momentum of the workers' mean gradient (state [1][d]), U = PolarNS(Mom), W <- W - eta U; nothing is packed or voted
 * for them and local_polar is ignored.  Plain parameters keep the majority-vote sign update (which is also what a
 * majority-vote SignAdam would apply: the sign of Adam's direction is the sign of its first moment).  MUON cannot
 * be combined with worker sharding (average the gradients across GPUs first and pass num_workers = 1) and needs
 * ns_steps >= 1 (the update is applied by the last Newton-Schulz epilogue). */
enum { SIGNMUON_RULE_SIGNMUON = 0, SIGNMUON_RULE_MUON = 1 };

enum { SIGNMUON_SCALE_FRO = 0, SIGNMUON_SCALE_SPECTRAL = 1 };

enum {
  SIGNMUON_FLAG_KEEP_POLAR = 1,   /* also store U_m = Y_K (bf16) so that signmuon_debug_tap can return it */
  SIGNMUON_FLAG_SIMT_GEMM = 2,    /* diagnostic: run the Newton-Schulz products on a plain CUDA-core
                                     kernel instead of the tensor-core kernel (slow; for fault isolation) */
  SIGNMUON_FLAG_GEMM_1CTA = 4,    /* run the tensor-core kernel with one CTA per 128 x 128 tile instead of
                                     CTA pairs on 256 x 256 tiles (same results; for comparison) */
  SIGNMUON_FLAG_LP_GRAM_BF16 = 32, /* run the first Gram product of the local polar step on the bf16 copy of the vote
                                     matrix instead of its FP8 (E4M3) copy (same result bit for bit; for comparison) */
  SIGNMUON_FLAG_NO_GRAM_SPACE = 64, /* run every Newton-Schulz iteration on the full matrix, also for the parameters
                                     whose iteration otherwise runs on their s x s Gram matrix (Alg. 4's loop evaluated
                                     as A_{k+1} = P_k A_k P_k, Y_K = (P_{K-1} ... P_0) Y_0: short sides up to 256 on
                                     chip; longer short sides of matrices at least 1.5 times as long as a chain of
                                     symmetric products through memory, when they hold 8 M (entry, worker) pairs
                                     together; same map, two passes over the matrix instead of 2 K; for comparison) */
  SIGNMUON_FLAG_SIGN_AGREEMENT = 16 /* count, every step, how many of each worker's sign bits equal the vote
                                     (one more small kernel; read with signmuon_sign_agreement) */
};

/* Stages of one step, for signmuon_run_stages (bit mask). A full step is all of them in this order. */
enum {
  SIGNMUON_STAGE_MOMENTUM = 1,    /* weight decay, momentum, Frobenius norms, plain-parameter update */
  SIGNMUON_STAGE_NS = 2,          /* K Newton-Schulz iterations per worker, sign + pack */
  SIGNMUON_STAGE_VOTE = 4,        /* majority vote (+ weight update when local polar is off) */
  SIGNMUON_STAGE_LOCAL_POLAR = 8, /* PolarNS of the vote matrix + weight update (local polar on) */
  SIGNMUON_STAGE_ALL = 15
};

/* What signmuon_debug_tap can return. */
enum {
  SIGNMUON_TAP_MOMENTUM = 0,   /* float32 [rows*cols] of (param, worker) */
  SIGNMUON_TAP_POLAR = 1,      /* bf16 [rows][ld] Y_K of (param, worker); needs SIGNMUON_FLAG_KEEP_POLAR */
  SIGNMUON_TAP_VOTE_BITS = 2,  /* uint32 words of the vote of a param (worker ignored) */
  SIGNMUON_TAP_WORKER_BITS = 3,/* uint32 words of (param, worker) inside the payload */
  SIGNMUON_TAP_NORM = 4        /* float32 [2]: 1/max(sigma,eps)^2 and 1/max(sigma,eps) of (param, worker) */
};

/* Creates a context from a HOST config (Alg. 2 "Input"). Touches no GPU.
 * Errors: INVALID_ARG (null, M outside [1,255], beta outside [0,1), K < 0, lambda < 0,
 * unknown enum), BAD_SHAPE (a side < 1 or > 2^24, more than 2^36 entries, a matrix parameter whose longer side
 * exceeds 128 * 65535), NO_MEMORY. On error *out is set to NULL. */
int signmuon_create(const signmuon_config* config, signmuon_ctx** out);

/* Bytes the caller must provide: `state` = momenta of all workers (float32 [M][d] per parameter,
 * parameters in creation order) - the only persistent optimizer state; `workspace` = scratch
 * (bf16 Newton-Schulz operands, Gram matrices, packed bits, norms, tile tables);
 * `host_staging` = extra device bytes needed only by signmuon_step_host: the weights once and the gradients
 * twice (may be queried as NULL). */
int signmuon_state_bytes(const signmuon_ctx* ctx, size_t* state, size_t* workspace, size_t* host_staging);

/* Attaches DEVICE buffers (owned by the caller, must outlive the context's use of them) and
 * prepares the device-side tables on `cuda_stream` (a cudaStream_t, NULL = legacy default stream).
 * `zero_state` != 0 clears the momenta (Mom_0 = 0); pass 0 when restoring a checkpointed state.
 * `dev_staging` may be NULL when signmuon_step_host is not used.
 * Also allocates (once per context) a few KB of pinned HOST memory that mirrors the parameter tables.
 * Errors: BUFFER_TOO_SMALL, MISALIGNED, UNSUPPORTED_ARCH, NO_MEMORY, CUDA. */
int signmuon_bind(signmuon_ctx* ctx, void* dev_state, size_t state_bytes, void* dev_workspace,
                  size_t workspace_bytes, void* dev_staging, size_t staging_bytes, int zero_state,
                  void* cuda_stream);

/* One optimizer step (Alg. 2 / Alg. 3 loop body) enqueued on `cuda_stream`.
 *   weights: HOST array of num_params DEVICE pointers, W_p [rows][cols] in weight_dtype, updated in place
 *   grads:   HOST array of num_params DEVICE pointers, G_p [M][rows][cols] in grad_dtype (worker-major), read only
 *   lr:      eta_t for this step; a negative value selects config.lr
 * The device keeps the pointer tables of the last four distinct (weights, grads) pointer sets: a call with a
 * set seen before uploads nothing; a new set costs one small asynchronous copy from pinned memory.
 * A context that computes only a subset of the workers (config.local_workers) cannot run the step in one call:
 * the payload exchange sits between the stages; signmuon_step then returns INVALID_ARG - use
 * signmuon_run_stages(MOMENTUM | NS), exchange, signmuon_run_stages(VOTE | LOCAL_POLAR) or signmuon_vote_update.
 * Errors: NOT_BOUND, INVALID_ARG, MISALIGNED, CUDA (sticky launch error). */
int signmuon_step(signmuon_ctx* ctx, void* const* weights, const void* const* grads, float lr,
                  void* cuda_stream);

/* Same step, restricted to the stages in `stage_mask` (SIGNMUON_STAGE_*), run in step order.
 * Lets a caller time or inspect the stages separately; running all stages in order over
 * several calls equals one signmuon_step. */
int signmuon_run_stages(signmuon_ctx* ctx, int32_t stage_mask, void* const* weights,
                        const void* const* grads, float lr, void* cuda_stream);

/* Same step with HOST-resident weights and gradients (same layouts as signmuon_step, but HOST
 * pointers inside the HOST arrays; pinned memory recommended): copies them to the staging buffer
 * bound by signmuon_bind, runs the step, copies the weights back, without synchronising the host.
 * The gradients travel on a stream of the library's own into one of two staging sets, so that, when calls follow
 * one another without a synchronisation in between, the gradient copy of a call overlaps the compute and the weight
 * copy-back of the call before it.  The weights are copied back on `cuda_stream` at the end of the step.  Their
 * upload goes first on `cuda_stream` when something before the vote stage needs them (plain parameters, coupled
 * weight decay, the Muon rule); otherwise it follows the gradients on the library's stream, ordered behind the
 * previous call's copy-back to the same host arrays, and only the vote stage waits for it.  As with any
 * asynchronous copy, the host arrays of a call must stay unchanged until that call's work has run: synchronise
 * `cuda_stream` (its work waits for both uploads) before changing them.  signmuon_bind creates that stream and
 * five events when a staging buffer is given; signmuon_destroy releases them.
 * Errors as signmuon_step, plus NOT_BOUND when no staging was bound. */
int signmuon_step_host(signmuon_ctx* ctx, void* const* host_weights, const void* const* host_grads,
                       float lr, void* cuda_stream);

/* The bytes worker `worker` would transmit for the last step (Alg. 3 "PackBits"; App. B s_1):
 * DEVICE pointer into the workspace (valid until the next step), its size in bytes and the
 * number of sign entries it carries.  May be called before bind with dev_ptr == NULL to get sizes. */
int signmuon_packed_payload(const signmuon_ctx* ctx, int32_t worker, const uint32_t** dev_ptr,
                            size_t* bytes, size_t* entries);

/* The gathered payload buffer (Alg. 3: "all-gather of B^(m)", App. B "Majority vote from gathered bits"): DEVICE
 * pointer to row 0, the distance between two workers' rows in bytes (a multiple of 128) and the number of rows
 * (num_workers).  Row m holds worker m's payload (signmuon_packed_payload(m)).  A context that computes a subset of
 * the workers writes its own rows in the Newton-Schulz stage; an exchange may write the other rows directly here
 * (e.g. an in-place all-gather when every rank owns the same number of consecutive workers) before the vote stage
 * runs.  Valid from signmuon_bind on; dev_ptr may be NULL to query the sizes only. */
int signmuon_payload_buffer(const signmuon_ctx* ctx, uint32_t** dev_ptr, size_t* row_pitch_bytes, int32_t* rows);

/* Majority vote, optional local polar step and weight update from gathered payloads (Alg. 3 after the all-gather;
 * Eq. 1): `payloads` is a HOST array of num_workers DEVICE pointers; entry m is worker m's packed payload
 * (signmuon_packed_payload's size and format), or NULL to use what row m of the payload buffer already holds (the
 * context's own workers, or rows an exchange wrote in place).  Non-NULL entries are copied into the payload buffer
 * on `cuda_stream` first.  Then runs the VOTE and LOCAL_POLAR stages: identical results on every GPU that
 * holds the same payloads and weights.  `grads` is not read by these stages and may repeat the pointers of the
 * preceding signmuon_run_stages call (it only selects the pointer table).
 * Errors: as signmuon_run_stages. */
int signmuon_vote_update(signmuon_ctx* ctx, const uint32_t* const* payloads, void* const* weights,
                         const void* const* grads, float lr, void* cuda_stream);

/* The exchange fused into the pack (Alg. 3's all-gather without a separate collective): after this call every
 * payload word this context packs - in the last Newton-Schulz epilogue, in the stand-alone pack kernel and in the
 * plain-parameter kernel - is stored not only into its own payload buffer but also, at the same offset, into the
 * payload buffer of every peer (plain stores into peer-mapped memory: NVLink peer access, CUDA IPC or any mapping
 * that makes the peer's buffer addressable from this GPU).  The stage that packs ends with a small kernel that
 * publishes the step's sequence number into slot `my_rank` of every peer's flag array; the vote stage starts with
 * a kernel that waits (bounded by the wait limit; TIMEOUT in the status word when it runs out) until every other
 * rank's slot of this context's own flag array has reached it.  All ranks must call the stages in lockstep.
 *   my_rank, num_ranks     this context's rank and the number of ranks (<= 64)
 *   num_peers (<= 7)       how many other ranks receive this context's words (0 detaches)
 *   peer_payload_buffers   HOST array of num_peers DEVICE pointers: row 0 of each peer's signmuon_payload_buffer
 *   peer_flags             HOST array of num_peers DEVICE pointers: each peer's signmuon_exchange_flags
 * Call after signmuon_bind (a new bind detaches the peers and zeroes the flags).
 * Errors: INVALID_ARG, NOT_BOUND, MISALIGNED. */
int signmuon_exchange_flags(const signmuon_ctx* ctx, uint32_t** dev_ptr);
int signmuon_set_payload_peers(signmuon_ctx* ctx, int32_t my_rank, int32_t num_ranks, int32_t num_peers,
                               uint32_t* const* peer_payload_buffers, uint32_t* const* peer_flags);

/* The int8 SUM variant of the exchange (Alg. 2: "sum_signs <- sum_m S^(m)", all-reduce with SUM, then
 * "S <- sign(sum_signs)", ties -> +1).
 *   signmuon_local_sign_sum: writes, for every bit position of a payload (32 per word, pad positions included),
 *     the sum of the +-1 signs of this context's own workers as one int8: DEVICE [32 * payload words] bytes,
 *     16-byte aligned - the buffer a SUM all-reduce over the GPUs then turns into sum_signs.  num_workers must
 *     not exceed 127.
 *   signmuon_vote_update_from_sums: takes the reduced sums, forms the vote (sum >= 0 -> +1) and runs the local
 *     polar step and the weight update like signmuon_vote_update.  The result is bit-identical to voting over
 *     the gathered payloads (App. B: sign(2 c - M)).
 * Errors: INVALID_ARG, NOT_BOUND, BUFFER_TOO_SMALL, MISALIGNED, CUDA. */
int signmuon_local_sign_sum(signmuon_ctx* ctx, int8_t* dev_sums, size_t bytes, void* cuda_stream);
int signmuon_vote_update_from_sums(signmuon_ctx* ctx, const int8_t* dev_sums, size_t bytes, void* const* weights,
                                   const void* const* grads, float lr, void* cuda_stream);

/* Word offset of parameter `param` inside a worker's payload and its word count. */
int signmuon_payload_segment(const signmuon_ctx* ctx, int32_t param, size_t* word_offset, size_t* words);

/* DEVICE pointer + size of an intermediate result of the last step (SIGNMUON_TAP_*);
 * `ld` (may be NULL) receives the row pitch in elements for matrix-shaped taps. */
int signmuon_debug_tap(const signmuon_ctx* ctx, int32_t what, int32_t param, int32_t worker,
                       const void** dev_ptr, size_t* bytes, int64_t* ld);

/* Synchronises `cuda_stream`, then reads the device status word: OK, TIMEOUT (a bounded wait in a
 * kernel gave up; results of that step are invalid) or CUDA.  TIMEOUT stays until the next signmuon_bind. */
int signmuon_status(signmuon_ctx* ctx, void* cuda_stream);

/* Failure detection.  Every wait inside the Newton-Schulz kernels (on a TMA transfer, a tensor-core commit, an
 * epilogue hand-over) is bounded: after `limit_ns` nanoseconds (0 selects the default of two seconds) the waiting
 * thread records TIMEOUT in the status word and its CTA drains and exits, so a step can fail but not hang.
 * signmuon_selftest_wait_timeout enqueues a one-thread kernel that performs exactly that wait on a barrier nothing
 * ever signals, with the given limit (at most two seconds): afterwards signmuon_status must report TIMEOUT, and
 * signmuon_bind clears it.  Lets a deployment check the detection path without disturbing a step.
 * Errors: INVALID_ARG, NOT_BOUND, CUDA. */
int signmuon_set_wait_limit(signmuon_ctx* ctx, uint64_t limit_ns);
int signmuon_selftest_wait_timeout(signmuon_ctx* ctx, uint64_t limit_ns, void* cuda_stream);

/* Start vectors of the power iteration (Alg. 5, "Sample v in R^c"), needed when ns_scale is
 * SIGNMUON_SCALE_SPECTRAL: the method draws them at random, so the caller passes them in.
 *   signmuon_power_start_size:    length in floats of the whole array (0 when the scale is FRO)
 *   signmuon_power_start_segment: where the vectors of matrix parameter `param` start inside it; worker m's
 *                                 vector (cols floats) follows at float_offset + m * floats_per_worker
 *   signmuon_set_power_start:     DEVICE array (16-byte aligned, owned by the caller, read by every following
 *                                 step until replaced; fill it with fresh draws between steps as desired).
 * Errors: INVALID_ARG (scale is FRO, plain parameter, null), NOT_BOUND, BUFFER_TOO_SMALL, MISALIGNED;
 * signmuon_step returns NOT_BOUND when the scale is SPECTRAL and no start vectors were set. */
int signmuon_power_start_size(const signmuon_ctx* ctx, size_t* floats);
int signmuon_power_start_segment(const signmuon_ctx* ctx, int32_t param, size_t* float_offset,
                                 size_t* floats_per_worker);
int signmuon_set_power_start(signmuon_ctx* ctx, const float* dev_vectors, size_t floats);

/* Sign agreement of the last step (Sec. 5.3 logs "sign agreement ratios" next to the communication volume):
 * host_agree[m] (HOST, num_workers entries) = number of entries whose sign bit of worker m equals the
 * majority vote; *host_entries (may be NULL) = entries per worker, so the ratio is agree / entries.
 * Needs SIGNMUON_FLAG_SIGN_AGREEMENT; synchronises `cuda_stream`.  Errors: INVALID_ARG, NOT_BOUND, CUDA. */
int signmuon_sign_agreement(signmuon_ctx* ctx, uint64_t* host_agree, uint64_t* host_entries, void* cuda_stream);

/* Number of kernels signmuon_step launches per call with the current configuration. */
int signmuon_launches_per_step(const signmuon_ctx* ctx, int32_t* launches);

/* Of those, the launches of the Newton-Schulz products (workers' iterations and local polar step together):
 * `gemm_launches` grouped tensor-core product launches (Alg. 4's Gram and apply products, and the s x s products of
 * iterations that run in Gram space through memory) and `chain_launches` launches of the on-chip Gram-space chain.
 * Either pointer may be null.  Errors: INVALID_ARG (null context). */
int signmuon_ns_launches_per_step(const signmuon_ctx* ctx, int32_t* gemm_launches, int32_t* chain_launches);

/* Newton-Schulz floating-point operations of one step: 4 s^2 l K per matrix and worker (plus one
 * more "worker" for the local polar step), s = min(rows, cols), l = max(rows, cols). */
int signmuon_ns_flops_per_step(const signmuon_ctx* ctx, double* flops);

/* Flops the tensor cores are actually asked for per step by the tile schedule of the bound context: whole
 * 256 x 256 x 64 (or 128 x 128 x 64) blocks per scheduled tile, so ragged edges count in full, while the mirror
 * tiles of the symmetric Gram products (Alg. 4: A = Y Y^T), which are never computed, do not count.  Differs from
 * signmuon_ns_flops_per_step, the algorithm's own 4 s^2 l K.  Errors: INVALID_ARG, NOT_BOUND. */
int signmuon_ns_executed_flops_per_step(const signmuon_ctx* ctx, double* flops);

/* Capacity of the built-in scratch of signmuon_momentum_norm_noalloc: one float per 8192 entries per
 * worker, i.e. num_workers * ceil(rows*cols / 8192) must not exceed it (about 5.4e8 entries over all
 * workers; e.g. 4096 x 4096 with 32 workers just fits). */
#define SIGNMUON_NOALLOC_MAX_PARTIALS 65536

/* Momentum + Frobenius-norm stage for ONE matrix, usable where device memory cannot be allocated.
 * (The paper has no counterpart: it is the first stage of signmuon_step - weight decay, momentum,
 * bf16 operand, 1/max(||Mom||_F, eps) - repackaged for a class of callers.)
 *
 * Some hosts of this library may not call cudaMalloc around an optimizer step: a step recorded into a
 * pipeline whose memory plan is already frozen, a plugin that must not grow its host framework's memory
 * pool, a latency-critical loop that cannot take the allocator lock.  signmuon_step serves them only if
 * they can still hand over a workspace; this call needs none.  Its only scratch - the per-block partial
 * sums of the norm reduction - lives in a fixed 256 KB array inside the library image, present on every
 * GPU that loads the library until the process exits.  The call itself allocates nothing and calls
 * nothing that allocates (one caveat: the first call on a device is where the CUDA runtime may load the
 * library's device code and place that array; warm the entry point up once, outside any stream capture,
 * before the region that must not allocate).
 *
 *   dev_grads        DEVICE [M][rows*cols] grad_dtype, read only
 *   dev_weights      DEVICE [rows*cols] weight_dtype, read only; may be NULL when weight_decay == 0
 *   dev_momentum     DEVICE [M][rows*cols] float32, updated in place
 *   dev_operand_bf16 DEVICE [M][rows*cols] bf16, written dense (row pitch = cols): bf16(momentum).  This is
 *                    the layout of signmuon_step's Newton-Schulz operand only when cols is a multiple of 8
 *                    (the regular path pads rows to a multiple of 8 elements)
 *   dev_scales       DEVICE [M][2] float32, written: 1/max(sigma,eps)^2 and 1/max(sigma,eps)
 * rows*cols must be a multiple of 8 and all array pointers 16-byte aligned.
 *
 * Limits and sharing: problems larger than SIGNMUON_NOALLOC_MAX_PARTIALS allows are refused with
 * SIGNMUON_ERR_TOO_LARGE before anything is launched.  Every call on a device uses the same array; a
 * call overwrites the part it uses before reading it, so no clearing is needed between calls, but calls
 * that may run concurrently on one GPU (different streams without ordering) race - keep them ordered.
 * The first call on each device resolves the array's device address; make that call outside any stream
 * capture.  Other errors: INVALID_ARG, BAD_SHAPE, MISALIGNED, UNSUPPORTED_ARCH (current device is not
 * compute capability 10.x), CUDA (one of this call's own two launches was refused). */
int signmuon_momentum_norm_noalloc(const void* dev_grads, int32_t grad_dtype, const void* dev_weights,
                                   int32_t weight_dtype, float* dev_momentum, void* dev_operand_bf16,
                                   float* dev_scales, int64_t rows, int64_t cols, int32_t num_workers,
                                   float momentum, float weight_decay, float eps, void* cuda_stream);

void signmuon_destroy(signmuon_ctx* ctx);

const char* signmuon_error_string(int code);

#ifdef __cplusplus
}
#endif
#endif /* SIGNMUON_H_ */
