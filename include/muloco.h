/*
 * muloco.h -- C ABI of the MuLoCo optimizer step for NVIDIA B200 (sm_100a).
 *
 * One library call per line of the paper's Algorithm 1 that touches optimizer
 * state: the inner step (Muon on hidden matrices, AdamW elsewhere) of K DiLoCo
 * workers held as replicas on ONE GPU, and the outer synchronisation
 * (pseudogradient, optional block quantisation, Nesterov outer SGD, broadcast).
 * Gradients are supplied by the caller.
 *
 * Conventions
 *   - Unless a parameter says "host", every data pointer is a DEVICE pointer
 *     to memory owned by the caller; the library never frees caller memory.
 *     Arrays OF pointers (pointer tables) are always host arrays.
 *   - The library owns only its workspace, its descriptor tables and the small
 *     host state; muloco_destroy releases them.
 *   - All matrices are row-major float32 unless stated; a vector is a 1 x n
 *     matrix.
 *   - Every call enqueues its work on the CUDA stream given at create time and
 *     returns without waiting for the GPU.  Argument errors are reported by the
 *     return value at once.  Conditions found on the device (non-finite
 *     pseudogradient, a bounded wait that ran out) are written to a device
 *     status word and reported by muloco_sync_status.  Nothing aborts or traps.
 *   - Accuracy, against the definitions evaluated in exact arithmetic on the same float32 state:
 *     the element-wise steps (momentum, AdamW, outer step) are within
 *     |err| <= 1e-6 * |x| + 1e-6 * rms(tensor) per element -- the second term is an absolute
 *     floor, wider than "1e-6 relative" for entries far below the tensor's root mean square,
 *     where one float32 rounding of a sum of larger terms already exceeds 1e-6 of the entry;
 *     quantiser codes, scales and dequantised values are exact; Newton-Schulz: see
 *     muloco_newton_schulz.
 *   - The tensor-core Newton-Schulz kernel is one persistent launch whose thread blocks hand
 *     tiles to one another; it needs all of them resident at once, i.e. the GPU to itself while it
 *     runs (kernels of the same stream are fine: they run before or after).  If another context
 *     or stream holds SMs for long, its waits run out and the call ends with MULOCO_ETIMEOUT
 *     instead of hanging.
 *   - Calls on one context are not thread-safe.
 *   - There is no CPU fallback: without a CUDA device every compute call
 *     returns MULOCO_ECUDA.
 */
#ifndef MULOCO_H
#define MULOCO_H

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define MULOCO_API __attribute__((visibility("default")))
#else
#define MULOCO_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct muloco_ctx muloco_ctx; /* opaque */

typedef enum {
  MULOCO_OK = 0,
  MULOCO_EINVAL = 1,     /* bad argument (NULL, out of range, J does not divide H ...) */
  MULOCO_ESHAPE = 2,     /* unsupported shape */
  MULOCO_ENOMEM = 3,     /* workspace allocation failed */
  MULOCO_ECUDA = 4,      /* CUDA runtime/driver error, or no device */
  MULOCO_ENONFINITE = 5, /* device saw a non-finite pseudogradient, a non-finite gradient /
                            momentum of a hidden matrix (its Frobenius norm), or a
                            non-finite gradient of an AdamW tensor                    */
  MULOCO_ETIMEOUT = 6,   /* a bounded wait inside a kernel ran out */
  MULOCO_ESTATE = 7      /* call order / state blob mismatch */
} muloco_status;

typedef enum { MULOCO_MUON = 0, MULOCO_ADAMW = 1 } muloco_kind;
typedef enum { MULOCO_NS_BF16 = 0, MULOCO_NS_FP32 = 1 } muloco_ns_mode;
typedef enum { MULOCO_Q_NONE = 0, MULOCO_Q_INT2 = 2, MULOCO_Q_INT4 = 4, MULOCO_Q_INT8 = 8 } muloco_quant;
typedef enum { MULOCO_F32 = 0, MULOCO_BF16 = 1 } muloco_dtype;

/* One parameter tensor of the model. */
typedef struct {
  int64_t rows, cols; /* a vector is rows = 1                                           */
  int32_t kind;       /* muloco_kind: Muon for hidden matrices, AdamW for the rest
                         (Section 5, "MuLoCo")                                          */
  int32_t fragment;   /* 0..J-1: the subset synchronised together (Section 2,
                         "Partitioned Communication")                                   */
  float wd_mult;      /* multiplies the weight decay: 1 = decay, 0 = none (gains)       */
  float lr_mult;      /* learning-rate multiplier; NaN selects the default:
                         sqrt(cols/rows) for Muon (Section 5), 1 for AdamW              */
} muloco_tensor_desc;

typedef struct {
  int32_t K, H, J;     /* workers, inner steps per round, fragments (J must divide H)   */
  float muon_lr;       /* eta in W <- W - eta O - eta lambda W (Section 2, "Muon")      */
  float muon_beta;     /* m <- beta m + g                                                */
  float muon_wd;       /* lambda                                                         */
  int32_t muon_nesterov; /* 1: orthogonalise g + beta m, 0: orthogonalise m            */
  int32_t ns_steps;    /* Newton-Schulz iterations, 5 in the paper                       */
  float ns_a, ns_b, ns_c; /* quintic coefficients, (3.4445, -4.7750, 2.0315)           */
  float ns_eps;        /* X0 = U / (||U||_F + ns_eps)                                    */
  int32_t ns_mode;     /* muloco_ns_mode                                                 */
  int32_t wd_uses_scaled_lr; /* 1: the decay term uses the shape-rescaled eta too       */
  float adam_lr, adam_beta1, adam_beta2, adam_eps, adam_wd; /* Section 4.3               */
  int32_t adam_bias_correction; /* 1: divide by 1 - beta^t                              */
  float outer_lr, outer_momentum; /* eta_out, mu of Eq. (3)                             */
  int32_t quant;       /* muloco_quant: quantise -> dequantise the pseudogradient       */
  int32_t quant_block; /* elements per absmax block along a row (32, 64 or 128), or 0 for
                          row-wise quantisation: one block per row (rows of up to ~50,000
                          elements; longer rows make muloco_outer_sync return MULOCO_ESHAPE) */
  int32_t grad_dtype;  /* muloco_dtype of the gradients given to muloco_inner_step      */
  int32_t quant_stages; /* 0 or 1: quantise the averaged pseudogradient once (benchmark form);
                           2: Algorithm 2 with the two quantisations of Section 2
                           ("Collectives for compressed communication"): every worker's delta
                           is quantised, the mean is taken in float32, the mean is quantised
                           again                                                            */
  uint64_t workspace_bytes; /* Newton-Schulz workspace budget; 0 lets the library pick  */
  int32_t error_feedback; /* 1: Algorithm 2's error feedback, E_i <- beta E_i + Delta_i,
                             send C(E_i), E_i <- E_i - C(E_i); needs the ef_k buffers and a
                             per-worker compressor: quant_stages == 2 with a quantiser, or
                             topk_fraction > 0                                              */
  float ef_beta;       /* beta of the error-feedback accumulator                          */
  float topk_fraction; /* 0: off.  In (0, 1]: top-k sparsification (Section 2, "Compressed
                          Communication") of every worker's delta, per tensor: with n elements,
                          kk = max(1, floor(topk_fraction * n)) (in double), the entries whose
                          magnitude is at least the kk-th largest are kept (ties all kept), the
                          rest become 0; the mean of the sparsified deltas is the
                          pseudogradient, nothing is compressed after the mean.  Needs
                          quant == MULOCO_Q_NONE; error_feedback may be set with it.  Tensors
                          of 2^31 elements or more make muloco_create return MULOCO_ESHAPE.    */
} muloco_config;

/* State buffers.  Every field is a HOST array of DEVICE pointers.
 * Per-worker tables have K * n_tensors entries, entry [k * n_tensors + i]. */
typedef struct {
  float* const* theta_k;  /* [K][n]  worker replicas theta_k                            */
  float* const* theta_g;  /* [n]     global parameters theta                            */
  float* const* outer_u;  /* [n]     outer momentum u                                   */
  float* const* state1_k; /* [K][n]  Muon momentum m, or Adam first moment              */
  float* const* state2_k; /* [K][n]  Adam second moment (ignored for Muon tensors)      */
  float* const* ef_k;     /* [K][n]  error-feedback accumulators E_i (Algorithm 2); the table
                             may be NULL unless cfg.error_feedback is set                */
} muloco_buffers;

/* Algorithm 1, initialisation.  Validates the arguments, records the tensor table,
 * allocates the library's own device memory (the Newton-Schulz workspace, small descriptor
 * and pointer tables; the *_host calls add a gradient staging area on first use), then
 * enqueues u <- 0, inner state <- 0 and theta_k <- theta_g for every worker.
 * `cuda_stream` is a cudaStream_t (NULL = the default stream).  n_tensors may
 * be 0 for a context that only serves muloco_newton_schulz / muloco_quantize.
 * On failure *out is NULL and the return value says why. */
MULOCO_API muloco_status muloco_create(const muloco_config* cfg, const muloco_tensor_desc* tensors,
                            int32_t n_tensors, const muloco_buffers* bufs, void* cuda_stream,
                            muloco_ctx** out);

/* Releases workspace and tables (waits for the stream first). NULL is allowed. */
MULOCO_API void muloco_destroy(muloco_ctx* ctx);

/* Algorithm 1, body of the inner loop (Eq. 1) with the gradient given: one inner optimizer
 * step for worker `worker` (0..K-1), or for all K workers batched when
 * worker == -1.  `grads` is a host table of device pointers: [n_tensors] for one
 * worker, [K][n_tensors] for all; each gradient has its tensor's shape and the
 * dtype named by cfg.grad_dtype.  Gradients are read only.
 * Hidden matrices (Section 2 "Muon", Section 5 "MuLoCo"):
 *     m <- beta m + g;  U = g + beta m (Nesterov) or m;  O = NS_5(U / (||U||_F + eps));
 *     W <- W - eta' O - eta' lambda W,  eta' = muon_lr * lr_scale * sqrt(cols/rows).
 * Other tensors: AdamW (Section 4.3) with step size adam_lr * lr_scale.
 * `lr_scale` is the learning-rate schedule's multiplier for this step. */
MULOCO_API muloco_status muloco_inner_step(muloco_ctx* ctx, int32_t worker, const void* const* grads,
                                float lr_scale);

/* As muloco_inner_step, but `host_grads` is a host table of HOST pointers
 * (pinned memory for full speed).  The gradients are copied to a device staging
 * area owned by the library (allocated on first use) by two copy streams of the
 * library's own (alternating tensors), one section (group of same-shape matrices, then the AdamW tensors)
 * at a time; the step's kernels wait for their section only, so copies overlap the
 * compute of other sections and of the previous step.  The host buffers must stay
 * unchanged until the step has run (muloco_sync_status, or any wait on the stream). */
MULOCO_API muloco_status muloco_inner_step_host(muloco_ctx* ctx, int32_t worker,
                                     const void* const* host_grads, float lr_scale);

/* Algorithm 1, outer step (Eqs. 2-3) for the tensors of fragment `fragment`
 * (0..J-1), or all tensors when fragment == -1, in one pass over memory:
 *     Psi = (1/K) sum_k (theta_g - theta_k)   (fp32, k ascending, then * 1/K)
 *     optional: Psi <- dequantise(quantise(Psi)) per block of quant_block elements
 *               along a row (absmax scale, round to nearest even, int8, int4 or int2)
 *     with quant_stages == 2 (Algorithm 2): every worker's delta theta_g - theta_k (or, with
 *               error feedback, E_k <- ef_beta E_k + delta) is quantised -> dequantised first
 *               (and E_k <- E_k - what was sent), the mean of those is taken in fp32 (k
 *               ascending, then * 1/K) and quantised -> dequantised again
 *     u <- mu u + eta_out Psi;   theta_g <- theta_g - mu u - eta_out Psi
 *     theta_k <- theta_g for every worker.
 * With K == 1, eta_out == 1, mu == 0 and no compression (plain data parallelism, Section 5's DP
 * baselines) the step is the identity on the worker: theta_g <- theta_1 bit for bit (H plain
 * inner steps, exactly), u <- theta_g - theta_1, one pass of 16 bytes per parameter.
 * Inner optimizer state is kept.  Syncing a fragment that is not due is allowed;
 * the schedule is the caller's (see muloco_fragments_due). */
MULOCO_API muloco_status muloco_outer_sync(muloco_ctx* ctx, int32_t fragment);

/* As muloco_outer_sync, then copies the new global parameters of every tensor
 * of the fragment to host memory: host_theta_g is a host table [n_tensors] of
 * HOST pointers (entries of tensors outside the fragment are not touched and
 * may be NULL).  The copies are enqueued on the context's stream. */
MULOCO_API muloco_status muloco_outer_sync_host(muloco_ctx* ctx, int32_t fragment, void* const* host_theta_g);

/* Worker-sharded outer synchronisation: the K_total = world * K workers of the method are spread
 * over `world` GPUs (one context per GPU, each holding K of them and its own copy of theta and
 * u), and Algorithm 1's all-reduce of the outer delta is taken apart into a reduce-scatter and
 * an all-gather (Section 2, "Collectives for compressed communication"; Appendix, "Assumptions
 * around the collective used"), which the CALLER runs between the three calls below, on the
 * context's stream (e.g. NCCL through torch.distributed):
 *     muloco_shard_delta      stage <- sum over this GPU's workers of (theta - theta_k)
 *                             (fp32, k ascending; with quant_stages == 2 every worker's delta,
 *                             or its error-feedback sum, is quantised -> dequantised first)
 *     reduce-scatter(sum)     stage [stage_floats]  ->  reduced [shard_floats] (shard `rank`)
 *     muloco_shard_step       Psi = reduced * 1/K_total; the (second) quantisation; Eq. 3 on
 *                             this GPU's shard of u and theta; theta_shard <- new theta
 *     all-gather              theta_shard [shard_floats]  ->  theta_all [stage_floats]
 *     muloco_shard_broadcast  theta and every local replica <- theta_all
 * Buffers are device float32 arrays in the library's staging layout: unit-major, 128 floats
 * per unit (a unit is one block of the quantiser, at most 128 elements of one row; unused lanes
 * hold zeros), padded with zero units so that every GPU's shard has the same number of whole
 * units; muloco_shard_layout gives the sizes.  u is kept only for the GPU's own shard.  With
 * world == 1 (no collective) the three calls give what muloco_outer_sync gives, bit for bit;
 * with more GPUs the sum over GPUs is in the collective's order.  Top-k sparsification and
 * row-wise quantisation are not available in this form (MULOCO_EINVAL).  Bytes on the wire per
 * GPU and sync: 2 * 4 * stage_floats * (world - 1) / world. */
MULOCO_API muloco_status muloco_shard_layout(muloco_ctx* ctx, int32_t fragment, int32_t world, int32_t rank,
                                             int64_t* stage_floats, int64_t* shard_floats);
MULOCO_API muloco_status muloco_shard_delta(muloco_ctx* ctx, int32_t fragment, int32_t world, float* stage);
MULOCO_API muloco_status muloco_shard_step(muloco_ctx* ctx, int32_t fragment, int32_t world, int32_t rank,
                                           const float* reduced, float* theta_shard);
MULOCO_API muloco_status muloco_shard_broadcast(muloco_ctx* ctx, int32_t fragment, int32_t world,
                                                const float* theta_all);

/* Streaming schedule (Section 2, "Partitioned Communication"): fragment j
 * (1-based) is due after inner step t > 0 when t mod H == (j H / J) mod H.
 * Writes the 0-based due fragments to out_frags (host, room for J) and returns
 * their count (0 if none, -1 on bad arguments). */
MULOCO_API int32_t muloco_fragments_due(const muloco_ctx* ctx, int64_t step, int32_t* out_frags);

/* Five-step quintic Newton-Schulz (Section 2, "Muon") on a batch of same-shape
 * matrices, outside any optimizer state: X is [batch][rows][cols] (x_dtype),
 * O has the same shape (o_dtype).  Each matrix is divided by its Frobenius norm
 * (+ ns_eps) first; matrices with rows > cols are iterated on their transpose.
 * ns_mode MULOCO_NS_BF16 runs the tensor-core engine (bf16 operands, fp32
 * accumulation), MULOCO_NS_FP32 the fp32 engine.  X and O must not overlap.
 * Accuracy against the iteration in exact arithmetic (relative Frobenius error):
 * 1e-4 for the fp32 engine, 2e-2 for the bf16 engine with up to the paper's five steps (more
 * steps amplify the roundings of the earlier ones: 2.4e-2 was seen with seven).  The bf16 engine holds its
 * bound only from min(rows, cols) = 64 on; matrices with a smaller min-dimension
 * (also inside muloco_inner_step) are always served by the fp32 engine, whatever
 * mode is asked, and meet the fp32 bound. */
MULOCO_API muloco_status muloco_newton_schulz(muloco_ctx* ctx, const void* X, int32_t x_dtype, void* O,
                                   int32_t o_dtype, int32_t batch, int64_t rows, int64_t cols,
                                   int32_t ns_mode);

/* Size of the fixed scratch behind muloco_newton_schulz_static (bytes). */
#define MULOCO_STATIC_SCRATCH_BYTES (8u << 20)

/* Newton-Schulz for callers that must not allocate device memory.  (The paper has
 * no counterpart: this is a packaging variant of muloco_newton_schulz in its fp32
 * mode, with the paper's coefficients, 5 steps and eps = 1e-7.)
 *
 * Who needs it: code running where a device allocation is off limits -- after a
 * framework's caching allocator has taken the whole GPU, so that a raw cudaMalloc
 * may fail or fragment the pool, or inside a latency-critical loop that cannot pay
 * for the device-wide synchronisation that allocating and freeing imply.  This call
 * needs no context (creating one allocates) and calls no cudaMalloc, cudaFree or
 * other allocating routine: its scratch is a fixed array of
 * MULOCO_STATIC_SCRATCH_BYTES inside the library image, which every GPU that loads
 * the library holds until the process exits.
 *
 * X: [batch][rows][cols] float32 device input, O: same shape float32 device output
 * (must not overlap X); batch <= 64.  The scratch must hold, per matrix with
 * s = min(rows, cols), l = max(rows, cols): 2*s*l + 2*s*s floats (each row padded
 * to 8 elements) plus small tables; a request that does not fit returns
 * MULOCO_ESHAPE and explains the sizes in errbuf -- use muloco_newton_schulz then.
 * errbuf (host, may be NULL) receives a NUL-terminated message on failure.
 * The work is enqueued on `cuda_stream` (a cudaStream_t, NULL = default stream) of
 * the CURRENT device; the call copies nothing from host memory (its small tables are
 * written by a kernel from the arguments), so nothing on the host has to outlive it.
 * Only argument and launch errors are reported: there is no context and no status
 * word, so a NaN or Inf in X is not detected -- the matrix that holds it comes out
 * non-finite and the call still returns MULOCO_OK (muloco_newton_schulz followed by
 * muloco_sync_status reports MULOCO_ENONFINITE for the same input).
 *
 * The first call on each device resolves the scratch's device address (once per
 * device, that device being current); make that first call before starting any
 * stream capture.  All calls on a device share the one scratch array, which keeps
 * whatever the last call left in it: calls whose GPU work overlaps in time
 * (different streams or threads) race with each other -- serialise them. */
MULOCO_API muloco_status muloco_newton_schulz_static(const float* X, float* O, int32_t batch,
                                                     int64_t rows, int64_t cols, void* cuda_stream,
                                                     char* errbuf, size_t errbuf_len);

/* The block quantiser on its own (the benchmark's per-block absmax form of the
 * linear quantisation of Section 2, "Compressed Communication"): psi is a
 * rows x cols float32 matrix; writes, where non-NULL, one int8 code per element
 * to `codes` (int4 codes are -7..7, unpacked), one float32 scale per block to
 * `scales` ([rows][ceil(cols/block)]) and the dequantised values to `dequant`.
 * bits is 8, 4 or 2. */
MULOCO_API muloco_status muloco_quantize(muloco_ctx* ctx, const float* psi, int64_t rows, int64_t cols,
                              int32_t bits, int8_t* codes, float* scales, float* dequant);

/* Test hook: the top-k sparsifier on its own (Section 2, "Compressed Communication"): x and out are
 * DEVICE arrays of n float32 (they may be the same array); out = x where |x| is at least the
 * kk-th largest magnitude, kk = max(1, floor(fraction * n)), else 0.  fraction in (0, 1].
 * Not for a hot path: it allocates and frees a few KB of device scratch and waits for the
 * stream before returning (the synchronisation's own scratch is allocated once, at create). */
MULOCO_API muloco_status muloco_topk_sparsify(muloco_ctx* ctx, const float* x, int64_t n, float fraction,
                                   float* out);

/* Test hook: the pseudogradient of tensor `tensor` (Eq. 2), exactly as
 * muloco_outer_sync forms it, written to psi_out (float32, tensor's shape),
 * without changing any state. */
MULOCO_API muloco_status muloco_pseudogradient(muloco_ctx* ctx, int32_t tensor, float* psi_out);

/* Small host state for checkpoint/resume: inner step counters per worker and
 * sync counters per fragment.  Call with blob == NULL to get the size. */
MULOCO_API muloco_status muloco_get_state(const muloco_ctx* ctx, void* host_blob, size_t* nbytes);
MULOCO_API muloco_status muloco_set_state(muloco_ctx* ctx, const void* host_blob, size_t nbytes);

/* Phase timers (CUDA events on the context's stream). */
enum {
  MULOCO_PH_PROLOGUE = 0, /* momentum + bf16/fp32 staging + norms                     */
  MULOCO_PH_NS = 1,       /* Newton-Schulz GEMMs, including the fused final update    */
  MULOCO_PH_ADAMW = 2,
  MULOCO_PH_SYNC = 3,
  MULOCO_PH_COPY = 4,     /* host<->device copies of the *_host calls (sum over the two
                             copy streams, which run side by side)                    */
  MULOCO_N_PHASES = 5
};
MULOCO_API muloco_status muloco_set_timing(muloco_ctx* ctx, int32_t enabled);
/* Waits for the stream, writes the milliseconds accumulated per phase since the
 * last call to ms[MULOCO_N_PHASES] and the number of kernel launches since the
 * last call to *launches (either may be NULL), then resets both. */
MULOCO_API muloco_status muloco_get_timings(muloco_ctx* ctx, float* ms, int64_t* launches);

/* Test hooks for the failure path of the tensor-core Newton-Schulz kernel, whose every
 * device-side wait (on a copy, on the tensor cores, on another CTA's tiles) has a time limit.
 *   MULOCO_DEBUG_WAIT_LIMIT_NS : that limit in nanoseconds (0 restores the default of 2 s).
 *   MULOCO_DEBUG_WITHHOLD_COPY : value != 0 makes the NEXT tensor-core launch of this context
 *       leave out one operand copy of its first tile, so that the waits for it run out: the
 *       kernel gives up cleanly (every CTA frees its tensor memory and returns) and
 *       muloco_sync_status reports MULOCO_ETIMEOUT.  One-shot.
 * After MULOCO_ETIMEOUT the context stays usable.  The step that timed out is incomplete: for
 * the hidden matrices of the affected shape group the momentum has been advanced, but the
 * parameters theta_k of some of its (worker, matrix) pairs have been updated, or partly
 * updated, and others not, and nothing records which.  A caller that wants to continue
 * restores theta_k and the momenta of that step from its own copy (a checkpoint of the
 * caller-owned tensors plus muloco_get_state / muloco_set_state) and repeats the step.
 *
 * Workspace canaries (the library's stand-in for a memory checker): every region of the
 * Newton-Schulz workspace (staged input, ring of intermediates, norm partials, scales, tile
 * counters) lies between guard zones whose adjoining 64 bytes hold a fixed pattern.
 *   MULOCO_DEBUG_CANARIES : value != 0 makes every Newton-Schulz chunk write the canaries
 *       before it runs and compare them after (this waits for the stream after every chunk: a
 *       debugging mode).  muloco_check_workspace reports the first canary found overwritten
 *       since its last call (MULOCO_ESTATE, text in muloco_last_error), else MULOCO_OK.
 *   MULOCO_DEBUG_CORRUPT_CANARY : test hook; value = index of a workspace region whose canary
 *       the host overwrites (one byte, by a memset on the stream) in the next chunk, so that
 *       the check has something to find.  One-shot.
 * A debug build of the library (-DMULOCO_DEBUG, build.build_library(debug=True)) adds
 * device-side checks of the indices the kernels derive; a failed check raises a flag that
 * muloco_sync_status reports as MULOCO_ECUDA ("out-of-range index"), and the access is skipped. */
enum { MULOCO_DEBUG_WAIT_LIMIT_NS = 1, MULOCO_DEBUG_WITHHOLD_COPY = 2, MULOCO_DEBUG_CANARIES = 3,
       MULOCO_DEBUG_CORRUPT_CANARY = 4 };
MULOCO_API muloco_status muloco_debug_set(muloco_ctx* ctx, int32_t what, int64_t value);
MULOCO_API muloco_status muloco_check_workspace(muloco_ctx* ctx);

/* Waits for the stream and returns the device status word as a muloco_status
 * (MULOCO_OK, MULOCO_ENONFINITE, MULOCO_ETIMEOUT, MULOCO_ECUDA); clears it. */
MULOCO_API muloco_status muloco_sync_status(muloco_ctx* ctx);

/* Text of the last error on this context (or of the last failed create when
 * ctx is NULL).  The string is owned by the library. */
MULOCO_API const char* muloco_last_error(const muloco_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* MULOCO_H */
