/*
 * asyncmesh.h -- C ABI of the B200 (sm_100a) AsyncMesh per-step update library.
 *
 * The library holds R data-parallel replicas x S pipeline stages of flat fp32
 * parameters on ONE GPU and advances them one optimisation step per call.  A
 * step fuses, per stage and coordinate (paper notation: m -> R, P -> S):
 *
 *   1. the local optimizer step of every replica          (Section 2.3, Eq. "sparta", line 1;
 *      AdamW with decoupled weight decay, moments local)
 *   2. the random subset S_j^t of coordinates, one per     (Section 2.3; Appendix Lemma 1:
 *      stage and step, shared by the stage's replicas       each element independently with prob. p)
 *   3. the snapshot of the local iterates on S_j^t, whose  (Section 3.1: the average launched at
 *      replica average becomes usable tau steps later        step t arrives at step t + tau)
 *   4. delayed sparse averaging on S_j^{t-tau} with the    (Section 3.1 Eq. "asparta"; Section 3.2
 *      EMA estimate of the average staleness                 Eq. "ema" and the corrected averaging)
 *   5. the pipeline look-ahead: last update direction      (Section 2.2)
 *      extrapolated by the stage's delay
 *
 * All pointers named "device" are CUDA device pointers on the configured
 * device; pointers named "host" are ordinary host pointers.  Every function
 * returns 0 (ASYNCMESH_OK) or a negative code, never throws and never aborts;
 * asyncmesh_last_error() gives the message of the calling thread's last
 * failure.  Calls on one handle must not overlap in time.  There is no CPU
 * fallback: without a usable CUDA device every call that needs one fails.
 */
#ifndef ASYNCMESH_H
#define ASYNCMESH_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ASYNCMESH_OK 0
#define ASYNCMESH_ERR_INVALID_ARG (-1)
#define ASYNCMESH_ERR_OOM (-2)
#define ASYNCMESH_ERR_CUDA (-3)
#define ASYNCMESH_ERR_BAD_STATE (-4)
#define ASYNCMESH_ERR_UNSUPPORTED (-5)
#define ASYNCMESH_ERR_DEVICE_STATUS (-6)

#define ASYNCMESH_MAX_REPLICAS 16u
#define ASYNCMESH_MAX_STAGES 64u
#define ASYNCMESH_MAX_TAU 64u

/* asyncmesh_config.optimizer */
#define ASYNCMESH_OPT_ADAMW 0u
#define ASYNCMESH_OPT_NADAMW 1u

/* asyncmesh_config.correction: the staleness estimate d_i of Section 3.2 */
#define ASYNCMESH_CORRECTION_EMA 0u   /* Eq. "ema": d <- (1 - lambda) d + lambda (w^_i^t - w^_i^{t-tau}) */
#define ASYNCMESH_CORRECTION_EAGER 1u /* d = (w^_i^t - w^_i^{t-tau}) / R, the eager-update rule the
                                         section's last paragraph names as a special case (there with
                                         p = 1 and tau = K; accepted here for any p, tau, K); lambda
                                         is ignored                                                */

/* asyncmesh_config.flags */
#define ASYNCMESH_FLAG_SMALL_RING 1u /* diagnostic: give each compact ring slot 1/8 of
                                        its normal capacity, so that the overflow
                                        report (DEVICE_STATUS) can be exercised    */
#define ASYNCMESH_FLAG_DIRECT_KERNEL 2u /* use the register-load ("direct") step kernel even
                                          where the shared-memory pipelined one applies  */
#define ASYNCMESH_FLAG_PIPELINED_KERNEL 4u /* use the compact ring and the pipelined kernel for
                                             any p (diagnostic: exercises its in-place path) */
#define ASYNCMESH_FLAG_OWNER_KERNEL 256u /* use the kernel in which the lane that owns a coordinate
                                           does all of its work, with the compact ring whatever p
                                           is (up to four replicas; it is the default there for
                                           the compact ring and for tau = 0, this flag only extends
                                           it to subsets the dense ring would otherwise serve)  */
#define ASYNCMESH_FLAG_TRACK_CONSENSUS 512u /* every step also accumulates the consensus error of each stage
                                              (Section 3.3) from the final weights the step kernel holds in
                                              registers: asyncmesh_consensus_error then returns the value of
                                              the last step without another pass over the weights.  Honoured
                                              where the owner kernel runs in its common form (up to four
                                              replicas; up to eight for tau = 0); elsewhere the flag changes
                                              nothing and the call makes its own pass as usual           */
#define ASYNCMESH_FLAG_BF16_EXCHANGE 16u /* the subset is exchanged in bfloat16 (the paper's
                                           quantisation study): every snapshot value entering the
                                           replica average is first rounded to bfloat16 (nearest
                                           even); the average is formed in fp32 and a replica's own
                                           staleness sample uses its own unrounded value         */
#define ASYNCMESH_FLAG_FP8_EXCHANGE 64u /* as BF16_EXCHANGE, with 8-bit floating point (E4M3: 4
                                          exponent and 3 mantissa bits, nearest even, magnitudes above
                                          448 clamp to 448, no scale factor; the paper does not say
                                          which 8-bit format it used).  Not together with BF16_EXCHANGE */
#define ASYNCMESH_FLAG_RING_AS_EXCHANGED 1024u /* with BF16_EXCHANGE or FP8_EXCHANGE and tau > 0: a second
                                                  reading of the reduced-precision exchange (Section 5.3,
                                                  paragraph "Robustness of Sparse Averaging"; Appendix B.2,
                                                  which do not say whether a replica keeps an unrounded copy
                                                  of what it sent).  The snapshot ring stores the values as
                                                  exchanged, 2 or 1 bytes each, and a replica's staleness
                                                  sample w^_i^t - w^_i^{t-tau} is taken against that rounded
                                                  value; d then carries the rounding error of the snapshot.
                                                  Implies the dense ring (tau slots of R x stride values:
                                                  half or a quarter of its fp32 size) and the direct kernel;
                                                  INVALID_ARG without an exchange flag, with tau = 0, or
                                                  together with SMALL_RING, PIPELINED_KERNEL or OWNER_KERNEL */
#define ASYNCMESH_FLAG_KEEP_PREVIOUS 128u /* keep w^{t-1}: before each step the weights are copied
                                            aside (one device-to-device copy per stage, 8 bytes per
                                            replica-coordinate of extra traffic, 4 bytes of memory),
                                            and asyncmesh_lookahead_weights accepts any delay    */
#define ASYNCMESH_FLAG_DENSE_RING 32u /* keep the snapshot ring dense (one position per coordinate
                                        and replica, tau slots) whatever p is: more memory and
                                        some more traffic, no compaction work                   */

/* state selectors of asyncmesh_read_state */
#define ASYNCMESH_STATE_W 0     /* weights w_i^t                               */
#define ASYNCMESH_STATE_M 1     /* Adam first moment                           */
#define ASYNCMESH_STATE_V 2     /* Adam second moment                          */
#define ASYNCMESH_STATE_D 3     /* EMA staleness estimate d_i^t (Eq. "ema")    */
#define ASYNCMESH_STATE_LOOK 4  /* look-ahead weights of the configured delay  */

typedef struct asyncmesh asyncmesh;

/* Device-memory callbacks.  alloc returns a device pointer aligned to at
 * least 256 bytes, or NULL; the library calls free exactly once per pointer. */
typedef void *(*asyncmesh_alloc_fn)(void *ctx, size_t bytes);
typedef void (*asyncmesh_free_fn)(void *ctx, void *device_ptr);

/*
 * Problem statement (Section 2.1: P stages x m replicas; Section 2.3: subset
 * per stage; Section 3.1: delay tau; Section 3.2: EMA coefficient lambda;
 * Section 2.2: stage-dependent delay delta_j).  Hyper-parameters are doubles;
 * each derived per-step scalar is formed in double and rounded to fp32 once.
 */
typedef struct asyncmesh_config {
    uint32_t R;                      /* replicas, 1..ASYNCMESH_MAX_REPLICAS            */
    uint32_t S;                      /* stages, 1..ASYNCMESH_MAX_STAGES                */
    const uint64_t *stage_numel;     /* host [S]: parameters of stage j, 1..2^32-1     */
    double p;                        /* subset probability, 0..1                       */
    uint32_t tau;                    /* averaging delay in steps, 0..ASYNCMESH_MAX_TAU */
    uint32_t flags;                  /* 0 or ASYNCMESH_FLAG_*                          */
    double ema_beta;                 /* the paper's lambda: weight of the NEW staleness
                                        sample in Eq. "ema"; 0 = no correction, 0..1   */
    double lr, beta1, beta2, eps, weight_decay; /* AdamW                              */
    uint64_t seed;                   /* Philox key of the subset rule                  */
    const uint32_t *lookahead_delay; /* host [S] or NULL (NULL: delta_j = S - 1 - j)   */
    int32_t device;                  /* CUDA device ordinal                            */
    int32_t avg_interval;            /* K: subsets are exchanged every K-th step (end of
                                        Section 3.2); 0 or 1 = every step; must divide tau */
    void *stream;                    /* cudaStream_t all work is issued on (NULL: the
                                        legacy default stream)                         */
    asyncmesh_alloc_fn alloc;        /* both NULL: cudaMalloc / cudaFree               */
    asyncmesh_free_fn free;
    void *alloc_ctx;
    uint32_t optimizer;              /* ASYNCMESH_OPT_ADAMW (0) or ASYNCMESH_OPT_NADAMW: Adam with
                                        Nesterov momentum and decoupled decay, the optimizer the
                                        paper runs asynchronous pipelines with (Appendix B.1,
                                        momentum beta1 = 0.99)                             */
    uint32_t correction;             /* ASYNCMESH_CORRECTION_EMA (0) or ASYNCMESH_CORRECTION_EAGER */
    double momentum_decay;           /* NAdamW: psi of mu_t = beta1 (1 - 0.5 * 0.96^(t psi));
                                        0 selects the customary 0.004                   */
    const uint64_t *coord_base;      /* host [S] or NULL (all 0): global index of this handle's
                                        coordinate 0 of stage j, when the handle holds one
                                        coordinate range of a larger stage (a shard; coordinates
                                        are independent of one another, Appendix A, so ranges of
                                        a stage can live on different GPUs with no exchange).
                                        The subset rule uses the global index, so shards select
                                        exactly what the unsharded stage would.  Multiples of 4;
                                        coord_base + stage_numel <= 2^32                 */
} asyncmesh_config;

/*
 * Create the state: per stage W, M, V (replica-major rows [R][row_stride]),
 * D (coordinate-major [row_stride][R]; replica-major with the dense ring), LOOK
 * (only where delta_j > 0), a copy of the previous weights (only with
 * ASYNCMESH_FLAG_KEEP_PREVIOUS) and the snapshot ring (compact: room for the
 * selected coordinates only, tau / K + 1 slots; dense, for large p: one position
 * per coordinate and replica, tau / K slots, of 4-byte values, or of 2- or 1-byte
 * values with ASYNCMESH_FLAG_RING_AS_EXCHANGED; K = avg_interval).  The library owns
 * all of it (obtained through cfg->alloc).
 * Moments, D and the ring start at zero, the step counter at 0, weights are
 * unset until asyncmesh_init_params.  The config and its arrays are copied.
 * Errors: INVALID_ARG (range checks above), OOM (allocator returned NULL: every
 * partial allocation is released), CUDA.
 */
int asyncmesh_create(const asyncmesh_config *cfg, asyncmesh **out);

/* Release everything.  NULL is accepted and returns ASYNCMESH_OK. */
int asyncmesh_destroy(asyncmesh *h);

/*
 * Set the initial weights w^0 of one replica of a stage (replica = -1: all
 * replicas, the "same initialisation" of the homogeneous setup, Section 3.3).
 * src holds n = stage_numel[stage] floats, on the device if src_on_device != 0
 * else on the host.  Also sets w^{-1} := w^0, i.e. look-ahead = w^0.
 * Only allowed before the first step (BAD_STATE afterwards).
 */
int asyncmesh_init_params(asyncmesh *h, uint32_t stage, int32_t replica,
                          const float *src, uint64_t n, int src_on_device);

/* Floats between consecutive replica rows of a stage (a multiple of 32,
 * >= stage_numel[stage]).  Gradient buffers use the same stride.  (Layout
 * bookkeeping: defines nothing of the paper's method.) */
int asyncmesh_row_stride(const asyncmesh *h, uint32_t stage, uint64_t *stride);

/*
 * One step t <- t + 1 of the whole mesh (items 1-5 above for every stage), in
 * one kernel launch on the handle's stream; returns without waiting for it.
 * grads: host array of S device pointers; grads[j] is [R][row_stride_j] fp32,
 * 16-byte aligned, row i = gradient of replica i evaluated by the caller
 * (Eq. "gd": at whatever delayed weights the pipeline used).  Caller-owned,
 * read-only, and free to reuse once the stream has passed this step.
 * ema_beta_t / lr_t < 0 keep the configured constants; values >= 0 replace them
 * for this step only (the paper decays both over training, Section 3.3 and
 * Appendix B.1); weight decay is applied as lr_t * weight_decay.
 */
int asyncmesh_step(asyncmesh *h, const float *const *grads);
int asyncmesh_step_ex(asyncmesh *h, const float *const *grads,
                      double ema_beta_t, double lr_t);

/*
 * The same step with gradients in HOST memory: grads_host[j] is [R][numel_j]
 * fp32, rows contiguous (no padding).  They are copied into library-owned
 * device staging buffers (allocated on the first call), stage by stage, on a
 * stream of the library's own (created on the first call), and the step runs as
 * one launch per stage on the handle's stream, each as soon as its stage's
 * gradients have arrived: the kernels of all but the last stage run while later
 * stages are still being copied.  The result is the same as that of
 * asyncmesh_step.  The host buffers may be reused once the handle's stream has
 * passed the step.  Pinned host memory makes the copies asynchronous; pageable
 * memory works and is slower.
 */
int asyncmesh_step_host(asyncmesh *h, const float *const *grads_host);
int asyncmesh_step_host_ex(asyncmesh *h, const float *const *grads_host,
                           double ema_beta_t, double lr_t);   /* per-step scalars as in asyncmesh_step_ex */

/*
 * Look-ahead weights of a stage: w^t + delay * (w^t - w^{t-1}) (Section 2.2).
 * Returns a library-owned device pointer [R][row_stride], valid until the next
 * step, the next call for the same stage with another delay, or destroy.
 * delay = the stage's configured delay: the buffer the fused step wrote; delay
 * = 0: the weights themselves; any other delay: computed now, on the stream,
 * into a per-stage buffer allocated on first use, from the weights and their
 * previous values -- only if the handle was created with
 * ASYNCMESH_FLAG_KEEP_PREVIOUS, otherwise UNSUPPORTED.
 */
int asyncmesh_lookahead_weights(asyncmesh *h, uint32_t stage, uint32_t delay,
                                const float **out_device, uint64_t *row_stride);

/*
 * Copy out the weights of one replica (replica = -1: the replica mean, summed
 * in replica order and divided by R -- the model the paper evaluates: Section 5.1
 * reports validation loss on the average of the replicas' weights).  dst receives n = stage_numel[stage] floats, on the device if
 * dst_on_device != 0 else on the host.  Waits for the stream; reports a pending
 * device status (ring overflow) as DEVICE_STATUS.
 */
int asyncmesh_read_params(asyncmesh *h, uint32_t stage, int32_t replica,
                          float *dst, uint64_t n, int dst_on_device);

/* Copy out one replica row of any state array (ASYNCMESH_STATE_*), replica in
 * [0, R).  Same conventions as asyncmesh_read_params. */
int asyncmesh_read_state(asyncmesh *h, uint32_t stage, int which, int32_t replica,
                         float *dst, uint64_t n, int dst_on_device);

/* The same for coordinates first .. first+count-1 of the row only. */
int asyncmesh_read_state_range(asyncmesh *h, uint32_t stage, int which, int32_t replica,
                               uint64_t first, uint64_t count, float *dst, int dst_on_device);

/*
 * Membership of the subset S_stage^step as the device computes it: bit (mu & 7)
 * of bitmap_host[mu >> 3] is coordinate mu; (numel + 7) / 8 bytes, host memory.
 * Rule: Philox-4x32-10 with key = (seed lo, seed hi) and counter
 * (mu >> 2, stage, (uint32) step, 0); coordinate mu takes word mu & 3 and is
 * in the subset iff word < floor(p * 2^32).
 */
int asyncmesh_subset_mask(asyncmesh *h, uint32_t stage, uint64_t step,
                          uint8_t *bitmap_host);

/*
 * Consensus error of a stage, sum_i ||w_i - wbar||^2 (Section 3.3), reduced on
 * the device in double precision.  Waits for the stream.  With
 * ASYNCMESH_FLAG_TRACK_CONSENSUS (where honoured) and at least one step taken it is
 * the value the last step accumulated on its way; otherwise a read-only pass over
 * the stage's weights.  The two agree to rounding of the double sum (its order
 * differs).
 */
int asyncmesh_consensus_error(asyncmesh *h, uint32_t stage, double *out_host);

/*
 * The consensus error again (the quantity asyncmesh_consensus_error returns), for
 * callers that cannot let the library allocate (the paper has no counterpart: this
 * is a packaging variant of that call, not part of the method).  Meant for hosts whose GPU memory is entirely owned by their
 * own pool, for loops that must not hit the device-wide synchronisation an
 * allocation may cause, and for hooks that run where the process may not grow:
 * it calls no cudaMalloc / cudaFree and no allocating library routine.  The
 * reduction's scratch (per-block partial sums) is a fixed 33 KB array inside
 * the library image, present on every GPU that loads the library until the
 * process exits.
 *   w_device    device, [R][row_stride] fp32 (e.g. from asyncmesh_lookahead_weights
 *               with delay 0), read-only, caller-owned
 *   n           coordinates per row, 1 .. 2^28 (65536 per block x 4096 blocks of
 *               scratch); larger n is rejected with INVALID_ARG and a message:
 *               split the rows and add the partial results
 *   out_host    host, receives sum_i ||w_i - wbar||^2 over the n coordinates
 *   device, stream   where to run; the call waits for the stream before returning
 * The first call on a device also looks up the scratch array's device address
 * (with lazy module loading that is also when the array comes into existence on
 * that device); make that first call before any stream capture.  All calls share the one
 * array and it keeps the last call's contents (every slot a call reads it has
 * written first, so nothing needs clearing); two calls whose kernels overlap on
 * the GPU (different streams, different threads) race on it and must be
 * serialised by the caller.
 */
int asyncmesh_consensus_error_noalloc(int device, void *stream, const float *w_device,
                                      uint32_t R, uint64_t n, uint64_t row_stride,
                                      double *out_host);

/*
 * Spread of the staleness estimates across replicas (the appendix figure on the
 * consensus error plots the "variance between EMA estimates in each replica",
 * mean and max across the model dimension): per coordinate the population
 * variance (1/R) sum_i (d_i - dbar)^2, formed in double on the device;
 * *mean_host = its mean over the stage's coordinates, *max_host = its maximum
 * (host doubles, both required).  Waits for the stream.
 */
int asyncmesh_ema_variance(asyncmesh *h, uint32_t stage, double *mean_host, double *max_host);

/* Steps taken so far.  (Bookkeeping, like asyncmesh_status and
 * asyncmesh_last_error: defines nothing of the paper's method.) */
int asyncmesh_step_count(const asyncmesh *h, uint64_t *t);

/*
 * Which step kernel the handle runs, as text, e.g.
 * "owner R=4 compact entries=32": the kernel family (direct, pipelined, owner),
 * the replica count it is compiled for, the ring mode (sync, compact, dense) and
 * the shape parameter of the family.  Fixed at create.  Copies at most cap bytes
 * including the terminating 0 into buf (host).  Measurements (DRAM traffic per
 * launch, for instance) are filed under this name.  Bookkeeping only.
 */
int asyncmesh_kernel_name(const asyncmesh *h, char *buf, size_t cap);

/*
 * Bytes the last step had to move at least: per replica-coordinate 16 read
 * (w, g, m, v) + 12 written (w, m, v), + 4 where the look-ahead is a separate
 * buffer, + 4p for the snapshot write, + 12p once averages are being consumed
 * (ring read, d read, d write).  Used as the numerator of the HBM roofline.
 * (Bookkeeping: defines nothing of the paper's method.)
 */
int asyncmesh_min_bytes_last_step(const asyncmesh *h, uint64_t *bytes);

/* Wait for the stream and report a device-side status word: OK, or
 * DEVICE_STATUS if a snapshot ring slot overflowed its capacity. */
int asyncmesh_status(asyncmesh *h);

/* Run the device's Philox-4x32-10 on n (counter, key) pairs: ctr_host [n][4],
 * key_host [n][2], out_host [n][4], all uint32 in host memory.  Test hook: it has no
 * handle, so its three temporary device buffers come from cudaMalloc / cudaFree, not
 * from a handle's allocator callbacks.  (The generator is the published one, Salmon et
 * al., SC'11; Section 2.3 of the paper only asks for a randomly sampled subset.) */
int asyncmesh_debug_philox(int device, const uint32_t *ctr_host,
                           const uint32_t *key_host, uint32_t *out_host, uint64_t n);

/* Message of the calling thread's most recent failure ("" if none). */
const char *asyncmesh_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* ASYNCMESH_H */
