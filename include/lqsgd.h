/*
 * lqsgd.h - C ABI of the LQ-SGD compression round for NVIDIA B200 (sm_100a).
 *
 * One call of lqsgd_step() runs the body of Algorithm 1 of "Trustworthy Efficient
 * Communication for Distributed Learning using LQ-SGD Algorithm" for a whole set of layer
 * gradients and W data-parallel workers whose gradients all live on one GPU:
 *
 *   M_w   = G_w + E_w                          error feedback        (Eq. 8)
 *   P_w   = Orthonormalize(M_w Q)              power step            (Alg. 1)
 *   P_bar = LogDequantize(mean_w LogQuantize(P_w, b_p, alpha))       (Eq. 4, Eq. 5, Eq. 1)
 *   Q_w   = M_w^T P_bar                        second power step     (Alg. 1)
 *   Q_bar = LogDequantize(mean_w LogQuantize(Q_w, b_q, alpha))
 *   G_hat = P_bar Q_bar^T                      reconstruction        (Eq. 6)
 *   E_w   = M_w - G_hat                        error update          (Eq. 7)
 *   Q     = Q_bar                              warm start of the next call
 *
 * Notation (Section IV): a layer gradient G is n x m, row-major, n = rows (C_out) and
 * m = cols (C_in*k*k); P is n x r, Q is m x r; r_eff = min(rank, n, m) columns are used.
 * A tensor with rows == 1 or cols == 1 is one-dimensional: it bypasses the low-rank path
 * and is averaged over the workers in fp32 (Eq. 1).
 *
 * Quantiser.  A b-bit code is one sign bit (the top bit of the code, set iff x < 0) and
 * b-1 magnitude bits holding the level index k in 0..L-1, L = 2^(b-1).  Levels are uniform
 * in the companded domain of Eq. 4, |q|_k = k/(L-1); k is the level nearest to
 * q(|x|/s), an exact half rounding up.  s is one fp32 scale per factor and layer, the largest
 * |x| over all workers; |x|/s is an IEEE fp32 division.  The worker average is the exact
 * integer sum S of the signed level indices divided by W(L-1), to which Eq. 5 is applied once.
 *
 * Memory.  The library allocates no device memory: the caller passes one workspace whose size
 * lqsgd_workspace_bytes() reports and keeps it alive, untouched, until lqsgd_destroy().  The
 * error buffers E_w and the warm-start Q live in that workspace and persist across steps.
 * All pointers named "dev_*" (and the entries of grads / ghat) are device pointers on the
 * device that was current at lqsgd_create(); pointers named "host_*" are host pointers.
 *
 * Errors.  Every function returns LQSGD_OK (0) or a negative lqsgd_error; nothing throws,
 * aborts or traps.  Argument errors are detected on the host before anything is launched.
 * Numerical conditions met on the device (a dependent column, a zero scale, a non-finite
 * value) never fault: they produce the defined result below and set a bit in the per-layer
 * status word (lqsgd_status).
 *
 * Threading.  A context may be used from one host thread at a time.  lqsgd_step() is
 * asynchronous on the given stream; steps issued on different streams must be ordered by the
 * caller.
 */
#ifndef LQSGD_H_
#define LQSGD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define LQSGD_VERSION 1

typedef enum lqsgd_error {
  LQSGD_OK = 0,
  LQSGD_ERR_INVALID_ARG = -1,         /* null pointer, bad struct_size, rank/bits/alpha/workers out of range */
  LQSGD_ERR_BAD_SHAPE = -2,           /* rows or cols < 1, or too large */
  LQSGD_ERR_WORKSPACE_TOO_SMALL = -3,
  LQSGD_ERR_MISALIGNED = -4,          /* workspace not 256-byte aligned, tensor pointer not aligned */
  LQSGD_ERR_CUDA = -5,                /* a CUDA runtime call failed; see lqsgd_last_cuda_error() */
  LQSGD_ERR_NO_STAGING = -6,          /* lqsgd_step_host() on a context created without LQSGD_FLAG_HOST_STAGING */
  LQSGD_ERR_OUT_OF_RANGE = -7,        /* layer / worker / state index out of range, or state not defined for that layer */
  LQSGD_ERR_TOO_LARGE = -8,           /* size beyond the fixed built-in scratch of lqsgd_orthonormalize_noalloc */
  LQSGD_ERR_CAPTURE = -9,             /* stream is capturing and the tensor pointers differ from the previous call's */
  LQSGD_ERR_PLAN = -10                /* lqsgd_plan_check: the work tables of this configuration fail an invariant (a defect of the library) */
} lqsgd_error;

/* Bits of the per-layer status word. */
#define LQSGD_STATUS_DEPENDENT_COLUMN 1u /* a column of M Q was zero or linearly dependent: it became a zero column */
#define LQSGD_STATUS_ZERO_SCALE_P     2u /* every P entry was 0: codes and P_bar are 0 */
#define LQSGD_STATUS_ZERO_SCALE_Q     4u /* every Q entry was 0: codes and Q_bar are 0 */
#define LQSGD_STATUS_NONFINITE        8u /* a scale was inf or nan: the layer's outputs are undefined (no fault) */
#define LQSGD_STATUS_TIMEOUT         16u /* a bounded device-side wait ran out: the step's outputs are undefined */

/* Config flags. */
#define LQSGD_FLAG_HOST_STAGING 1u /* reserve device staging in the workspace so that lqsgd_step_host() works */
#define LQSGD_FLAG_REGISTER_PATH 2u /* stream every layer with the register-path kernels (no bulk-copy staging) */
#define LQSGD_FLAG_AVERAGE_VALUES 4u /* variant of the exchange: Eq. 5 on every worker's quantised factor, then the mean
                                        of Eq. 1 over the dequantised values (a parameter server that decodes what it
                                        receives, Section V).  Default, as Algorithm 1 writes it: mean of the quantised
                                        values, then Eq. 5 once.  Codes, scales and payload are the same in both. */

#define LQSGD_FLAG_QUANTIZE_VECTORS 8u /* variant: the 1-D tensors go through the same exchange as a factor (one fp32 scale
                                         = max over workers and entries, bits_p bits per entry, Eq. 4 / Eq. 5) instead of
                                         travelling as fp32.  Payload: [s_P, s_Q per matrix][one scale per 1-D tensor]
                                         [their code streams][P streams][Q streams].  Ignored with bits_p = 32; not
                                         available with workers on several GPUs (lqsgd_round_begin refuses). */
#define LQSGD_FLAG_COLUMN_SCALES 16u /* variant: one scale per COLUMN of a factor, s_j = max over workers and rows of
                                        |x[:, j]|, instead of one per factor; column j is normalised by s_j in Eq. 4 and
                                        rescaled by s_j after Eq. 5.  A matrix then sends 2 r_eff scales: in the payload
                                        s_P[0..r_eff) is followed by s_Q[0..r_eff) (8 r_eff bytes at scale_offset), and
                                        LQSGD_STATE_SCALES is fp32 [2][r_eff].  The zero-scale status bits are set when
                                        any column's scale is 0 (that column's codes and averages are 0). */

#define LQSGD_FLAG_ONE_LAUNCH 32u /* run the round as ONE cooperative kernel that keeps M = G + E in the SMs' shared memory
                                     from the first product to the error update (12 + 4/W instead of 24 + 4/W bytes of
                                     memory traffic per worker-element), when the set qualifies: W * sum(n m) fp32 values
                                     fit in the shared memory of all SMs together (about 27 MB on a B200), rank <= 8,
                                     plain Algorithm 1 exchange or its variants except quantised 1-D tensors, one power
                                     iteration, all workers on this GPU.  A set that does not qualify runs as the usual
                                     sequence of kernels (lqsgd_launches_per_step tells which: 1 = one launch).  Same
                                     results up to the order of the floating-point sums.  Off by default: the sequence of
                                     kernels is the faster of the two on the sets measured so far. */

#define LQSGD_FLAG_GUARD_WORDS 64u /* debugging aid: every piece the library carves out of the workspace (error buffers,
                                      factors, partial sums, payloads, tables ...) is followed by 256 bytes of a fixed
                                      pattern that no kernel may write; lqsgd_check_guards tells whether any changed,
                                      i.e. whether a kernel wrote past the end of its piece.  Costs a little workspace. */

typedef struct lqsgd_ctx lqsgd_ctx;

typedef struct lqsgd_shape {
  int32_t rows; /* n */
  int32_t cols; /* m */
} lqsgd_shape;

/* Inputs of Algorithm 1 (rank r, bits b_p and b_q, curvature alpha) plus the worker count. */
typedef struct lqsgd_config {
  uint32_t struct_size; /* sizeof(lqsgd_config), for versioning */
  int32_t rank;         /* r, 1..64 (any integer); from 9 up the products of aligned layers run on the tensor cores */
  int32_t bits_p;       /* b_p, total bits per P scalar including the sign, 2..8; 32 = no quantiser: the
                           factor is sent as fp32 and averaged directly (the PowerSGD exchange of Section III-B) */
  int32_t bits_q;       /* b_q, likewise for Q */
  float alpha;          /* alpha of Eq. 4 / Eq. 5, finite and > 0 */
  int32_t workers;      /* W, 1..256 */
  uint64_t seed;        /* seed of Q_0 ~ N(0,1) (Alg. 1 initialisation) */
  uint32_t flags;       /* LQSGD_FLAG_* */
  int32_t world_workers; /* 0, or the number of workers of ALL processes taking part in the averages when the
                            workers are spread over several GPUs (a multiple of `workers`); see lqsgd_round_begin */
  int32_t power_iters;   /* 0 or 1: Algorithm 1 (one power step per round).  2..8 (an option): the power step with its
                            two exchanges is repeated on the same M = G + E, each time from the Q_bar just obtained; the
                            payload holds the streams of the last repetition (each repetition sends as much).  Needs a
                            zero buffer of the largest matrix in the workspace; not with workers on several GPUs. */
} lqsgd_config;

/* Where one layer's data sits inside a worker's payload (byte offsets from the payload start). */
typedef struct lqsgd_layer_layout {
  int32_t is_matrix;     /* 1: low-rank path, 0: one-dimensional tensor sent as fp32 */
  int32_t rank_eff;      /* r_eff (0 for a 1-D tensor) */
  uint64_t scale_offset; /* matrix: fp32 s_P then fp32 s_Q (LQSGD_FLAG_COLUMN_SCALES: r_eff values each);
                            quantised 1-D tensor: its fp32 scale */
  uint64_t p_offset;     /* matrix: P code stream, p_bytes = ceil(n * r_eff * b_p / 8) */
  uint64_t p_bytes;
  uint64_t q_offset;     /* matrix: Q code stream, q_bytes = ceil(m * r_eff * b_q / 8) */
  uint64_t q_bytes;
  uint64_t vec_offset;   /* 1-D tensor: rows*cols fp32 values, or (LQSGD_FLAG_QUANTIZE_VECTORS) its code stream */
  uint64_t vec_bytes;
} lqsgd_layer_layout;

/* State that lqsgd_get_state / lqsgd_set_state can copy.  Shapes are dense (no padding),
 * row-major.  "per worker" states take a worker index, the others ignore it. */
typedef enum lqsgd_state {
  LQSGD_STATE_E = 0,       /* fp32 n x m, per worker: error buffer (Eq. 7); settable */
  LQSGD_STATE_Q = 1,       /* fp32 m x r_eff: warm-start Q (Q_0, then Q_bar of the last step); settable */
  LQSGD_STATE_P_RAW = 2,   /* fp32 n x r_eff, per worker: M Q of the last step, before Orthonormalize */
  LQSGD_STATE_P = 3,       /* fp32 n x r_eff, per worker: orthonormal P of the last step */
  LQSGD_STATE_P_BAR = 4,   /* fp32 n x r_eff: dequantised worker average of P */
  LQSGD_STATE_Q_W = 5,     /* fp32 m x r_eff, per worker: M^T P_bar of the last step */
  LQSGD_STATE_CODES_P = 6, /* uint8 n x r_eff, per worker: one unpacked code per byte (not with bits 32) */
  LQSGD_STATE_CODES_Q = 7, /* uint8 m x r_eff, per worker */
  LQSGD_STATE_SCALES = 8   /* fp32 [2]: s_P, s_Q of the last step (LQSGD_FLAG_COLUMN_SCALES: fp32 [2][r_eff]) */
} lqsgd_state;

/* Bytes of device workspace a context for these layers needs (Algorithm 1 state E, Q, plus
 * factors, partial sums, codes, payload and tables).  Host-only; launches nothing. */
int lqsgd_workspace_bytes(const lqsgd_shape* host_shapes, int32_t n_layers,
                          const lqsgd_config* host_config, size_t* host_bytes_out);

/* Creates a context on the current device.  dev_workspace: caller-owned device memory,
 * 256-byte aligned, at least lqsgd_workspace_bytes() long; the library carves it and owns its
 * contents until lqsgd_destroy().  Initialises E_0 = 0 and Q_0 ~ N(0,1) from config->seed
 * (Alg. 1 initialisation; the same Q_0 for every worker) and uploads the planning tables:
 * it issues copies and a memset on the legacy default stream and synchronises it.
 * The context itself is host memory owned by the library.  Device memory is never allocated; a context whose layer set
 * has both large layers and small ones with rows that are not 16-byte aligned also owns one non-blocking CUDA stream
 * and two events (released by lqsgd_destroy): in every pass the small layers' kernel runs on that stream beside the
 * large layers' kernel, forked from and joined to the caller's stream inside the call, also under stream capture. */
int lqsgd_create(const lqsgd_shape* host_shapes, int32_t n_layers, const lqsgd_config* host_config,
                 void* dev_workspace, size_t workspace_bytes, lqsgd_ctx** ctx_out);

/* One round of Algorithm 1 (error feedback to error update) for every layer.
 * host_grads: host array of W * n_layers device pointers, worker-major
 *   (host_grads[w * n_layers + l] = G of layer l on worker w), fp32 row-major contiguous,
 *   read-only; a matrix whose cols is a multiple of 4 must be 16-byte aligned.
 * host_ghat: host array of n_layers device pointers; host_ghat[l] receives G_hat of layer l
 *   (or the worker mean of a 1-D tensor), same shape as the gradient; overwritten.
 *   Must not alias any gradient.
 * cuda_stream: a cudaStream_t (NULL = legacy default stream).  The call only enqueues work;
 *   results, payload and state are valid once the stream has reached the end of that work.
 *   The pointer arrays themselves are consumed before the call returns.
 * Pointer tables: the context keeps device copies of the tables of the last 16 distinct pointer
 *   sets it was called with; a call with one of them enqueues kernels only (no copy between two
 *   rounds), any other set costs one small host-to-device copy on the stream.
 * CUDA graphs: the call may be made on a capturing stream when its tensor pointers equal those
 *   of an earlier call on this context whose table is still kept (the captured work is then
 *   kernels only; the graph reads and writes those same tensors at every replay, and its table
 *   is kept for the life of the context).  With other pointers a capturing stream gets
 *   LQSGD_ERR_CAPTURE and nothing is enqueued: the upload of the pointer table cannot be part of
 *   a graph.  (Also returned once 16 tables belong to captured graphs and a 17th set arrives.) */
int lqsgd_step(lqsgd_ctx* ctx, const float* const* host_grads, float* const* host_ghat,
               void* cuda_stream);

/* Declares that every CUDA graph captured from this context's steps has been destroyed (or will never be
 * replayed again): the pointer tables those captures pinned may be reused from now on.  Without this call a
 * trainer that re-captures its step with new tensors would, after 16 captured pointer sets, get
 * LQSGD_ERR_CAPTURE for every new set.  Replaying an old graph after this call reads whatever table has
 * taken its slot since: do not.  Host-only. */
int lqsgd_release_graph_tables(lqsgd_ctx* ctx);

/* lqsgd_step followed, inside the reconstruction pass, by the model update that ends an
 * iteration of Algorithm 1:  w <- w - lr * G_hat  for every layer (for a 1-D tensor G_hat is the
 * worker mean).  host_weights: host array of n_layers device pointers, fp32, shaped and aligned
 * like the gradients, updated in place; an entry may be NULL (that layer is not updated).
 * host_ghat may be NULL, or hold NULL entries: G_hat of those layers is then not written at all,
 * which saves its 4/W bytes per worker-element of traffic; every layer needs at least one of the two.
 * Everything else as lqsgd_step. */
int lqsgd_step_update(lqsgd_ctx* ctx, const float* const* host_grads, float* const* host_ghat,
                      float* const* host_weights, float lr, void* cuda_stream);

/* ---- Workers on several GPUs: the round in pieces, with the exchanges left to the caller. ----
 * Algorithm 1 has two All-Reduce steps per iteration, one for each quantised factor (Section IV-A).
 * With the workers of one process on one GPU that exchange is a sum inside lqsgd_step.  When
 * other processes hold more workers (config.world_workers = total over all ranks, each rank
 * simulating `workers` of them), a rank runs the round as
 *
 *   lqsgd_round_begin(grads, ghat, weights, lr)   pass 1, Orthonormalize, local scales of P, and this rank's
 *                                                  share of every 1-D tensor's mean into one flat buffer
 *   all-reduce MAX over ranks of  view(LQSGD_XCHG_SCALES_P)     (one fp32 per matrix; r_eff per matrix padded to the
 *                                                                padded rank with LQSGD_FLAG_COLUMN_SCALES)
 *   lqsgd_round_pack(0)                            quantise + pack this rank's P with those scales
 *   all-gather of                 view(LQSGD_XCHG_STREAMS_P)    (workers x P-stream bytes, contiguous)
 *   lqsgd_round_reduce(0, gathered, n_ranks)       exact integer sum over ALL workers' codes,
 *                                                  Eq. 5, pass 2, local scales of Q
 *   all-reduce MAX of view(LQSGD_XCHG_SCALES_Q);  lqsgd_round_pack(1);  all-gather of
 *   view(LQSGD_XCHG_STREAMS_Q);  lqsgd_round_reduce(1, gathered, n_ranks)
 *   all-reduce SUM of view(LQSGD_XCHG_VECTORS)     (the 1-D tensors, fp32, all in one buffer; any time after begin)
 *   lqsgd_round_end()                              pass 3 (G_hat, E, optional model update); the 1-D tensors'
 *                                                  means go to their G_hat tensors and into the weights
 *
 * The collectives run on the same stream between the calls (NCCL, or any other transport: the
 * library only reads and writes the buffers).  `gathered` is n_ranks x the bytes of the STREAMS
 * view, rank after rank, in caller memory.  The wire carries exactly the b-bit streams
 * (r(n+m)b bits per worker, Section IV-C) plus one scale per factor and layer - five collectives per round,
 * whatever the number of layers.  With bits = 32 the streams are the fp32 factors and the scales are not used
 * (the PowerSGD exchange of Section III-B).  Results are identical, bit for bit, to one process simulating all
 * world_workers workers (the 1-D means up to the order of their sum).  Calls out of order return
 * LQSGD_ERR_INVALID_ARG; quantised 1-D tensors and several power iterations are not available across ranks.
 * ghat / weights as in lqsgd_step_update (weights may be NULL). */
#define LQSGD_XCHG_SCALES_P 0
#define LQSGD_XCHG_SCALES_Q 1
#define LQSGD_XCHG_STREAMS_P 2
#define LQSGD_XCHG_STREAMS_Q 3
#define LQSGD_XCHG_VECTORS 4
int lqsgd_round_begin(lqsgd_ctx* ctx, const float* const* host_grads, float* const* host_ghat,
                      float* const* host_weights, float lr, void* cuda_stream);
int lqsgd_round_pack(lqsgd_ctx* ctx, int32_t which, void* cuda_stream);
int lqsgd_round_reduce(lqsgd_ctx* ctx, int32_t which, const void* dev_gathered, int32_t n_ranks, void* cuda_stream);
int lqsgd_round_end(lqsgd_ctx* ctx, void* cuda_stream);
int lqsgd_exchange_view(const lqsgd_ctx* ctx, int32_t which, void** dev_ptr_out, size_t* host_bytes_out);

/* Same round with HOST tensors: copies every gradient host->device into the staging area,
 * runs lqsgd_step, copies every G_hat and all W payloads device->host, and synchronises the
 * stream before returning.  host_grads / host_ghat are arrays of host pointers laid out as in
 * lqsgd_step (pinned memory makes the copies asynchronous to each other, pageable works);
 * host_payload (may be NULL) receives W * payload_bytes bytes, worker after worker.
 * The staging area holds a worker's tensors in layer order, each starting on a 16-byte boundary; host tensors
 * that follow one another in memory the same way (one flat gradient buffer per worker, tensors 16-byte aligned)
 * are copied in one piece instead of one copy per tensor, and likewise the G_hat outputs.
 * Needs LQSGD_FLAG_HOST_STAGING. */
int lqsgd_step_host(lqsgd_ctx* ctx, const float* const* host_grads, float* const* host_ghat,
                    void* host_payload, void* cuda_stream);

/* Size of one worker's payload in bytes (Section IV-C: r(n+m)b bits per matrix, each code
 * stream padded to a byte, + 8 bytes of scales per matrix (8 r_eff with LQSGD_FLAG_COLUMN_SCALES)
 * + 4 bytes per 1-D scalar). */
int lqsgd_payload_bytes(const lqsgd_ctx* ctx, size_t* host_bytes_out);

/* Device view of what worker `worker` sends in the last enqueued step: valid until the next
 * step.  Order: [s_P, s_Q of every matrix][every 1-D tensor, fp32][P code streams][Q code
 * streams], each in layer order; a code stream is a little-endian bit stream in which element
 * i of the row-major n x r_eff (or m x r_eff) factor occupies bits [i*b, (i+1)*b). */
int lqsgd_payload(const lqsgd_ctx* ctx, int32_t worker, const void** dev_ptr_out, size_t* host_bytes_out);

int lqsgd_payload_layout(const lqsgd_ctx* ctx, int32_t layer, lqsgd_layer_layout* host_out);

/* Copies one piece of state to / from caller device memory (dense, row-major; see lqsgd_state),
 * asynchronously on cuda_stream.  Setting E or Q is how a checkpoint is restored. */
int lqsgd_get_state(const lqsgd_ctx* ctx, int32_t which, int32_t layer, int32_t worker,
                    void* dev_dst, void* cuda_stream);
int lqsgd_set_state(lqsgd_ctx* ctx, int32_t which, int32_t layer, int32_t worker,
                    const void* dev_src, void* cuda_stream);

/* Copies the per-layer status words of the last step into host_flags[n_layers];
 * synchronises cuda_stream. */
int lqsgd_status(const lqsgd_ctx* ctx, uint32_t* host_flags, void* cuda_stream);

/* Figures of the last round for one layer (a logging aid; nothing on the round's path computes them). */
typedef struct lqsgd_layer_stats {
  uint32_t status;         /* the layer's status word (LQSGD_STATUS_*) */
  int32_t rank_eff;        /* r_eff; 0 for a 1-D tensor, whose other fields are then 0 except payload_bytes */
  float scale_p, scale_q;  /* s_P, s_Q of Eq. 4's normalisation (LQSGD_FLAG_COLUMN_SCALES: the largest column scale) */
  float pivot_ratio;       /* conditioning of the factor given to Orthonormalize (Algorithm 1): with M Q = P R, R upper
                              triangular, min_j R_jj / max_j R_jj, the smallest over this GPU's workers; 0 when a column
                              was dropped (LQSGD_STATUS_DEPENDENT_COLUMN) */
  uint32_t pad_;
  uint64_t codes_p, codes_q; /* factor entries quantised by Eq. 4 over this GPU's workers: W n r_eff and W m r_eff
                                (0 with bits 32) */
  uint64_t near_p, near_q;   /* of them, entries whose |x| / s lies within one fp32 step of a decision threshold: the
                                two fp32 neighbours of |x| / s fall into different levels.  Only for these may an
                                implementation that rounds |x| / s differently in the last place produce another code */
  uint64_t payload_bytes;    /* this layer's bytes in one worker's payload (scales + P stream + Q stream, or the 1-D
                                tensor's values) */
} lqsgd_layer_stats;

/* Fills host_out for one layer from what the last step left in the workspace (one small kernel over the layer's
 * factors on cuda_stream, then a copy of three words); synchronises cuda_stream.  Call it after a step on the same
 * stream, or after synchronising the step's stream.  Matrix layers whose round has not run yet report zeros. */
int lqsgd_step_stats(const lqsgd_ctx* ctx, int32_t layer, lqsgd_layer_stats* host_out, void* cuda_stream);

/* Profiling aid.  host_events: LQSGD_N_PHASES + 1 cudaEvent_t handles owned by the caller (or
 * NULL to cancel).  The NEXT lqsgd_step records them on its stream at the phase boundaries and
 * then forgets them: event i before phase i, the last one after phase LQSGD_N_PHASES - 1.
 * Phases: 0 = pass 1 (error feedback + M Q), 1 = orthonormalise / quantise / average P,
 * 2 = pass 2 (M^T P_bar), 3 = quantise / average Q, 4 = pass 3 (G_hat and E).  The handles are
 * copied before the call returns. */
#define LQSGD_N_PHASES 5
int lqsgd_set_phase_events(lqsgd_ctx* ctx, void* const* host_events);

/* TEST SUPPORT - exercises the path a bounded device-side wait takes when it runs out, without any fault.
 * The streaming passes wait on shared-memory barriers for their asynchronous copies; every such wait gives up
 * after a fixed number of timed polls, the CTA's roles then leave their loops, copies in flight are waited for,
 * tensor memory is released, the layer's status word gets LQSGD_STATUS_TIMEOUT and the kernel returns.  This
 * call arms the NEXT step only: in pass `pass` (1, 2 or 3; pass 2 only where it runs on the tensor cores) the
 * loader of CTA 0 issues no copies from its stage number `stage` on (counted from 0 over the CTA's tiles); with
 * pass = 4 (a context that runs the round as one launch) CTA 0 stays away from grid barrier number `stage`; and
 * every bounded wait of that step gives up after `wait_limit` polls (16 .. 2^18, about a microsecond each)
 * instead of the built-in 2^18.  All addresses stay valid and nothing spins without a limit; the step's outputs
 * (E of the affected layer included) are undefined, as after any time-out: restore E and Q with
 * lqsgd_set_state, or use a fresh context, before relying on results again.  If the armed pass has no such
 * stage the step runs normally.  Host-only; never needed in production. */
int lqsgd_test_expire_wait(lqsgd_ctx* ctx, int32_t pass, int32_t stage, uint32_t wait_limit);

/* Profiling aid for contexts that run the round as ONE launch (see LQSGD_FLAG_ONE_LAUNCH), where no event can be
 * recorded between the steps: the kernel itself notes the GPU's global timer (nanoseconds) as its first CTA starts,
 * ends its pass 1, leaves each grid barrier, and ends.  Copies the stamps of the last completed round into
 * host_ns[LQSGD_TIMELINE_MAX] and their number into *host_count (0 for a multi-kernel context); synchronises
 * cuda_stream.  Stamps, in order: start | end of pass 1 on CTA 0 | Orthonormalize begins | (with tall layers:
 * Cholesky and solve begin; else the same instant as the next) | P_bar and pass 2 begin | Q_w reduction begins |
 * Q_bar and pass 3 begin | end. */
#define LQSGD_TIMELINE_MAX 12
int lqsgd_round_timeline(const lqsgd_ctx* ctx, uint64_t* host_ns, int32_t* host_count, void* cuda_stream);

/* Contexts created with LQSGD_FLAG_GUARD_WORDS: checks the guard blocks between the pieces of the workspace after
 * everything enqueued on cuda_stream so far, and synchronises it.  *host_changed_words receives the number of
 * 32-bit guard words that no longer hold their pattern (0 = no kernel wrote outside its piece),
 * *host_first_offset (may be NULL) the byte offset in the workspace of the first of them, or -1.
 * LQSGD_ERR_INVALID_ARG for a context without guards. */
int lqsgd_check_guards(const lqsgd_ctx* ctx, int64_t* host_changed_words, int64_t* host_first_offset, void* cuda_stream);

/* Host-only self-check of the work tables the library would build for this configuration on a device with sm_count
 * SMs (148 on a B200; the tile sizes depend on it): no device is touched, nothing is allocated on one.  Verifies
 * that every pass's tiles cover every (layer, worker, row, column) exactly once, that the partial sums each tile
 * writes (Section IV-A's two products, summed over column or row chunks) are exactly the ones the following step
 * adds up, that the factor blocks and exchange chunks cover every factor element once, and that the second-level
 * sums of layers with many partial sums take every partial once.  Returns LQSGD_OK, the configuration's own error
 * (as lqsgd_workspace_bytes), or LQSGD_ERR_PLAN with a description of the first failed invariant in msg (may be
 * NULL; at most msg_len bytes including the terminator).  Meant for tests: a planner defect shows here, on the
 * CPU, for any shape, before a kernel runs on wrong tables. */
int lqsgd_plan_check(const lqsgd_shape* shapes, int32_t n_layers, const lqsgd_config* cfg, int32_t sm_count, char* msg,
                     size_t msg_len);

/* Test support for lqsgd_plan_check: the calling thread's NEXT lqsgd_plan_check first damages its (private) copy of
 * the tables and must then report LQSGD_ERR_PLAN: kind 1 drops a tile of pass 1, 2 gives two tiles of pass 2 the same
 * partial-sum slot, 3 drops the last tile of pass 3 (for a tile with ranges of workers: its last range), 4 drops a
 * second-level sum (configurations with none stay undamaged), 5 drops an exchange chunk of Q.  0 disarms.  Nothing a context uses is touched. */
int lqsgd_test_plan_defect(int32_t kind);

/* Kernel launches one lqsgd_step enqueues (for launch accounting). */
int lqsgd_launches_per_step(const lqsgd_ctx* ctx, int32_t* host_out);

/* Orthonormalises the columns of one rows x rank factor with NO workspace and NO allocation.
 * (The paper has no counterpart: this is a packaging of the Orthonormalize step for callers that
 * cannot obtain device memory - every byte is owned by another allocator or a start-up budget -
 * or may not call cudaMalloc because it stalls the device, e.g. from a serving loop or from a
 * callback inside another library.  They pass only the input and the output.)
 * dev_p_in: fp32, dense row-major rows x rank, 4-byte aligned, read-only.  dev_p_out: same shape,
 * overwritten with the thin-QR Q factor (positive-diagonal R; a zero or dependent column becomes
 * zero); may be the same pointer as dev_p_in, must not overlap it otherwise.  dev_status_out:
 * NULL, or one device uint32 that receives LQSGD_STATUS_* bits.  Asynchronous on cuda_stream.
 * Intermediate storage (block Gram matrices, R^-1: about 1 MiB) is a fixed array inside the
 * library image, present once on every GPU that loads the library until the process exits:
 *  - rows > LQSGD_NOALLOC_MAX_ROWS or rank > 16 returns LQSGD_ERR_TOO_LARGE, nothing is launched;
 *  - all calls on a device share that array (it keeps the previous call's contents; the call
 *    clears what must start at zero): calls that can overlap on the GPU race - order them on one
 *    stream or with events;
 *  - the first call on each device queries the array's device address (no allocation); make
 *    that first call before any stream capture begins.
 * Calls no cudaMalloc / cudaFree and no allocating library routine. */
#define LQSGD_NOALLOC_MAX_ROWS 65536
int lqsgd_orthonormalize_noalloc(const float* dev_p_in, float* dev_p_out, int32_t rows, int32_t rank,
                                 uint32_t* dev_status_out, void* cuda_stream);

/* Frees the host-side context.  The workspace stays the caller's. */
void lqsgd_destroy(lqsgd_ctx* ctx);

const char* lqsgd_strerror(int code);
/* Text of the last CUDA error this library saw on the calling thread ("" if none). */
const char* lqsgd_last_cuda_error(void);
int lqsgd_version(void);

#ifdef __cplusplus
}
#endif
#endif /* LQSGD_H_ */
