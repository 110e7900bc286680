/* libef: one two-way compressed step of dist-EF-blockSGDM on a single B200.
 *
 * The library implements the data-parallel hot path of Algorithm 4 (distributed blockwise
 * momentum SGD with error feedback) of arXiv 1905.10936 for M simulated workers that all
 * live on one GPU.  One iteration t is
 *
 *     for each worker i in [0, M):  ef_worker_step(ctx, i, g_{t,i})     (or one ef_worker_step_all)
 *     ef_server_step(ctx)
 *
 * Further down: the stepsize sequence and the weight-decay side path, per-block diagnostics,
 * the same iteration in pieces for one worker per GPU with a block-sharded server (fused
 * messages), layouts cut inside blocks, the paper's comparison compressors (signum with
 * majority vote, top-k), and a few entry points without a counterpart in the paper
 * (measurement aid, checked build, no-allocation worker step).
 *
 * All entry points are plain C.  "device" pointers are CUDA device pointers of the current
 * device, "host" pointers are ordinary host pointers.  The library never allocates device
 * memory: the caller hands over one workspace (size from ef_workspace_bytes) and keeps
 * owning it.  Every call only enqueues work on the CUDA stream given to ef_init and returns
 * without synchronising; results are ordered on that stream.
 *
 * Because the step calls (ef_worker_step, ef_server_step) only enqueue kernels on that stream,
 * a caller may record them into a CUDA graph by capturing the stream; the host-side counters
 * and call-order checks then see the captured calls only, not the replays.
 *
 * A context is not thread-safe: use it from one host thread at a time.  Different contexts
 * are independent (the no-allocation entry point at the end of this file is the exception: its
 * calls share one scratch array per device).
 *
 * There is no CPU fallback: on a device that is not compute capability 10.x ef_init fails
 * with EF_ERR_UNSUPPORTED_DEVICE.
 *
 * Packed sign layout (a convention of this library; the paper only fixes "one bit per sign
 * in {-1,+1}", Appendix A): block b owns ceil(d_b/32) consecutive 32-bit words, blocks in
 * order, every block starting on a word boundary.  Element k of the block is bit (k mod 32),
 * least significant bit first, of the block's word floor(k/32).  Bit 1 means the element is
 * negative (decodes to -1), bit 0 means it is >= 0 (decodes to +1; sign(+-0) = +1).  Unused
 * high bits of a block's last word are 0.  Scales are B consecutive floats, scale_b =
 * ||v_{G_b}||_1 / d_b (Section 3.2).  The decoded message is Delta_j = (bit ? -1 : +1) * scale_b.
 */
#ifndef EF_H_
#define EF_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ef_ctx ef_ctx;   /* opaque host object; owns no device memory */

enum ef_status {
    EF_OK = 0,
    EF_ERR_INVALID_ARG = 1,        /* a size, index, pointer or hyper-parameter is out of range */
    EF_ERR_BAD_STATE = 2,          /* call order violated (see ef_worker_step / ef_server_step) */
    EF_ERR_WORKSPACE = 3,          /* workspace null or smaller than ef_workspace_bytes */
    EF_ERR_ALIGNMENT = 4,          /* a device pointer is not 16-byte aligned */
    EF_ERR_CUDA = 5,               /* a CUDA runtime call failed; see ef_last_cuda_error */
    EF_ERR_UNSUPPORTED_DEVICE = 6, /* current device is not compute capability 10.x */
    EF_ERR_TIMEOUT = 7,            /* a bounded device-side wait gave up (reported by ef_check_status) */
    EF_ERR_TOO_LARGE = 8,          /* ef_worker_step_noalloc: n exceeds EF_NOALLOC_MAX_ELEMS */
    EF_ERR_NO_MEMORY = 9,          /* a host allocation failed (the library allocates no device memory) */
    EF_ERR_BOUNDS = 10             /* checked build only: a kernel refused a work item that reached
                                      outside its arrays (reported by ef_check_status) */
};

/* Flags for ef_workspace_bytes / ef_init. */
#define EF_FLAG_HOST_STAGING 1u    /* reserve two d-float staging buffers for ef_worker_step_host */
/* How the per-block L1 sums of blocks larger than one tile are completed.  By default the
 * library chooses: inside the main kernels for small (launch-bound) problems, in a tiny
 * follow-up kernel for large (bandwidth-bound) ones.  Both give bit-identical scales.  At
 * most one of the two flags may be set. */
#define EF_FLAG_FUSED_SCALE 2u     /* always complete the sums inside the main kernels */
#define EF_FLAG_SPLIT_SCALE 4u     /* always use the follow-up kernel */
#define EF_FLAG_WEIGHT_DECAY 8u    /* reserve the d-float decay momentum for ef_set_weight_decay */
#define EF_FLAG_DIAGNOSTICS 16u    /* worker steps also record per-block sums (ef_worker_diagnostics);
                                      implies the follow-up scale kernel, excludes EF_FLAG_FUSED_SCALE */
#define EF_FLAG_ONE_LOCAL_WORKER 32u /* this process is ONE worker of M (the paper's setting: one worker
                                      per GPU) and the server of some block range: the workspace holds
                                      the state of a single worker (index 0 in every per-worker call),
                                      the other M-1 workers' messages arrive through
                                      ef_server_step_range.  ef_server_step, ef_worker_step_all over M
                                      gradients and the signum calls need all M workers locally. */
#define EF_FLAG_SERVER_NO_BULK 512u  /* The server kernel stages its inputs in shared memory with bulk
                                      copies (TMA) when the layout allows it (every block but the last a
                                      multiple of 128 elements, M <= 16) and with per-thread asynchronous
                                      copies otherwise; this flag forces the latter (for comparisons;
                                      results are identical). */
#define EF_FLAG_PROGRAMMATIC_LAUNCH 1024u /* Launch the kernels with programmatic stream serialization: each
                                      may be scheduled while its predecessor on the stream drains and waits
                                      on the device for the predecessor's results; the worker kernel loads
                                      the worker's own state, and the one-launch server kernel its x values,
                                      before that wait.  On B200 this shortens the launch-bound layouts whose
                                      worker launch is a single wave of CTAs (flat 2^20, M = 2: 16.4 -> 14.5-15.4 us
                                      per step from a CUDA graph) and does nothing for the others, so by
                                      default it is on only there (one-launch server call and all CTAs of
                                      the M workers resident at once) and this flag forces it everywhere;
                                      EF_FLAG_SEPARATE_UPDATE keeps ordinary launches.  Results are
                                      identical.  While it is on, kernels of the
                                      caller that write x or a worker's state through the raw pointers
                                      directly before a call must not signal programmatic completion early. */
#define EF_FLAG_SEPARATE_UPDATE 2048u /* On layouts of few chunks in which no block spans more than 16 chunks,
                                      ef_server_step runs the server lines and the parameter update as ONE
                                      kernel launched in thread-block clusters (a cluster per block; the
                                      block's scale is agreed at the cluster barrier and every CTA updates
                                      its own chunk of x); this flag keeps the two kernels every other
                                      layout uses (for comparisons; results are identical). */

/* Maximum number of simulated workers. */
#define EF_MAX_WORKERS 4096

/* Workspace size in bytes for a problem (Algorithm 4, "Input" and "Initialize" lines):
 * d parameters, B blocks given by B+1 non-decreasing host offsets with offsets[0] = 0,
 * offsets[B] = d and every block non-empty (1/d_b appears in Prop. 1), M workers.
 * Pure host computation; needs no GPU.  Errors: EF_ERR_INVALID_ARG. */
int ef_workspace_bytes(int64_t d, int32_t B, const int64_t* offsets /* host, B+1 */,
                       int32_t M, uint32_t flags, size_t* bytes /* out */);

/* Creates a context and initialises the state of Algorithm 4 in the workspace:
 * x_0 = 0, m_{-1,i} = 0, e_{0,i} = 0, etilde_0 = 0, t = 0 (Algorithm 4, "Initialize").
 * mu in [0, 1) is the momentum parameter, eta > 0 the stepsize eta_0.  The stepsize stays at
 * this value until ef_set_eta changes it; while it is constant the factor eta_{t-1}/eta_t of
 * Algorithm 4 is exactly 1 (at t = 0 it multiplies a zero residual).
 * workspace: device, 256-byte aligned, at least ef_workspace_bytes; borrowed until ef_destroy.
 * cuda_stream: a cudaStream_t (0 = default stream) on which all work of this context runs.
 * Errors: INVALID_ARG, WORKSPACE, ALIGNMENT, UNSUPPORTED_DEVICE, NO_MEMORY (host), CUDA.  On
 * error *out = NULL and nothing was launched. */
int ef_init(ef_ctx** out, int64_t d, int32_t B, const int64_t* offsets /* host, B+1 */,
            int32_t M, float mu, float eta, uint32_t flags,
            void* workspace /* device */, size_t workspace_bytes, void* cuda_stream);

/* Worker side of one iteration for worker i (Algorithm 4, the "on each worker i" lines):
 *   m_{t,i} = mu m_{t-1,i} + g_{t,i};  p_{t,i} = mu m_{t,i} + g_{t,i} + e_{t,i};
 *   Delta_{t,i} = C_B(p_{t,i}) (packed signs + one scale per block, Section 3.2);
 *   e_{t+1,i} = p_{t,i} - Delta_{t,i}.
 * grad: device, d floats, 16-byte aligned, borrowed until the enqueued kernel has run.
 * Writes the packed words and scales readable through ef_worker_words / ef_worker_scales.
 * Workers may be stepped in any order, each exactly once per iteration.
 * Non-finite gradients are not checked; they propagate into the block's scale.
 * Errors: INVALID_ARG (i, null), ALIGNMENT, BAD_STATE (worker i already stepped in this
 * iteration), CUDA. */
int ef_worker_step(ef_ctx* ctx, int32_t i, const float* grad /* device */);

/* All M workers in one launch: the same computation as ef_worker_step(ctx, i, grads + i*stride)
 * for i = 0 .. M-1 (the workers are independent of each other, Algorithm 4), with one kernel
 * launch instead of M.  grads: device, 16-byte aligned; stride: elements between the gradients
 * of consecutive workers, >= d and a multiple of 4.  No worker may have been stepped yet in
 * this iteration.  Results are bit-identical to the per-worker calls.
 * Errors: INVALID_ARG, ALIGNMENT, BAD_STATE, CUDA. */
int ef_worker_step_all(ef_ctx* ctx, const float* grads /* device, M gradients */, int64_t stride);

/* Same as ef_worker_step with the gradient in HOST memory (pinned memory recommended): the
 * gradient is copied to a staging buffer on an internal copy stream, double-buffered so that
 * the copy of worker i+1 overlaps the kernel of worker i.  grad is borrowed until the copy
 * has completed (ordered before everything later enqueued on the context's stream).
 * Requires EF_FLAG_HOST_STAGING at ef_init, else EF_ERR_BAD_STATE. */
int ef_worker_step_host(ef_ctx* ctx, int32_t i, const float* grad /* host */);

/* Server side of one iteration (Algorithm 4, the "on server" lines) plus the parameter
 * update every worker performs after the pull (Algorithm 4, x_{t+1} = x_t - eta Deltatilde_t;
 * all replicas of x are identical, so it is done once):
 *   ptilde_t = (1/M) sum_i Delta_{t,i} + etilde_t;  Deltatilde_t = C_B(ptilde_t);
 *   etilde_{t+1} = ptilde_t - Deltatilde_t;  x_{t+1} = x_t - eta Deltatilde_t.
 * The average is evaluated as sum over ascending i of (+-)(scale_{i,b} / M) in fp32.
 * Errors: BAD_STATE unless every worker has been stepped exactly once since the last
 * server step; CUDA. */
int ef_server_step(ef_ctx* ctx);

/* Diagnostics of worker i's last step (needs EF_FLAG_DIAGNOSTICS): B x 4 doubles, row b =
 * { ||p_b||_1, ||p_b||_2^2, ||g_b||_1, ||g_b||_2^2 } accumulated inside the worker kernel at no
 * extra memory traffic (||p_b||_1 is the compressor's own fp64 sum; the other three combine four
 * elements in fp32 before the fp64 accumulation: relative error below 1e-6).  From them follow the quantities of Section 3.2 / Fig. 1:
 * phi(p) = min_b ||p_b||_1^2 / (d_b ||p_b||_2^2) (Prop. 1), the non-block compressor's
 * delta = ||p||_1^2 / (d ||p||_2^2), and the coefficient of variation of |g| inside block b,
 * sqrt(d_b ||g_b||_2^2 / ||g_b||_1^2 - 1).  Device pointer, valid until ef_destroy, ordered on
 * the context's stream; NULL without the flag or on a bad index. */
const double* ef_worker_diagnostics(ef_ctx* ctx, int32_t i);

/* Stepsize of the coming iteration (Algorithms 2-4 take a stepsize sequence {eta_t}).  In that
 * iteration both the workers' and the server's residual enter rescaled by eta_{t-1}/eta_t
 * (computed in fp32; p = fma(ratio, e, mu m + g)), where eta_{t-1} is the stepsize of the last
 * completed iteration (the value given to ef_init before any iteration has run).  Without this
 * call the stepsize stays constant and the ratio is exactly 1.  Only between iterations.
 * Errors: INVALID_ARG (eta <= 0 or not finite), BAD_STATE (in the middle of an iteration). */
int ef_set_eta(ef_ctx* ctx, float eta);

/* Weight decay lambda >= 0, kept out of the compressor as in Appendix A: every worker (here:
 * once) keeps a decay momentum mtilde_t = mu mtilde_{t-1} + lambda x_t and the update becomes
 * x_{t+1} = x_t - eta_t (Deltatilde_t + mu mtilde_t + lambda x_t).  Needs EF_FLAG_WEIGHT_DECAY at
 * ef_init (the momentum starts at 0).  lambda = 0 switches it off.  Only between iterations.
 * Errors: INVALID_ARG, BAD_STATE (flag missing, or in the middle of an iteration). */
int ef_set_weight_decay(ef_ctx* ctx, float lambda);
float* ef_decay_momentum(ef_ctx* ctx);    /* mtilde, d floats (NULL without the flag); may be edited between iterations */

/* Copies the server's message of the last ef_server_step (packed words, then scales) to host
 * memory, asynchronously on the context's stream.  words: ef_num_words words; scales: B floats.
 * Errors: INVALID_ARG (null), CUDA. */
int ef_read_update_host(ef_ctx* ctx, uint32_t* words /* host */, float* scales /* host */);

/* Zero-copy device views, valid until ef_destroy; contents are ordered on the context's stream.
 * i in [0, M); NULL on a bad index. */
const uint32_t* ef_worker_words(ef_ctx* ctx, int32_t i);   /* ef_num_words words */
const float*    ef_worker_scales(ef_ctx* ctx, int32_t i);  /* B floats */
const uint32_t* ef_server_words(ef_ctx* ctx);
const float*    ef_server_scales(ef_ctx* ctx);
float*          ef_params(ef_ctx* ctx);   /* x, d floats; the caller may write x_0 or edit x between iterations */
int64_t         ef_num_words(ef_ctx* ctx);/* W = sum_b ceil(d_b / 32) */

/* State access for tests and checkpoints.  All pointers are device pointers to d floats,
 * 16-byte aligned.  i in [0, M) names a worker; i = -1 names the server (residual only).
 * The residual is stored internally in a deferred form (the corrected vector p_t plus the
 * block scale); ef_get_residual writes the residual e_{t+1} = p_t - Delta_t itself.
 * ef_set_state overwrites momentum (ignored for the server, may be NULL there) and residual.
 * The two getters may be called at any time, also in the middle of an iteration: they are
 * ordered on the context's stream and return worker i's state after its last enqueued step
 * (m_{t,i} and e_{t+1,i} once worker i has been stepped in iteration t).  ef_set_state is only
 * allowed between iterations.
 * Errors: INVALID_ARG, ALIGNMENT, CUDA; ef_set_state also BAD_STATE (called in the middle of an
 * iteration). */
int ef_get_momentum(ef_ctx* ctx, int32_t i, float* dst);
int ef_get_residual(ef_ctx* ctx, int32_t i, float* dst);
int ef_set_state(ef_ctx* ctx, int32_t i, const float* momentum, const float* residual);
int ef_step_count(ef_ctx* ctx, int64_t* t /* out: completed iterations */);

/* Synchronises the context's stream and reads the device status word that kernels set when a
 * bounded device-side wait runs out (only the bulk-staged server kernel waits at all: on an
 * mbarrier that counts the bytes of its own copies, with an iteration limit).  Returns EF_OK,
 * EF_ERR_TIMEOUT (the results of the affected call are undefined; the word is cleared) or
 * EF_ERR_CUDA.  The step calls themselves never synchronise, so a caller who wants the check
 * calls this, e.g. once per iteration or at checkpoints. */
int ef_check_status(ef_ctx* ctx);
uint32_t* ef_status_word(ef_ctx* ctx);   /* the word itself (device, inside the workspace): 0 = no event;
                                            monitoring code may copy it instead of calling ef_check_status */

/* Checked build.  Compiled with -DEF_DEBUG, every kernel validates its work item (tile or chunk
 * descriptor: block id, length, element and word ranges) against the problem's sizes before it
 * touches memory; an item that reaches outside is skipped and EF_ERR_BOUNDS is reported by
 * ef_check_status.  Nothing traps or asserts, so the context and the device stay usable.  (A
 * memory checker for the device is not always available; this is the library's own net.)
 * ef_debug_build: 1 if this library is the checked build.  ef_debug_shift_tile: test hook of the
 * checked build only (EF_ERR_BAD_STATE otherwise): moves the start of one tile descriptor
 * (tile = -1: the last one) by `delta` elements, between iterations, so that a test can see the
 * check refuse it. */
int ef_debug_build(void);
int ef_debug_shift_tile(ef_ctx* ctx, int64_t tile, int64_t delta);

/* Tracing: every entry point that enqueues work runs inside an NVTX range named after itself
 * ("ef_worker_step", "ef_server_step", ...), so that a profiler can group or filter the kernels
 * by call; without an attached tool the ranges do nothing. */

/* Number of kernels this context has launched so far (for launch accounting). */
int64_t ef_launch_count(ef_ctx* ctx);

/* ---- The parameter-server protocol in pieces (Algorithm 2 / Algorithm 4: each worker pushes
 * Delta_{t,i} to the server and pulls Deltatilde_t; Section 4.2 sends "more parameter servers"
 * to relieve the server and notes that sending a block's sign vector and its scale as two
 * separate messages costs latency, and that they should be fused).  The server side of
 * ef_server_step split by block range, plus the message format for the exchange:
 *
 * Fused message of a block range [b0, b1): block after block, one 32-bit unit holding the
 * block's scale (a float) followed by the block's ceil(d_b/32) packed words; ef_message_units
 * gives its length in 32-bit units.  Because blocks are laid out in order, the message of a
 * sub-range is a contiguous slice of the message of a larger range: the slice for [c0, c1)
 * starts ef_message_units(ctx, b0, c0) units into the message of [b0, b1) (0 for c0 == b0).
 * A worker can therefore pack all its blocks once and send each server its slice; servers'
 * update slices, concatenated in block order (an all-gather), form the whole update.
 *
 * ef_pack_message: writes the fused message of blocks [b0, b1) of worker `who`'s last worker
 *   step (who = -1: of the server's last step on those blocks) to dst (device).
 * ef_server_step_range: the server lines of Algorithm 4 on blocks [b0, b1) only:
 *     ptilde = (1/M) sum_i Delta_i + etilde;  Deltatilde = C_B(ptilde);  etilde = ptilde - Deltatilde
 *   msgs == NULL: the workers' messages are the context's own (all M workers local);
 *   otherwise worker i's fused message for exactly the blocks [b0, b1) starts at
 *   msgs + i * msg_stride (device; 32-bit units; this GPU's memory: receive buffers), i < M.
 *   The result (words, scales of the range) is readable through ef_server_words/scales and
 *   ef_pack_message(ctx, -1, ...).  The parameters are NOT updated.
 * ef_apply_update: x <- x - eta Deltatilde on blocks [b0, b1) (with the weight-decay side path
 *   if enabled); update == NULL: from the context's own server step on those blocks, otherwise
 *   from a fused message for exactly the blocks [b0, b1) (device).
 * Call order inside an iteration: all local workers stepped; then any sequence of
 * ef_server_step_range on disjoint ranges and ef_apply_update on disjoint ranges; the iteration
 * is complete (step count, stepsize bookkeeping) once ef_apply_update has covered every block.
 * Covering [0, B) with msgs == NULL and update == NULL equals ef_server_step bit for bit.
 * Errors: INVALID_ARG (range, null dst, msg_stride shorter than the message), BAD_STATE (workers
 * not all stepped, a block served or applied twice in one iteration, update == NULL for a block
 * this context has not served, msgs == NULL without all M workers local), CUDA. */
int64_t ef_message_units(ef_ctx* ctx, int32_t b0, int32_t b1);      /* -1 on a bad range */
int ef_pack_message(ef_ctx* ctx, int32_t who, int32_t b0, int32_t b1, uint32_t* dst /* device */);
int ef_server_step_range(ef_ctx* ctx, int32_t b0, int32_t b1,
                         const uint32_t* msgs /* device or NULL */, int64_t msg_stride);
int ef_apply_update(ef_ctx* ctx, int32_t b0, int32_t b1, const uint32_t* update /* device or NULL */);

/* ---- The same protocol with the messages stored where their readers are (Section 4.2's remedy
 * for the server bottleneck is to spread the blocks over several servers; a worker's message
 * then has one destination per block).  Instead of packing a message and handing it to a
 * collective, the kernels store it directly: into this device's memory or, with peer access
 * enabled by the caller, into another device's receive buffer.  The library only stores through
 * the pointers it is given; making the stores visible to the reader (end of the stream's work
 * plus whatever barrier the caller uses between devices) is the caller's business.
 *
 * ef_worker_step_push: ef_worker_step, except that the packed words go to the destinations
 *   instead of the context's word buffer: block b's fused message, [scale | ceil(d_b/32) words]
 *   as above, is written at block_dst[b].  block_dst is a DEVICE array of B device pointers
 *   (4-byte aligned targets; the array is read by the enqueued kernels and must stay unchanged
 *   until they have run).  The scales are also kept in the context (ef_worker_scales);
 *   ef_worker_words(i) is NOT written, so until worker i's next plain step ef_pack_message(i)
 *   and the calls that read the workers' own words (ef_server_step, ef_server_step_range with
 *   msgs == NULL) answer BAD_STATE.  Not for contexts with cut blocks (BAD_STATE).
 * ef_push_message: ef_pack_message with n_dst destinations (1..64): the message of blocks
 *   [b0, b1) is written to each dst[q], a HOST array of n_dst device pointers (read during the
 *   call).  With the servers' update slices pushed into every worker's update buffer this is the
 *   pull of Algorithm 4 without a separate gather.
 * Errors: INVALID_ARG (null pointers, index, range, n_dst), ALIGNMENT (grad), BAD_STATE, CUDA. */
int ef_worker_step_push(ef_ctx* ctx, int32_t i, const float* grad /* device */,
                        uint32_t* const* block_dst /* device array of B device pointers */);
int ef_push_message(ef_ctx* ctx, int32_t who, int32_t b0, int32_t b1, int32_t n_dst,
                    uint32_t* const* dst /* host array of n_dst device pointers */);

/* ---- Blocks cut across devices.  The method is per element except for one number per block,
 * ||p_b||_1 (Section 3.2), so a layout may be cut inside a block (e.g. an embedding larger than a
 * device's share): each device holds a piece as a block of its own context and the only exchange
 * is the sum of the pieces' fp64 L1 sums, one number per cut block and call.
 * ef_set_block_divisors: full_len[b] (host, B entries) is the size d_b of the whole block that
 *   local block b belongs to; full_len[b] > the local length marks a piece.  Before the first
 *   iteration only; not together with EF_FLAG_DIAGNOSTICS.
 * After a worker step (and after ef_server_step_range) the scales of pieces are open:
 *   ef_block_sums writes, for who = worker index or -1 = server, the B per-block sums to dst
 *   (device, B doubles; 0 for blocks held whole); the caller adds them up over the devices (an
 *   all-reduce) and hands the totals to ef_complete_scales, which forms scale_b = total_b / d_b
 *   for the pieces.  Until then the packed words of the step are valid but the scales of the
 *   pieces are not, and calls that need them (the next worker step of that worker,
 *   ef_pack_message, ef_server_step_range on local messages, ef_apply_update from the own server
 *   step) return EF_ERR_BAD_STATE.  ef_server_step is not available on such a layout: use
 *   ef_server_step_range(0, B) -> ef_block_sums(-1) -> reduce -> ef_complete_scales(-1) ->
 *   ef_apply_update(0, B).
 * Errors: INVALID_ARG, BAD_STATE, CUDA. */
int ef_set_block_divisors(ef_ctx* ctx, const int64_t* full_len /* host, B */);
int ef_block_sums(ef_ctx* ctx, int32_t who, double* dst /* device, B */);
int ef_complete_scales(ef_ctx* ctx, int32_t who, const double* totals /* device, B */);

/* ---- signum / signSGD with majority vote: the paper's comparison method (Section 1: only the
 * 1-bit gradient sign travels between workers and server, in both directions; baselines of
 * Sections 4.1 and 4.2; Table 1: 2Md bits per iteration).  It runs on the same context and
 * state as the error-feedback path (momentum m_i, parameters x, the packed-word buffers, same
 * packed layout; no scales are produced), one iteration being
 *     for each worker i:  ef_vote_worker_step(ctx, i, g_{t,i})      (or ef_vote_worker_step_all)
 *     ef_vote_server_step(ctx)
 *   worker i:  m_{t,i} = mu m_{t-1,i} + g_{t,i};  message = sign(m_{t,i}), readable through
 *              ef_worker_words (mu = 0 gives signSGD);
 *   server:    vote = sign(sum_i sign(m_{t,i})) coordinate-wise, readable through
 *              ef_server_words;  x_{t+1} = x_t - eta vote.
 * Conventions where the paper is silent: sign(+-0) = +1; a tied vote (possible only for even M;
 * Section 4.2 notes an odd M never ties) is sent as +1, the message being one bit.
 * Arguments, ordering rules and errors are those of ef_worker_step / ef_worker_step_all /
 * ef_server_step; in addition the worker calls of one iteration must all belong to the same
 * method, and the server call must match them (else BAD_STATE).  The stepsize is the one set by
 * ef_init / ef_set_eta; weight decay does not apply to this method. */
int ef_vote_worker_step(ef_ctx* ctx, int32_t i, const float* grad /* device */);
int ef_vote_worker_step_all(ef_ctx* ctx, const float* grads /* device, M gradients */, int64_t stride);
/* As ef_worker_step_host: grad is a HOST buffer (pinned for an asynchronous copy), staged through
 * the context's two staging buffers (EF_FLAG_HOST_STAGING, else BAD_STATE).  The voted signs are
 * read back with ef_read_update_host (its scales output is not meaningful for this method). */
int ef_vote_worker_step_host(ef_ctx* ctx, int32_t i, const float* grad /* host */);
int ef_vote_server_step(ef_ctx* ctx);

/* ---- top-k: the second example of a delta-approximate compressor after Definition 1
 * (Section 2): it keeps the k coordinates of largest absolute value (delta = k/d).  Together
 * with its error-feedback residual this is the worker's compress line and residual line of
 * Algorithm 2 with C = top-k:  Delta = C(v),  e = v - Delta.
 *   v[n]          device, 16-byte aligned: the corrected vector to compress
 *   idx_out[k]    device: the kept coordinates in increasing order
 *   val_out[k]    device: their values, val_out[r] = v[idx_out[r]]
 *   resid_out[n]  device, 16-byte aligned, or NULL: v - C(v) (exactly 0 at the kept coordinates,
 *                 v elsewhere); may alias v
 * Among equal magnitudes the lower index is kept (the paper does not say), +0 and -0 have the
 * same magnitude, NaN is unspecified.  workspace: device, 256-byte aligned, at least
 * ef_topk_workspace_bytes(n) bytes (histograms, per-chunk counts and a list of candidate keys:
 * about n/2 bytes), owned by the caller and overwritten by every call; calls that share a
 * workspace must not overlap on the GPU.
 * Work is enqueued on cuda_stream without synchronisation; the library allocates nothing.
 * Errors: INVALID_ARG (n < 1, k outside [1, n], null), WORKSPACE, ALIGNMENT,
 * UNSUPPORTED_DEVICE, CUDA. */
int ef_topk_workspace_bytes(int64_t n, size_t* bytes /* out */);
int ef_topk_compress(const float* v, int64_t n, int64_t k, int64_t* idx_out, float* val_out,
                     float* resid_out, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Measurement aid (the paper has no counterpart): no-compute stream kernels with the access mix
 * of the step kernels, one 4096-element chunk per CTA and 128-bit accesses like them, so that a
 * measured rate can be set against the ceiling of a kernel of the same shape.
 *   EF_PROBE_3R2W  reads a, b, c and rewrites b, c in place (the worker step: g, m, e -> m, e)
 *   EF_PROBE_1R1W  reads and rewrites b in place (the server and update passes)
 *   EF_PROBE_COPY  c <- a
 * a, b, c: device, n floats each, 16-byte aligned, distinct buffers; n a positive multiple of
 * 4096.  b and c are overwritten.  Enqueued on cuda_stream, no synchronisation.
 * Errors: INVALID_ARG, ALIGNMENT, CUDA. */
#define EF_PROBE_3R2W 0
#define EF_PROBE_1R1W 1
#define EF_PROBE_COPY 2
int ef_stream_probe(int32_t mode, const float* a, float* b, float* c, int64_t n, void* cuda_stream);

/* (The paper has no counterpart for this entry point; it exists for deployment reasons.)
 * The worker step of one block for callers that must not allocate device memory where they
 * step the optimizer: code that runs while another framework owns the allocator or the stream
 * (callbacks, plugins with a fixed arena), and latency-critical loops that cannot afford the
 * device-wide synchronisation an allocation may imply.  Unlike the context API it takes no
 * workspace: its scratch (one fp64 partial sum per 4096 elements and an arrival counter, 33 KB)
 * is a fixed array inside the library image, which every GPU that loads the library keeps until
 * the process exits.  The call itself performs no cudaMalloc/cudaFree and uses no allocating
 * library routine.
 *
 * Computes, for ONE block of n elements and state kept by the caller (all device pointers):
 *   momentum[n]        in/out  m <- mu*m + grad
 *   residual[n]        in/out  deferred residual buffer: holds p of the previous call on entry
 *                              and p = mu*m + grad + e on exit, where e_j = p_prev_j - s_prev *
 *                              sign(p_prev_j); start from zeros
 *   residual_scale[1]  in/out  s_prev on entry, the new scale on exit; start from zero
 *   words[ceil(n/32)]  out     packed signs of p (layout as described at the top of this file)
 *   scale[1]           out     ||p||_1 / n
 * i.e. exactly what ef_worker_step computes for a layout with a single block, bit for bit.
 * grad, momentum and residual must be 16-byte aligned.  Work is enqueued on cuda_stream; no
 * host synchronisation.
 *
 * Limits and sharing: n <= EF_NOALLOC_MAX_ELEMS, else EF_ERR_TOO_LARGE and nothing is launched.
 * All calls on a device share the one scratch array: calls that may overlap on the GPU (different
 * streams, or several host threads) race on it and must be serialised by the caller; calls
 * queued on one stream are safe.  The array keeps the previous call's contents; the call clears
 * the one cell that has to start at zero itself.
 *
 * The first call on each device looks up the array's device address (a short, one-time set-up
 * under a lock); make that first call outside any stream capture.
 * Errors: INVALID_ARG, TOO_LARGE, ALIGNMENT, UNSUPPORTED_DEVICE, CUDA. */
#define EF_NOALLOC_MAX_ELEMS (1 << 24)
int ef_worker_step_noalloc(const float* grad, float* momentum, float* residual,
                           float* residual_scale, int64_t n, float mu,
                           uint32_t* words, float* scale, void* cuda_stream);

const char* ef_strerror(int status);
int ef_last_cuda_error(ef_ctx* ctx);      /* the cudaError_t of the last EF_ERR_CUDA, else 0 */

/* Frees the host object.  Does not touch the workspace.  NULL is allowed. */
int ef_destroy(ef_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif  /* EF_H_ */
