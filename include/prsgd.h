/*
 * prsgd.h -- C ABI of the PR-SGD hot path for NVIDIA B200 (sm_100a).
 *
 * Parallel Restarted SGD (Yu, Yang, Zhu, AAAI-19, Algorithm 1): N workers hold
 * N copies x_i of an m-dimensional model.  Every iteration each worker takes a
 * local SGD step x_i <- x_i - gamma * G_i on its own minibatch; every I
 * iterations the node average y = (1/N) sum_i x_i replaces every x_i.  Here all
 * N workers live on one GPU, stacked as the rows of one [N, m_pad] fp32 array,
 * and F_i is an MLP with ReLU hidden layers and softmax cross-entropy averaged
 * over the minibatch.
 *
 * General rules
 *  - Every function returns an int status: PRSGD_OK (0) or a negative error
 *    code.  Nothing throws, aborts or exits across this boundary.
 *  - "d_" arguments are DEVICE pointers, "h_" arguments are HOST pointers;
 *    where a pointer may be either, an explicit on_device flag says which.
 *  - The library allocates NO device memory.  The caller owns the parameter
 *    store, the bf16 shadow, the scratch area and the data pools, and must keep
 *    them alive until prsgd_destroy.  The library owns only the host-side
 *    context.
 *  - All device work is enqueued on the CUDA stream given to prsgd_create
 *    (a cudaStream_t passed as void*; NULL = the legacy default stream).  Calls
 *    that return data to the host synchronise that stream; all others are
 *    asynchronous.
 *  - Errors found on the host (bad argument, misalignment, wrong state) are
 *    returned by the call itself.  Errors found on the device (a bounded wait
 *    inside a kernel that ran out) are recorded in a status word in the scratch
 *    area and reported by the next prsgd_sync / prsgd_get_* call.
 *  - One context may be used by one host thread at a time.
 *  - Worker i is row i of the store, always.
 *
 * Layout of one row of the store (and of the bf16 shadow, in elements):
 *    W_1 | b_1 | W_2 | b_2 | ... | W_L | b_L
 *  W_l is row-major [d_l, d_{l-1}].  Every segment starts at a multiple of 32
 *  elements (128 bytes in the fp32 store); the gap words and the tail up to
 *  m_pad are zero and stay zero.  prsgd_layout reports the offsets.  The
 *  "canonical" order used by get/set calls is the same sequence without gaps
 *  (m floats).
 */
#ifndef PRSGD_H_
#define PRSGD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PRSGD_OK                  0
#define PRSGD_ERR_ARG            -1  /* NULL pointer, negative count, value out of range            */
#define PRSGD_ERR_ALIGN          -2  /* device pointer not 256-byte aligned, or a dimension the
                                        selected precision cannot tile (see prsgd_model_spec)       */
#define PRSGD_ERR_SIZE           -3  /* size beyond a stated maximum                                */
#define PRSGD_ERR_STATE          -4  /* call order: e.g. local_steps before bind_data               */
#define PRSGD_ERR_CUDA           -5  /* a CUDA runtime/driver call failed; see prsgd_last_error     */
#define PRSGD_ERR_DEVICE_TIMEOUT -6  /* a bounded wait inside a kernel expired (status word set)    */
#define PRSGD_ERR_NONFINITE      -7  /* the parameter store holds a NaN or an infinity (found by the
                                        finite check, see prsgd_check_finite)                       */

#define PRSGD_PRECISION_FP32 0       /* fp32 GEMM operands, fp32 accumulation (CUDA cores)          */
#define PRSGD_PRECISION_BF16 1       /* bf16 GEMM operands from the shadow, fp32 accumulation in
                                        TMEM (tcgen05), fp32 master weights updated in place        */

#define PRSGD_X_FP32 0
#define PRSGD_X_BF16 1

#define PRSGD_MAX_LAYERS 16

typedef struct prsgd_ctx prsgd_ctx;   /* opaque; created by prsgd_create, freed by prsgd_destroy */

/* The model F_i and the sampling of zeta_i^t.  The paper leaves F_i generic
 * (Introduction, problem statement); this is the F_i of the workloads. */
typedef struct {
  int32_t  n_layers;       /* L >= 1, at most PRSGD_MAX_LAYERS                                      */
  const int32_t* dims;     /* HOST array of L+1 entries d_0..d_L, copied by the callee              */
  int32_t  batch;          /* B, per-worker minibatch size, 1..256; BF16: 16, 32 or 64              */
  int32_t  precision;      /* PRSGD_PRECISION_*; BF16 needs d_0..d_{L-1} to be multiples of 64      */
  int64_t  pool_samples;   /* P, samples in each worker's pool, a positive multiple of B            */
  uint64_t draw_seed;      /* seed of the minibatch draw, see prsgd_draw_block                      */
} prsgd_model_spec;

/* Element offsets inside one row.  w_off[l], b_off[l] for layer l+1, l = 0..L-1. */
typedef struct {
  int64_t m;               /* parameters per worker, canonical (no gaps)                            */
  int64_t m_pad;           /* row length in elements, multiple of 32                                */
  int64_t w_off[PRSGD_MAX_LAYERS];
  int64_t b_off[PRSGD_MAX_LAYERS];
} prsgd_layout_t;

/* Row layout of the parameter store for this model (host only, no GPU needed). */
int prsgd_layout(const prsgd_model_spec* spec, prsgd_layout_t* out);

/* Bytes the caller must provide: params = N*m_pad*4; shadow = N*m_pad*2 for
 * BF16 precision, else 0; scratch = activations (the first layer's twice for BF16
 * precision), deltas, logits, losses, the draw table, two m_pad-float rows (staging,
 * canonical order), counters and the status words.  Host only. */
int prsgd_workspace_bytes(int32_t N, const prsgd_model_spec* spec,
                          size_t* params_bytes, size_t* shadow_bytes, size_t* scratch_bytes);

/* Algorithm 1, input line: N workers, learning rate gamma > 0, synchronisation
 * interval I >= 0 (I = 0: never average automatically; I = 1: parallel
 * mini-batch SGD).  d_params / d_shadow / d_scratch: caller-owned device
 * memory of at least the sizes above, 256-byte aligned (d_shadow may be NULL
 * for FP32).  The store and the scratch are zero-filled; the iteration counter
 * starts at t = 0.  Parameters must then be set with prsgd_set_params. */
int prsgd_create(int32_t N, const prsgd_model_spec* spec, float gamma, int32_t I,
                 void* d_params, void* d_shadow, void* d_scratch,
                 void* cuda_stream, prsgd_ctx** out);

/* Free the host context.  Device memory stays with the caller. */
int prsgd_destroy(prsgd_ctx* ctx);

/* Per-worker data pools D_i (Introduction: each worker samples zeta_i from its
 * own distribution).  d_X: [N][P][d_0] row-major, x_dtype PRSGD_X_FP32 for
 * FP32 precision and PRSGD_X_BF16 for BF16 precision; d_Y: [N][P] int32 class
 * labels in [0, d_L).  Device pointers, 256-byte aligned, kept by reference. */
int prsgd_bind_data(prsgd_ctx* ctx, const void* d_X, int32_t x_dtype, const int32_t* d_Y);

/* Copy fresh pool contents from HOST memory (same shapes and dtype as bound)
 * into the bound device pools, asynchronously on the context's stream.  Pinned
 * host memory makes the copy overlap-capable; pageable memory also works. */
int prsgd_upload_data(prsgd_ctx* ctx, const void* h_X, const int32_t* h_Y);

/* Double-buffered variant of prsgd_upload_data, for callers that stream fresh samples every epoch:
 * prsgd_stage_data copies the NEXT pool contents from host memory into a pair of SPARE device pools
 * (same shapes as the bound ones, caller-owned, 256-byte aligned) on `copy_stream`, a stream of the
 * caller's other than the context's, so that the copy overlaps the local steps in flight;
 * prsgd_swap_data makes the staged pools the bound ones for all work enqueued afterwards (the
 * context's stream waits for the staged copy), and the previously bound pools become free to be
 * staged into next (the copy stream waits until the work that read them is done).  Asynchronous;
 * pinned host memory is needed for the overlap. */
int prsgd_stage_data(prsgd_ctx* ctx, const void* h_X, const int32_t* h_Y, void* d_X_spare, int32_t* d_Y_spare,
                     void* copy_stream);
int prsgd_swap_data(prsgd_ctx* ctx);

/* x_i^0 (Algorithm 1, input line: every worker starts from the same point).
 * src holds m floats in canonical order.  worker >= 0: only that row is
 * written; worker = -1: every row receives the same m floats.  Refreshes the
 * bf16 shadow.  src_on_device says where src lives. */
int prsgd_set_params(prsgd_ctx* ctx, const float* src, int32_t worker, int src_on_device);

/* Whole stacked state [N][m] (canonical order per row), e.g. to resume a run. */
int prsgd_set_params_stacked(prsgd_ctx* ctx, const float* src, int src_on_device);
int prsgd_get_params_stacked(prsgd_ctx* ctx, float* dst, int dst_on_device);

/* One worker's x_i, m floats, canonical order.  Synchronises the stream. */
int prsgd_get_params(prsgd_ctx* ctx, float* dst, int32_t worker, int dst_on_device);

/* Iterations t+1 .. t+k of Algorithm 1.  Each iteration: every active worker i
 * draws its minibatch block prsgd_draw_block(seed, i, t, P/B), evaluates
 * G_i^t = grad F_i(x_i^{t-1}; block) and updates x_i^t = x_i^{t-1} - gamma G_i^t
 * in place (Eq. parallel-sgd-x-update); when I > 0 and t mod I == 0 the node
 * average is formed from the updated models and written to every row, so each
 * epoch of I iterations starts from a common point (the paragraph after
 * Algorithm 1; Algorithms 2 and 3 are stated in this form).
 * local_steps(a) followed by local_steps(b) equals local_steps(a + b).
 * k >= 0.  Asynchronous. */
int prsgd_local_steps(prsgd_ctx* ctx, int64_t k);

/* Average and restart now, whatever t is: y = (1/N) sum_i x_i summed in worker
 * order i = 0..N-1 in fp32, then every row (and the shadow) is overwritten
 * with y.  After this call all N rows hold identical bits.  Asynchronous. */
int prsgd_average(prsgd_ctx* ctx);

/* xbar^t = (1/N) sum_i x_i^t (Eq. node-average-x), m floats in canonical
 * order, WITHOUT modifying the store.  When the library knows that all rows hold
 * the same bits (right after an average, see PRSGD_OPT_SHARED_RESTART) that row
 * is returned as it stands instead of summing N copies of it.  Synchronises the
 * stream when dst is on the host. */
int prsgd_get_average(prsgd_ctx* ctx, float* dst, int dst_on_device);

/* The same read-out without stopping the training stream: the mean (Eq. node-average-x) is formed into
 * the context's staging row on the context's stream, and its copy to h_dst (m floats, HOST memory,
 * page-locked for the copy to be asynchronous) runs on copy_stream, which must be a different stream.
 * The call returns at once; h_dst is valid once copy_stream has been synchronised by the caller.
 * Later prsgd_local_steps calls may run while the copy is in flight (they do not touch the staging
 * row); the next read-out waits for it.  Device errors surface at the next prsgd_sync. */
int prsgd_get_average_async(prsgd_ctx* ctx, float* h_dst, void* copy_stream);

/* Mean minibatch loss F_i(x_i^{t-1}; zeta_i^t) of every worker at the last
 * iteration run; h_dst holds N floats (HOST).  Synchronises the stream. */
int prsgd_get_losses(prsgd_ctx* ctx, float* h_dst);

/* Block index every worker drew at the last iteration run (N int32, HOST). */
int prsgd_get_draws(prsgd_ctx* ctx, int32_t* h_dst);

/* Schedule controls.  set_lr: gamma^s of Algorithm 2.  set_interval: I.
 * set_active: Algorithm 3 -- h_mask holds N bytes, worker i takes local steps
 * only while h_mask[i] != 0 (an inactive worker keeps its point, the
 * zero-gradient convention of the Extensions section); NULL = all active.
 * get_step / set_step read and write the iteration counter t (resume). */
int prsgd_set_lr(prsgd_ctx* ctx, float gamma);
int prsgd_set_interval(prsgd_ctx* ctx, int32_t I);
int prsgd_set_active(prsgd_ctx* ctx, const uint8_t* h_mask);
int prsgd_get_step(prsgd_ctx* ctx, int64_t* t);
int prsgd_set_step(prsgd_ctx* ctx, int64_t t);

/* Algorithm 2 (PR-SGD with time-varying learning rates) as one call: for s = s_begin..s_end the epoch
 * starts from the node average, then K^s = ceil(s^(1/3) / N) local steps with rate
 * gamma^s = N / s^(2/3) (Theorem 2) times gamma_scale (1 gives the theorem's constants, which are
 * far too large for a neural network with unknown L; the scale keeps the shape of the schedule).
 * The context's own gamma and I are left as they were.  prsgd_alg2_schedule returns K^s and gamma^s
 * (host only).  The iteration counter advances by sum_s K^s, as in the re-indexing after Algorithm 2. */
int prsgd_alg2_schedule(int32_t N, int64_t s, int64_t* K_s, float* gamma_s);
int prsgd_run_time_varying(prsgd_ctx* ctx, int64_t s_begin, int64_t s_end, float gamma_scale);

/* One epoch of Algorithm 3 (heterogeneous workers): all workers start from the node average, worker
 * i takes h_I_i[i] local steps (HOST array of N entries >= 0), workers that have finished keep their
 * point (the zero-gradient convention of the Extensions section).  The iteration counter advances
 * by max_i I_i; the models are left un-averaged, the next epoch (or prsgd_average) averages them. */
int prsgd_run_heterogeneous_epoch(prsgd_ctx* ctx, const int32_t* h_I_i);

/* Workers spread over several GPUs (one context per GPU, each holding a shard of the N workers).
 * Inside an epoch workers need no synchronisation; the only exchange is the node average, which the
 * paper suggests to obtain by an all-reduce of the local models (Section 2, "Communication
 * Reduction").  The library provides the two local halves; the all-reduce of the m_pad-float row
 * between them belongs to the caller (NCCL).
 *  - prsgd_set_worker_offset: global index of this context's row 0; the minibatch draw of local
 *    row i is that of worker first_worker + i.
 *  - prsgd_set_global_workers: the N of the whole job (all contexts together, >= first_worker + the
 *    context's own N; 0 = this context is the whole job).  Theorem 2's K^s and gamma^s are functions
 *    of that N, so prsgd_run_time_varying takes its schedule from it; on a context that holds only a
 *    shard that call returns PRSGD_ERR_STATE, because the epoch's starting average needs every GPU:
 *    the caller drives the epochs with prsgd_alg2_schedule(N_global, s), prsgd_set_lr,
 *    prsgd_local_steps and its all-reduce.
 *  - prsgd_partial_sum: d_dst[j] = sum over the local rows of P[i][j], fp32 in row order, for the
 *    padded columns j in [col0, col0 + ncols); d_dst is a device row of m_pad floats.
 *  - prsgd_assign_rows: every local row (and the bf16 shadow) gets d_src[j] / divisor on the same
 *    column range; with divisor = the global N this is the restart at the node average.
 *  - prsgd_local_steps_sum: iterations t+1 .. t+k like prsgd_local_steps (needs I = 0), except that the
 *    k-th one runs in the fused update + average form with the division left out: afterwards EVERY local
 *    row holds sum_i x_i^{t+k} over the local rows (what prsgd_partial_sum would have computed from the
 *    updated rows, without that extra pass over the store).  Row 0 of the store (m_pad floats at d_params) is
 *    then the buffer to all-reduce, and prsgd_assign_rows(d_params, N_global, ...) completes the average; until
 *    it has covered the whole row the store holds sums, not models.  Same bits as prsgd_local_steps(k) +
 *    prsgd_partial_sum + prsgd_assign_rows.  Not with averaged momentum buffers.
 * col0 and ncols are multiples of 4 (column ranges let the caller pipeline the all-reduce chunk by
 * chunk); rows are 16-byte aligned device pointers.  With a single context,
 * partial_sum + assign_rows(divisor = N) leaves the same bits as prsgd_average.  Asynchronous. */
int prsgd_set_worker_offset(prsgd_ctx* ctx, int32_t first_worker);
int prsgd_set_global_workers(prsgd_ctx* ctx, int32_t N_global);
int prsgd_partial_sum(prsgd_ctx* ctx, float* d_dst, int64_t col0, int64_t ncols);
int prsgd_local_steps_sum(prsgd_ctx* ctx, int64_t k);
int prsgd_assign_rows(prsgd_ctx* ctx, const float* d_src, float divisor, int64_t col0, int64_t ncols);

/* Local step with momentum, as in the paper's experiment (Experiment section, figure captions:
 * momentum 0.9): per worker v_i <- mu v_i + G_i, x_i <- x_i - gamma v_i, v_i starting at 0.
 * d_velocity: caller-owned device memory of the same size as the parameter store (N*m_pad*4
 * bytes, 256-byte aligned), zeroed by this call and laid out like the store.  The paper does not
 * say what happens to the momentum buffers at a restart: with average_velocity = 0 every worker
 * keeps its own, with 1 they are averaged together with the models.  On the tensor-core path an
 * averaging iteration takes the fused update + average with momentum too (every worker's new buffer
 * tile goes back to its own row, or the averaged tile to every row); on the FP32 path it runs as
 * update followed by the averaging kernel.  d_velocity = NULL switches back to plain SGD.  mu in [0, 1). */
int prsgd_enable_momentum(prsgd_ctx* ctx, float mu, void* d_velocity, int average_velocity);
/* The momentum buffers, [N][m] in canonical order.  Synchronises the stream. */
int prsgd_get_velocity_stacked(prsgd_ctx* ctx, float* dst, int dst_on_device);

/* Options.  PRSGD_OPT_FUSED_AVERAGE (default 1): on an averaging iteration the
 * update and the average run as one pass over the store instead of an update
 * pass followed by prsgd_average's pass; both produce identical bits. */
#define PRSGD_OPT_FUSED_AVERAGE 1
/* PRSGD_OPT_PROFILE (default 0): when 1, every kernel launch is bracketed by a
 * pair of CUDA events on the context's stream; read the sums with
 * prsgd_get_profile.  Costs two event records per launch. */
#define PRSGD_OPT_PROFILE 2
/* PRSGD_OPT_GRAPH (default 1): whole averaging periods (I iterations that begin right after an
 * average, k >= I, I > 0, profiling off) are captured once as a CUDA graph and replayed; the kernels
 * read the iteration number from a device counter, so one capture serves every period.  Settings
 * that change the launches (gamma, I, options, mask on/off, momentum, the bound pools) key separate
 * captures.  Results are bit-identical to direct launches; 0 switches the replay off. */
#define PRSGD_OPT_GRAPH 4
/* PRSGD_OPT_UPDATE_TILE (default 0): column width of the 128-row tile the tensor-core update
 * kernel works on: 64 (four pipeline stages per SM), 128 (two), or 0 = chosen per launch from
 * the layer size.  A tuning knob only: every setting produces the same bits. */
#define PRSGD_OPT_UPDATE_TILE 3
/* PRSGD_OPT_FUSED_EPILOGUES (default 1, tensor-core path): the softmax cross-entropy gradient runs
 * in the epilogue of the last forward GEMM and each bias step in the epilogue that forms that layer's
 * dZ, when the class count d_L is at most 128.  With 0 (or d_L > 128) they run as kernels of their
 * own.  The two forms agree to fp32 rounding (the stand-alone bias kernel sums the bf16-rounded dZ). */
#define PRSGD_OPT_FUSED_EPILOGUES 5
/* PRSGD_OPT_EARLY_LOADS (default 1, tensor-core path): a kernel requests the weight tiles of its first
 * pipeline stages before it waits for the previous launch to complete, when that launch cannot be
 * writing them (every layer's forward GEMM but the first, every dX GEMM, the master tiles of every
 * update; never while a worker mask is set).  Same bits either way. */
#define PRSGD_OPT_EARLY_LOADS 6
/* PRSGD_OPT_NEXT_FORWARD (default 1, tensor-core path, more than one layer): on a plain SGD iteration
 * that is not an averaging one and is followed by another iteration of the same prsgd_local_steps call,
 * the update of layer 1 also multiplies each freshly stepped tile of W_1 with the next minibatch, so that
 * the next iteration starts with a_1 in place: its first forward launch is skipped and the bf16 copy of
 * W_1, which only that launch reads, is not written on such iterations (it is valid whenever a call
 * returns).  Same bits as the separate launches. */
#define PRSGD_OPT_NEXT_FORWARD 7
/* PRSGD_OPT_DX_IN_UPDATE (default 1, tensor-core path): on a plain SGD iteration the update launch of a
 * layer l >= 2 also forms dZ_{l-1} from the bf16 values its weights had before the step, which it
 * derives from the fp32 tiles it holds, so the separate dX launch and its second read of the layer's
 * bf16 weights are saved.  1 = for layers with at least three 64-wide column blocks per SM over all
 * workers (fewer do not balance) and for single-row-tile layers, 2 = for every layer, 0 = never.  Not
 * for a layer that takes the fused update + average on an averaging iteration.  Same bits as the
 * separate launches (also with momentum and with a worker mask). */
#define PRSGD_OPT_DX_IN_UPDATE 8
/* PRSGD_OPT_SHARED_RESTART (default 1, tensor-core path): right after a node average every worker holds the
 * same point (the restart of Algorithm 1), so the iteration that follows reads worker 0's weights for every
 * worker wherever a launch only reads them (forward, dX) or reads all N copies of a tile before it writes any
 * (the fused update + average): one HBM read serves all N workers.  The library keeps track of whether the
 * rows are equal (after prsgd_average, an averaging iteration, prsgd_set_params for all workers, or
 * prsgd_assign_rows calls that cover the row in ascending order); a caller that writes into the store
 * through its own pointer instead of these calls must switch the option off.  Same bits either way. */
#define PRSGD_OPT_SHARED_RESTART 10
/* PRSGD_OPT_FORWARD_CHAIN (default 1, tensor-core path, 2 to 8 layers left to run): the forward GEMMs of an
 * iteration run as ONE launch whose CTAs walk the items of all layers without draining in between; an item
 * of layer l waits (bounded, status word on expiry) only for a_{l-1} of its own worker, counted per
 * (layer, worker) in the scratch area, since workers do not depend on one another inside an iteration.
 * With 0 every layer is a launch of its own.  Same bits either way. */
#define PRSGD_OPT_FORWARD_CHAIN 11
/* PRSGD_OPT_WORKER_GROUPS (default 1 = off; 2..4, tensor-core path): inside an epoch the workers need no
 * synchronisation (the text after Algorithm 1), so the plain iterations between two averages are enqueued as
 * G independent chains of launches, one per contiguous group of N/G workers, on G streams the library creates
 * for itself; they fork from the context's stream and join it again before the averaging iteration.  While
 * one group's long update kernels run, another group's short launches find free SMs.  Not while a worker
 * mask or profiling is on.  Same bits as one chain for all workers. */
#define PRSGD_OPT_WORKER_GROUPS 12
/* PRSGD_OPT_DX_SHARED_PAIR (default 1, tensor-core path): stage layout of the 64-wide update + dX launch.  1: the
 * two bf16 tiles (old and stepped weights) exist once, behind the stages, and a stage holds only the fp32 tile
 * and the operand boxes, which makes room for a deeper pipeline; 0: every stage has its own pair.  A tuning knob:
 * same bits either way. */
#define PRSGD_OPT_DX_SHARED_PAIR 13
/* PRSGD_OPT_HEAD_KERNEL (default 1, tensor-core path, at least two layers, at most 128 classes, width of the last
 * hidden layer 128, 256, 512 or 1024, plain SGD step, PRSGD_OPT_DX_IN_UPDATE and PRSGD_OPT_FUSED_EPILOGUES at
 * their defaults): everything an iteration does with the class layer -- logits, softmax cross-entropy gradient
 * and loss, the step of W_L and b_L (Eq. parallel-sgd-x-update), dZ of the layer below and the step of its
 * bias -- is one launch in which a thread-block cluster per worker splits the last hidden layer's features among
 * its CTAs (128 each) and sums the logit shares in a fixed order.  1: when all those CTAs fit on the GPU at once
 * (workers x width / 128 <= SM count); 2: always; 0: never, the last forward GEMM and the class layer's update are
 * launches of their own.  The two forms agree to fp32 rounding of the logits (different summation order, fast
 * exponential), not bit for bit; each is deterministic. */
#define PRSGD_OPT_HEAD_KERNEL 14
/* PRSGD_OPT_TILED_WEIGHTS (default 1, tensor-core path): inside a row of the store, of the bf16 copy and of the
 * momentum buffers the weight segment of a hidden layer whose height d_l is a multiple of 128 is kept as 128 x 64
 * tiles, one after another (tile (r / 128, c / 64) at index (r / 128) (d_{l-1} / 64) + c / 64, row-major inside
 * a tile), so that every tile a kernel loads or stores is one contiguous piece of memory; the class layer, layers of
 * other heights and the fp32 path keep row-major segments.  Nothing changes at this interface: every call that
 * takes or returns parameters (prsgd_set_params*, prsgd_get_params*, prsgd_get_average*, prsgd_get_velocity_stacked)
 * speaks the canonical order, offsets and m_pad are the same, and prsgd_partial_sum / prsgd_assign_rows work on
 * columns of the rows as they are (all ranks of a job use the same setting).  Changing the option re-orders the
 * store in place (a pass over all rows).  Same bits either way. */
#define PRSGD_OPT_TILED_WEIGHTS 19
/* PRSGD_OPT_OVERLAP_UPDATE (default 1, tensor-core path, three layers or more, every worker active):
 * on iterations whose layer-1 update also forms the next iteration's first activation (PRSGD_OPT_NEXT_FORWARD) and
 * whose layer 2 runs dX and update as separate launches, layer 2's update is enqueued AFTER layer 1's and starts
 * beside it: it needs nothing that launch produces, so its CTAs take the SMs that launch leaves idle (whole row
 * blocks per CTA seldom fill the GPU) and the others as they fall free, claiming tiles from a device counter.  The
 * next iteration's a_1 goes to a second buffer meanwhile.  Same arithmetic per tile: same bits. */
#define PRSGD_OPT_OVERLAP_UPDATE 20
/* PRSGD_OPT_MERGED_SMALL_AVERAGE (default 1, tensor-core path, fused averaging iterations): the weight segments of
 * layers too small for the fused update + average (the class layer) are averaged by the launch that averages the
 * bias segments, at the end of the iteration, instead of by a launch of their own after the layer's update.  Same
 * arithmetic (fp32 sum in worker order, one division): same bits. */
#define PRSGD_OPT_MERGED_SMALL_AVERAGE 18
/* PRSGD_OPT_HEAD_FORWARD (default 0; needs the cluster launch of PRSGD_OPT_HEAD_KERNEL, at least three layers and
 * shared memory for two pipeline stages behind the class layer's tiles): when 1, the CTAs of a worker's cluster
 * first form the 128 features of the last hidden activation they need, a_{L-1} = relu(W_{L-1} a_{L-2} + b_{L-1}),
 * each streaming its row tile of W_{L-1}, and keep them in shared memory: one launch fewer per iteration, and
 * a_{L-1} is never written to global memory.  Same bits as the separate forward launch (same products in the same
 * order).  Off by default: measured slower (the two launches overlap the second one's start-up with the first
 * one's streaming, which one launch cannot). */
#define PRSGD_OPT_HEAD_FORWARD 17
/* PRSGD_OPT_COMMON_POINT (default 1, tensor-core path, plain SGD step, fused average, PRSGD_OPT_SHARED_RESTART on):
 * an averaging iteration that STARTS from N equal rows (every iteration when I = 1, which the paper notes is
 * parallel mini-batch SGD; otherwise the first step after prsgd_average when I divides its number) forms the
 * new average as x - (gamma / N) sum_i G_i: one weight-gradient GEMM per tile over the minibatches of all
 * workers, one step, N row stores (Eq. parallel-sgd-x-update summed over i, then Algorithm 1's average).  All
 * such layers share one launch after the iteration's dX launches, and the tiles of its last, partly filled round
 * are each formed by several CTAs that store a share of the rows (2: whole tiles only).
 * Equal to update-then-average up to fp32 rounding, not bit for bit; deterministic.  0: the N stepped models are
 * formed and summed one by one. */
#define PRSGD_OPT_COMMON_POINT 15
/* PRSGD_OPT_SPLIT_BLOCKS (default 0, tensor-core path, no worker mask): the update launch of layer 1 that also forms
 * the next a_1 walks row blocks of 128 output features, whole blocks per CTA.  1: their column tiles are dealt out
 * in equal runs, one per SM, whenever whole blocks would leave SMs idle or in a short last round (128 blocks on
 * 148 SMs, 512 blocks = 3.46 rounds) and the launch is large; a row block cut by a run boundary gets its forward
 * sum from the partial sums of its two or three CTAs, added in run order by whichever finishes last (no CTA waits
 * for another).  2: also for small launches.  The weights are bit-identical either way; a_1 of a cut row block is
 * summed in another order (fp32 rounding) and is deterministic.  Off by default: the launch is bound by the
 * memory system, not by its longest CTA, and equal runs gained nothing measurable. */
#define PRSGD_OPT_SPLIT_BLOCKS 16
/* PRSGD_OPT_CHECK_FINITE (default 0): when 1, prsgd_sync also runs prsgd_check_finite. */
#define PRSGD_OPT_CHECK_FINITE 9
int prsgd_set_option(prsgd_ctx* ctx, int32_t option, int64_t value);

/* Kernel families of the hot path, for prsgd_get_profile. */
#define PRSGD_KERNEL_FORWARD        0  /* grouped forward GEMM + bias + ReLU                        */
#define PRSGD_KERNEL_SOFTMAX        1  /* softmax cross-entropy gradient                            */
#define PRSGD_KERNEL_DX             2  /* grouped input-gradient GEMM + ReLU mask                   */
#define PRSGD_KERNEL_UPDATE         3  /* grouped weight-gradient GEMM + in-place SGD update        */
#define PRSGD_KERNEL_UPDATE_AVERAGE 4  /* the same with the node average fused in                   */
#define PRSGD_KERNEL_AVERAGE        5  /* stand-alone node average (+ broadcast)                    */
#define PRSGD_KERNEL_MISC           6  /* broadcast of x^0, shadow refresh                          */
#define PRSGD_KERNEL_HEAD           7  /* class layer: logits, softmax-CE gradient, step, dZ below  */
#define PRSGD_KERNEL_FAMILIES       8

/* Device time (milliseconds, from the event pairs) and launch count of one
 * kernel family since the previous call for that family; both counters are
 * then reset.  Synchronises the stream.  Zero unless PRSGD_OPT_PROFILE is on. */
int prsgd_get_profile(prsgd_ctx* ctx, int32_t family, double* ms_total, int64_t* launches);

/* Number of kernels this context has launched so far. */
int prsgd_get_launch_count(prsgd_ctx* ctx, int64_t* count);

/* Wait for the stream, then report any device-side error recorded so far. */
int prsgd_sync(prsgd_ctx* ctx);

/* Finite check of the whole parameter store (and of the momentum buffers when momentum is on): one
 * pass that reads every word and counts those whose exponent field is all ones (NaN, +-infinity).
 * Algorithm 1's averaging step spreads a single worker's NaN to all N workers, so a caller that
 * wants to stop a diverged run checks before it averages or checkpoints.  Returns PRSGD_OK when
 * every value is finite, PRSGD_ERR_NONFINITE otherwise; *count (may be NULL) receives the number of
 * non-finite words, *first_worker (may be NULL) the lowest row that holds one (-1 if none).  Nothing
 * traps and the store is not modified.  Synchronises the stream. */
int prsgd_check_finite(prsgd_ctx* ctx, int64_t* count, int32_t* first_worker);

/* Failure path, exercised without faulting the GPU.  Every wait inside the tensor-core kernels is
 * bounded; when one expires the kernel records a code in the scratch status words and returns, later
 * local-step and averaging launches of the context (both precisions) become no-ops (a kernel reads the
 * word while it sets up, so the one launch whose set-up overlapped the failing kernel may still run;
 * the parameters are to be set again after a timeout in any case: prsgd_set_params* keep working),
 * and prsgd_sync / prsgd_get_* return PRSGD_ERR_DEVICE_TIMEOUT.  prsgd_selftest_wait_expiry launches a one-warp kernel that waits about
 * limit_us microseconds (1..1000000) on a barrier nothing ever signals, so that exactly this happens;
 * prsgd_clear_device_error zeroes the status words and makes the context usable again (the
 * parameters are as the last successful launch left them). */
int prsgd_selftest_wait_expiry(prsgd_ctx* ctx, int32_t limit_us);
int prsgd_clear_device_error(prsgd_ctx* ctx);

/* Text of the last error of this context (or of the last context-free call
 * when ctx is NULL).  Library-owned, valid until the next call. */
const char* prsgd_last_error(prsgd_ctx* ctx);

/* The averaging step of Algorithm 1 on a bare array: for every column j,
 * y_j = (1/N) sum_{i=0..N-1} P[i*row_stride + j] (fp32, summed in row order),
 * then P[i*row_stride + j] = y_j for every i.  d_P is a device pointer,
 * 16-byte aligned; row_stride >= m in elements and a multiple of 4; N >= 1,
 * m >= 0.  Asynchronous on cuda_stream.  Uses no scratch memory. */
int prsgd_average_rows(float* d_P, int64_t N, int64_t m, int64_t row_stride, void* cuda_stream);

/* Node average of a bare [N, row_stride] array WITHOUT any allocation and
 * without touching the array: y_j = (1/N) sum_i P[i*row_stride + j], j < m,
 * summed in row order in fp32 exactly as prsgd_get_average does, delivered to
 * dst (m floats; dst_on_device says whether dst is device or host memory).
 * The paper has no counterpart to this call; it exists for callers that must
 * not allocate: a monitoring or logging thread that wants xbar^t while the
 * training stream is busy cannot afford cudaMalloc (it synchronises the whole
 * device and stalls the step in flight), and a process running under a fixed
 * device-memory budget has nothing left to allocate from.  Such callers often
 * hold only pageable host memory, which a kernel cannot write, so the mean is
 * staged in device memory: here that staging row is a fixed array inside the
 * library (PRSGD_NOALLOC_MAX_M floats = 4 MiB, held by every GPU that loads the
 * library until the process exits) instead of caller-provided scratch.
 *  - m must be in 0..PRSGD_NOALLOC_MAX_M, otherwise PRSGD_ERR_SIZE; d_P 16-byte
 *    aligned, row_stride >= m and a multiple of 4, N >= 1.
 *  - The first call on each device looks up the array's device address (that
 *    device must be current, as for every call); make that first call outside
 *    any stream capture.  No call allocates or frees anything.
 *  - All calls on one device share the staging row.  A call overwrites the
 *    first m entries before reading them back and relies on no earlier
 *    content, but two calls whose GPU work can overlap (different streams, or
 *    different host threads) race on it: serialise them.
 *  - Work is enqueued on cuda_stream; with dst on the host the stream is
 *    synchronised before returning, with dst on the device the call is
 *    asynchronous. */
#define PRSGD_NOALLOC_MAX_M (1 << 20)
int prsgd_mean_rows_noalloc(const float* d_P, int64_t N, int64_t m, int64_t row_stride,
                            float* dst, int dst_on_device, void* cuda_stream);

/* The minibatch draw zeta_i^t as an integer: the (i+1)-th output of a
 * SplitMix64 stream keyed by the t-th output of the SplitMix64 stream seeded
 * with `seed`, modulo n_blocks.  Pure host function; the device code evaluates
 * the same function.  Returns a value in [0, n_blocks); n_blocks must be > 0. */
uint64_t prsgd_draw_block(uint64_t seed, int32_t worker, int64_t t, uint64_t n_blocks);

#ifdef __cplusplus
}
#endif
#endif /* PRSGD_H_ */
