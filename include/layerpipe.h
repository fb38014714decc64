/*
 * layerpipe.h -- C ABI of the LayerPipe training hot path for NVIDIA B200 (sm_100a).
 *
 * The library trains a chain of layers with the paper's delayed-gradient scheme:
 * per layer the forward contraction (Eqs. 1-2), then a backward pass split into two
 * independent tasks, the activation gradient ("delta", Eqs. 3-4) and the weight
 * gradient ("G", Eq. 5), and the delayed update W(n) = W(n-1) - eta G(n-M) (Eq. 6)
 * with the weight / activation stashes that retiming leaves on the W->delta and
 * a->backward edges (Section III-A).  The paper's processors are stages mapped onto
 * streams of ONE GPU; there is no multi-GPU path.
 *
 * Conventions
 *   - every function returns LP_OK (0) or a negative LP_ERR_* code; nothing throws,
 *     aborts or prints.  lp_last_error() gives a human-readable reason.
 *   - "host" / "device" in a parameter comment says where the pointer must live.
 *   - the caller owns every buffer it passes.  The library allocates no device memory:
 *     all of its state lives inside the caller's workspace (lp_workspace_size bytes,
 *     256-byte aligned, must outlive the handle).  Initial weights are copied.
 *   - layouts at the boundary: FC weights W[out][in] row-major fp32 (the paper's
 *     out x in matrix of Eq. 1); minibatch [batch][in] row-major.
 *   - lp_step is asynchronous and never synchronises the device.
 *   - a handle is not thread-safe; use one host thread per handle.
 */
#ifndef LAYERPIPE_H_
#define LAYERPIPE_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct lp_ctx* lp_handle;

enum {
  LP_OK = 0,
  LP_ERR_INVALID_ARG = -1,  /* null pointer, bad index, bad shape; no side effects      */
  LP_ERR_UNSUPPORTED = -2,  /* not an sm_100 device, or a layer kind not built yet       */
  LP_ERR_WORKSPACE = -3,    /* workspace too small or misaligned                         */
  LP_ERR_CUDA = -4,         /* a CUDA call failed; the handle is latched into this state */
  LP_ERR_TIMEOUT = -5,      /* a bounded device-side wait gave up (see lp_device_status) */
  LP_ERR_NOT_READY = -6     /* the requested step's data is not (or no longer) held      */
};

enum { LP_FC = 0, LP_CONV = 1 };
enum { LP_ACT_NONE = 0, LP_ACT_RELU = 1, LP_ACT_GELU = 2 }; /* GELU = exact erf form */
enum { LP_SCHED_LAYERPIPE = 0, /* delta and G of a layer are separate concurrent tasks;   */
                               /* delta^{l-1} is released as soon as delta finishes        */
       LP_SCHED_FUSED_B = 1 }; /* PipeDream-style: delta, G, update = ONE serial task      */
enum { LP_F32 = 0, LP_BF16 = 1 };
enum { LP_CAPTURE_GRADS = 1u, /* keep G of the latest step readable by lp_get_grads            */
       LP_TIME_TASKS = 2u,     /* bracket every kernel with timing events (see lp_get_task_time) */
       LP_UNFUSED_UPDATE = 4u, /* write G to memory and run Eq. 6 as a separate kernel. Default:  */
                               /* the update is fused into the epilogue of the G contraction and  */
                               /* G is only stored when LP_CAPTURE_GRADS is set                    */
       LP_SERIAL_TASKS = 8u,   /* measurement aid: enqueue every task on the caller's stream, so  */
                               /* that no two kernels overlap and LP_TIME_TASKS times each alone  */
       LP_RECOMPUTE = 16u,     /* activation recomputation instead of stashing, see below         */
       LP_TRACE_TASKS = 32u }; /* failure detection aid: a one-thread kernel after every task     */
                               /* writes a progress mark to pinned host memory, which             */
                               /* lp_task_progress reads while the device is still busy           */
/* LP_RECOMPUTE (Section III-A names both stashing and recomputation as what the delays between a and
 * the backward pass may stand for): a layer whose input is produced inside its own stage, and whose
 * delay would need a stash of more than four minibatches, keeps that input (with the stored z and
 * the pooling positions that go with it) only until the next layer has read it; when the backward
 * pass of the minibatch reaches the stage, the producing forward task runs again on the stashed
 * weight version.  One more forward contraction per such layer buys (d_l - 2) x batch x features
 * x 2 bytes of stash.  The results are bit-identical to the stashing run. */

/* One layer of the chain (Eqs. 1-2: z = W a (+ b), a = f(z)). */
typedef struct {
  int kind;                      /* LP_FC | LP_CONV                                        */
  int in, out;                   /* FC: features in / out.  CONV: channels in / out        */
  int H, W, R, S, stride, pad;   /* CONV only: input height/width, filter, stride, padding */
  int act;                       /* LP_ACT_*; the last layer must be LP_ACT_NONE           */
  int pool;                      /* 0, or 2 = 2x2 stride-2 max pool after the activation   */
  int has_bias;                  /* 0 = the paper's bias-free Eq. 1                        */
} lp_layer;

typedef struct {
  int batch;          /* minibatch size B                                                  */
  float lr;           /* eta of Eq. 6                                                      */
  float momentum;     /* mu: m <- mu m + G, W <- W - eta m; 0 = plain Eq. 6                */
  int schedule;       /* LP_SCHED_*                                                        */
  int input_dtype;    /* dtype of lp_step's batch: LP_F32 | LP_BF16                        */
  unsigned flags;     /* LP_CAPTURE_GRADS, ...                                             */
} lp_config;

/*
 * Algorithm 1 (partitioning for balanced pipeline generation) on an integer cost model:
 * T_fix[l] = 2 x MACs of layer l (forward + G), T_flex[l] = MACs (delta; 0 for layer 0).
 * Layers are walked in reverse, processors filled up to T_p = ceil(T_tot / n_stages);
 * a delta that does not fit is split into delta'' (stays beside layer l+1) and delta'
 * (next processor); if more than n_stages processors are needed T_p is relaxed by 1%
 * and the allocation restarts.  All outputs are host arrays owned by the caller.
 *   stage_out[n_layers]        stage holding layer l's forward, G and update
 *   delay_out[n_layers]        d_l = stages_used - 1 - stage(l)
 *   dgrad_stage_out[2*n_layers], dgrad_amount_out[2*n_layers]
 *                              the (at most two) pieces of layer l's delta work:
 *                              [2l] = piece placed first (delta'' or the whole),
 *                              [2l+1] = delta' (amount 0 and stage -1 if unsplit)
 *   stages_used, Tp_out, relax_rounds_out   scalars (may be NULL)
 * Errors: LP_ERR_INVALID_ARG for null arrays, n_layers < 1, n_stages < 1, bad shapes.
 */
int lp_plan(const lp_layer* layers, int n_layers, int batch, int n_stages,
            int* stage_out, int* delay_out, int* dgrad_stage_out,
            long long* dgrad_amount_out, int* stages_used, long long* Tp_out,
            int* relax_rounds_out);

/* Same allocation from caller-supplied integer costs (e.g. profiled times); this is the
 * form in which the paper's worked example (Table II -> Table III) is stated. */
int lp_plan_costs(const long long* T_fix, const long long* T_flex, int n_layers, int n_stages,
                  int* stage_out, int* delay_out, int* dgrad_stage_out,
                  long long* dgrad_amount_out, int* stages_used, long long* Tp_out,
                  int* relax_rounds_out);

/* Bytes of device workspace lp_create needs for this network.  `delays` host [n_layers]
 * (NULL = one per stage after the layer, from `stage`); `stage` host [n_layers] (NULL =
 * lp_plan).  Pure host arithmetic; needs no GPU. */
int lp_workspace_size(const lp_layer* layers, int n_layers, int n_stages, const int* stage,
                      const int* delays, const lp_config* cfg, size_t* bytes_out);

/*
 * Build a trainer.  `stage` / `delays`: host [n_layers] or NULL as above; a delay d_l
 * means minibatch n reads weight version max(0, n - d_l) of layer l in BOTH its forward
 * and its delta pass (weight stashing, Section III-A); the ring of layer l holds
 * d_l + 1 bf16 versions.  W0_host[l] (fp32, [out][in]) and b0_host[l] (fp32 [out], may be
 * NULL = zeros or has_bias = 0) are copied before the call returns.  workspace_dev:
 * device, 256-byte aligned, >= lp_workspace_size bytes; zeroed by this call.
 * Uses the current CUDA device; creates its own streams and events: three streams (forward,
 * delta, G + update) per group of stages.  Streams overlap only while each owns a hardware
 * work queue, and a process has CUDA_DEVICE_MAX_CONNECTIONS of those (8 if unset, at most 32),
 * fixed when its CUDA context is created: set the variable to 32 before the first CUDA call.
 * lp_create reads the variable and folds the stages onto (value - 2) / 3 stream triples so that
 * no two of its streams share a queue (LP_STREAM_TRIPLES in the environment overrides the count).
 * Kernel selection: a handle uses one kind of tensor-memory allocation -- a fully connected network
 * whose layers are mostly wide (batch, inputs and outputs all >= 1024) runs every contraction on SM
 * pairs (tcgen05 cta_group::2), every other network runs single-CTA kernels only.  LP_CONV_PAIR=1
 * in the environment also puts wide convolution layers on SM pairs: a measurement mode, not for
 * long runs (networks that alternate the two kinds on the same SMs have stalled in tcgen05.alloc
 * after some 10^6 pair CTAs).  Two handles of different kinds should not run concurrently on one GPU.
 */
int lp_create(lp_handle* out, const lp_layer* layers, int n_layers, int n_stages,
              const int* stage, const int* delays, const lp_config* cfg,
              const float* const* W0_host, const float* const* b0_host,
              void* workspace_dev, size_t workspace_bytes);

/*
 * Enqueue every task of one minibatch: cast+stash of the batch, forward of all layers,
 * loss, and per layer delta / G / update under the handle's schedule.  batch_dev: device,
 * [batch][in] of cfg.input_dtype; labels_dev: device int32 [batch], values in [0, classes).
 * `stream` (a cudaStream_t, may be 0) orders the call after the caller's earlier work;
 * the batch and labels are consumed by the first kernel, which runs on `stream`, so the
 * caller may overwrite them after later work on `stream`.  Tasks of consecutive calls
 * overlap on the device as far as the delays allow.
 */
int lp_step(lp_handle h, const void* batch_dev, const int* labels_dev, void* stream);

/*
 * Operational parallelism (Section III-B, Fig. 5(c)-(d); Algorithm 1's OP(T_idle, T_flex)): the
 * delta contraction of layer l is divided BY OUTPUT CHANNELS into delta'' -- borrowed by the
 * processor that holds layer l+1 -- and delta', which stays with layer l; the two pieces are
 * independent and run concurrently.  piece_stage / piece_amount: host [2 * n_layers] in the layout
 * lp_plan / lp_plan_costs write ([2l] = delta'' or the whole, [2l+1] = delta'; amount 0 = no such
 * piece).  For every layer with two pieces the columns of delta^{l-1} are divided in the ratio of
 * the amounts, rounded to whole tiles of the contraction kernel (at least one tile each); piece
 * [2l] is enqueued on the delta stream of stage piece_stage[2l], piece [2l+1] on that of
 * piece_stage[2l+1], each with the unchanged f' epilogue, and delta^{l-1} counts as written when
 * both have finished.  Layers whose delta kernel has a single column tile, or runs split-K, keep
 * one piece.  The numbers do not change: every output element is produced by the same
 * instructions in the same order as in the unsplit launch.  split_col_out (host [n_layers], may be
 * NULL) receives the first column of delta' (0 = unsplit).  Must be called before the first
 * lp_step; LP_SCHED_FUSED_B runs the pieces back to back inside its one backward task.
 */
int lp_set_delta_split(lp_handle h, const int* piece_stage, const long long* piece_amount, int* split_col_out);

/* Make `stream` wait for everything enqueued so far (all updates applied: every layer
 * holds version = number of lp_step calls). Does not block the host. */
int lp_flush(lp_handle h, void* stream);

/* Copy layer `layer`'s fp32 master weights (host W_out [out][in], b_out [out], either may
 * be NULL) after waiting for its last enqueued update; *version = updates applied. */
int lp_get_weights(lp_handle h, int layer, float* W_out, float* b_out, long long* version);

/* G (host dW_out [out][in]) and bias gradient (host db_out [out]) of minibatch `step`;
 * needs LP_CAPTURE_GRADS (or LP_UNFUSED_UPDATE) and only the most recently enqueued step is
 * held -> otherwise LP_ERR_NOT_READY. Blocks the host until that step's G task has finished. */
int lp_get_grads(lp_handle h, int layer, long long step, float* dW_out, float* db_out);

/*
 * Verification access.  These three calls exist so that every task of the step can be
 * checked in isolation against a reference fed with the SAME operands: write operands
 * into the handle's buffers, run one task, read its outputs.  All three block the host
 * until the device is idle and must not be mixed with steps still in flight.
 * Host data is fp32; bf16 buffers are converted (round-to-nearest-even on write).
 *
 *   buffer            shape of host array          `index` selects
 *   LP_BUF_INPUT      [batch][in]   a^{l-1}, stashed input of layer l    minibatch (slot = index mod slots)
 *   LP_BUF_Z          [batch][out]  stored z^l (GELU layers only)        minibatch
 *   LP_BUF_DELTA      [batch][out]  delta^l = dE/dz^l                    minibatch
 *   LP_BUF_LOGITS     [batch][classes] z^L (layer ignored)               minibatch
 *   LP_BUF_LABELS     [batch] labels as floats (layer ignored)           minibatch
 *   LP_BUF_LOSS       [1] (layer ignored)                                minibatch
 *   LP_BUF_RING_W     [out][in]  bf16 weight version                     ring slot
 *   LP_BUF_RING_B     [out]      fp32 bias version                       ring slot
 *   LP_BUF_MASTER_W/B, LP_BUF_MOM_W/B, LP_BUF_GRAD_W/B   [out][in] / [out]   (index ignored)
 *   LP_BUF_POOL_IDX   [pooled pixels][channels]  position 0..3 of the maximum in its 2x2 window   minibatch
 * For convolution layers "batch" rows become batch*H*W pixel rows (NHWC) and [out][in] becomes
 * [Cout][R][S][Cin].  A first convolution layer with 9*Cin <= 64 stores its input as the matrix of
 * 3x3 patches; LP_BUF_INPUT of that layer is still exchanged as the image [batch][H][W][Cin]
 * (a write builds every pixel's patch row, a read returns the centre taps).
 */
enum { LP_BUF_INPUT = 0, LP_BUF_Z = 1, LP_BUF_DELTA = 2, LP_BUF_LOGITS = 3, LP_BUF_LABELS = 4, LP_BUF_LOSS = 5,
       LP_BUF_RING_W = 6, LP_BUF_RING_B = 7, LP_BUF_MASTER_W = 8, LP_BUF_MASTER_B = 9, LP_BUF_MOM_W = 10,
       LP_BUF_MOM_B = 11, LP_BUF_GRAD_W = 12, LP_BUF_GRAD_B = 13, LP_BUF_POOL_IDX = 14 };
int lp_debug_read(lp_handle h, int buffer, int layer, long long index, float* out_host);
int lp_debug_write(lp_handle h, int buffer, int layer, long long index, const float* in_host);

/* Run ONE task of minibatch `step` on the buffers as they stand (slots and weight version
 * chosen exactly as lp_step would for that minibatch) and wait for it.  Does not advance
 * the step counter.  LP_TASK_FORWARD: Eqs. 1-2; LP_TASK_LOSS: loss and delta^L;
 * LP_TASK_DELTA: Eqs. 3-4 for layer >= 1 (writes delta^{layer-1}); LP_TASK_G: Eq. 5 -- with
 * the fused update (default) this kernel also applies Eq. 6 to W and writes ring slot
 * (step+1) mod slots; LP_TASK_UPDATE: Eq. 6 for the bias (fused mode) or for W and bias
 * (LP_UNFUSED_UPDATE). */
enum { LP_TASK_FORWARD = 0, LP_TASK_LOSS = 1, LP_TASK_DELTA = 2, LP_TASK_G = 3, LP_TASK_UPDATE = 4 };
int lp_debug_run_task(lp_handle h, int task, int layer, long long step);

/* Plan actually in use: host arrays [n_layers] (any may be NULL). ring_slots = d_l + 1. */
int lp_get_schedule(lp_handle h, int* stage, int* delay, int* ring_slots);

/* For minibatch `step`: per layer the weight version read by forward (v_fwd) and by delta
 * (v_bwd) and the ring slot it sat in.  Host arrays [n_layers].  Integer bookkeeping of
 * the last 4096 steps. */
int lp_get_version_log(lp_handle h, long long step, int* v_fwd, int* v_bwd, int* slot);

/* Mean cross-entropy of minibatch `step` (one of the last 256 steps); blocks the host
 * until that step's loss kernel has finished. */
int lp_get_loss(lp_handle h, long long step, float* loss);

/* 0, or the status word written by a kernel: a bounded wait that expired (values 1..26: returns
 * LP_ERR_TIMEOUT), or a label outside [0, classes) met by the loss kernel (value 64: returns
 * LP_ERR_INVALID_ARG; that row contributes no one-hot term and the minibatch's loss is NaN --
 * the label is never used as an address).  *detail receives the word.  Blocks until the device
 * is idle. */
int lp_device_status(lp_handle h, int* detail);

/* Which tasks the device has not finished (needs LP_TRACE_TASKS; the paper has no counterpart: it is
 * how a stalled pipeline is diagnosed without waiting for it).  Writes to text[capacity] (host, NUL
 * terminated, truncated to fit) one line per scheduler stream with unfinished work -- tasks done of
 * tasks enqueued, whether the next one has started, and the next up to three unfinished tasks as
 * kind(layer, minibatch) -- then, copied on a stream of its own: the status word, how many CTAs of the
 * SM-pair kernel have passed each of its phases, how many tensor-memory allocations took more than
 * 20000 cycles, and every SM on which a CTA sits inside tcgen05.alloc (with the kernel it belongs to
 * and the columns this library's CTAs hold there).  Does not wait for the scheduler's streams; call it
 * from any host thread while another is blocked in a synchronisation.  LP_ERR_NOT_READY without
 * the flag. */
int lp_task_progress(lp_handle h, char* text, int capacity);

/* Needs LP_TIME_TASKS.  For task kind LP_TASK_* (plus LP_TASK_CAST = 5): number of kernel
 * launches timed since the last lp_reset_task_times and the sum of their durations in
 * milliseconds, each measured with CUDA events on the stream the kernel ran on.  Blocks
 * until the device is idle.  At most 32768 launches are timed between resets. */
enum { LP_TASK_CAST = 5 };
int lp_get_task_time(lp_handle h, int task, long long* launches, double* total_ms);
int lp_reset_task_times(lp_handle h);
/* The same sums for one layer: Algorithm 1's `profile` step.  With LP_TIME_TASKS | LP_SERIAL_TASKS
 * these are the costs of the tasks alone on the GPU: T_fix[l] = forward + G (+ update), T_flex[l] =
 * delta, in any integer unit (e.g. nanoseconds), are what lp_plan_costs takes. */
int lp_get_layer_task_time(lp_handle h, int task, int layer, long long* launches, double* total_ms);
/* Needs LP_TIME_TASKS.  The timeline behind lp_get_task_time: for the first min(capacity, launches)
 * timed launches of `task`, in launch order, start_ms[i] and end_ms[i] (host arrays) receive the
 * kernel's begin and end in milliseconds after the first event timed since the last reset (of any
 * task kind).  *count_out = entries written.  Blocks until the device is idle. */
int lp_get_task_timeline(lp_handle h, int task, int capacity, float* start_ms, float* end_ms, int* count_out);

/* Number of kernels this handle has launched so far. */
long long lp_kernel_launches(lp_handle h);

/* Tuning hook for experiments: force the GEMM tile width (64, 128, 256, or 512 = 256 x 256 tile on an
 * SM pair with tcgen05 cta_group::2, plain matrices only; 0 = automatic), the
 * shared-memory pipeline depth (0 = automatic) and the split-K factor of the forward / delta
 * contractions (0 = automatic, 1 = off; adding 256 forces one tile per CTA, adding 512 forces
 * persistent CTAs that loop over tiles) for handles created afterwards. */
int lp_set_tuning(int tile_n, int stages, int split_k);

const char* lp_last_error(lp_handle h); /* valid until the next call on h; h may be NULL */
int lp_destroy(lp_handle h);

/*
 * The three contractions of an FC layer in isolation, on caller-owned device buffers
 * (bf16 operands, fp32 accumulate, fp32 result C[M][ldc]); for kernel-level checks.
 *   which = 0  forward  (Eq. 1):  C[M][N] = A[M][K] . B[N][K]^T     (A = a, B = W)
 *   which = 1  delta    (Eq. 4):  C[M][N] = A[M][K] . B[K][N]       (A = delta, B = W)
 *   which = 2  G        (Eq. 5):  C[M][N] = A[K][M]^T . B[K][N]     (A = delta, B = a)
 * lda / ldb / ldc are row pitches in elements; lda and ldb must be multiples of 8, ldc of
 * 4; all base pointers 16-byte aligned.  `stream` is a cudaStream_t.
 */
int lp_gemm_bf16(int which, int M, int N, int K, const void* A_dev, int lda,
                 const void* B_dev, int ldb, float* C_dev, int ldc, void* stream);

/* Status word of the lp_gemm_bf16 launches on the current device since the last call: waits for
 * the device, returns LP_OK (word 0) or LP_ERR_TIMEOUT (a bounded wait inside a kernel ran out;
 * *detail, may be NULL, receives the word: 1 producer, 2 MMA issuer, 3 / 4 epilogue, 11..13 the
 * same roles of the SM-pair kernel), and clears the word. */
int lp_gemm_status(int* detail);

/* Verification of the bounded waits (Eq. 1 contraction as lp_gemm_bf16 with which = 0, K > 64).
 * Every wait on a barrier inside the kernels gives up after a cycle limit, records a status
 * word and lets the kernel drain and return, so that a broken hand-off can never hang the GPU.
 * This call makes one such wait run out ON PURPOSE, in the only harmless way: the TMA producer
 * is told to skip the last k-block of every tile, so the MMA issuer waits for a fill that never
 * comes, for `limit_cycles` SM cycles (1e3 .. 2e9) instead of the default of about two seconds.
 * Nothing faults and nothing spins unbounded; C receives partial sums.  Afterwards
 * lp_gemm_status must report LP_ERR_TIMEOUT and the next ordinary launch must be correct. */
int lp_debug_gemm_starved(int M, int N, int K, const void* A_dev, int lda, const void* B_dev, int ldb,
                          float* C_dev, int ldc, long long limit_cycles, void* stream);

/*
 * Softmax cross-entropy without a handle, a workspace or any allocation.  (The paper has
 * no counterpart: it is the loss kernel of lp_step offered to callers that cannot give the
 * library memory to work in.)
 *
 * Who needs it: code that evaluates the loss outside a trainer -- a validation pass, a
 * unit test of a custom head -- from a context where device memory cannot be requested:
 * the process has handed the whole device to a pooling allocator it must not bypass, it
 * runs under a fixed memory budget agreed at start-up, or it sits in a latency-critical
 * loop where a cudaMalloc (which may synchronise the device) is not acceptable.  Such a
 * caller has the logits and the labels and room for the outputs, but nothing to pass as
 * the per-row scratch the kernel needs.
 *
 * Computes exactly what the loss task of lp_step computes:
 *   delta_dev[r][c] = bf16( (softmax(logits_dev[r])[c] - [c == labels_dev[r]]) / batch )
 *   *loss_dev       = mean over rows of -log softmax(logits_dev[r])[labels_dev[r]]
 * logits_dev: device fp32 [batch][ld_logits]; labels_dev: device int32 [batch], values in
 * [0, classes) -- a label outside that range is never used as an address: its row gets no
 * one-hot term and *loss_dev becomes NaN; delta_dev: device bf16 [batch][ld_delta], ld_delta >= classes rounded up to
 * a multiple of 8 (the lanes up to that multiple are written as zeros); loss_dev: device
 * fp32 [1].  All caller-owned.  `stream` is a cudaStream_t (may be 0); the call is
 * asynchronous.
 *
 * The scratch (one fp32 per row plus a counter) is a fixed array inside the library image:
 * LP_XENT_STATIC_MAX_BATCH rows, about 64 KiB, resident on every GPU that loads the
 * library for as long as the process lives.  Consequences the caller must know:
 *   - batch > LP_XENT_STATIC_MAX_BATCH (or batch < 1, classes < 1, bad pitches, null
 *     pointers) -> LP_ERR_INVALID_ARG, nothing is launched; lp_last_error(NULL) says which.
 *   - all calls on one GPU share that array.  The call clears the part that must start
 *     at zero, so leftovers of an earlier call are harmless, but two calls that overlap
 *     on the device (different streams, no ordering between them) race on it and give
 *     wrong losses.  Order them.
 *   - the first call on each device looks up the array's device address (a host-side
 *     query, no allocation).  Make that first call outside any stream capture.
 * Calls no cudaMalloc / cudaFree and no routine that allocates.
 */
#define LP_XENT_STATIC_MAX_BATCH 16384
int lp_softmax_xent_static(const float* logits_dev, int ld_logits, const int* labels_dev, void* delta_dev,
                           int ld_delta, float* loss_dev, int batch, int classes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* LAYERPIPE_H_ */
