/*
 * abs_b200 -- C ABI of the B200 implementation of the ABS parameter-server
 * round loop (adaptive bounded staleness, arXiv 2301.08895).
 *
 * One context simulates N workers and one server on one GPU.  A round is
 * Algorithm 1's "server executes" block: wait for the K^t fastest uploads,
 * apply Eq. 3, adapt K (Eq. 5) and the staleness threshold (Eq. 4), update the
 * ages and restart over-stale workers (Eq. 6).  Worker uploads are minibatch
 * gradients (Eq. 2 with U = 1) evaluated at the model version the worker
 * holds; the bounded staleness lets the library keep only S + 1 model versions
 * in a ring instead of one model per worker.
 *
 * Conventions
 *  - Every function returns ABS_OK (0) or a negative ABS_E* code; nothing
 *    throws, aborts or prints.  abs_last_error() gives the text of the last
 *    failure on the calling thread.
 *  - "device" pointers are CUDA device addresses of the current device,
 *    "host" pointers are ordinary memory.  The library allocates no device
 *    memory: the caller passes one workspace (size from abs_workspace_bytes)
 *    that must stay valid and untouched until abs_destroy.
 *  - All work is enqueued on the caller's stream; abs_run_rounds synchronises
 *    that stream once before it returns.
 *  - Parameter vector layout (w0 and abs_get_params): for each layer in order
 *    W[in][out] row-major followed by b[out]; least squares has w[d] only.
 *  - Times are integer ticks, 2^20 per time unit.
 */
#ifndef ABS_B200_H
#define ABS_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ABS_OK            0
#define ABS_EINVAL       -1  /* bad argument (text names it) */
#define ABS_ENOSPACE     -2  /* workspace, trace capacity or round capacity too small */
#define ABS_EUNSUPPORTED -3  /* unknown kind, or local_steps > 1 for a model the local-step kernel does not cover */
#define ABS_ESTATE       -4  /* call order */
#define ABS_ECUDA        -5  /* a CUDA call failed; sticky for the context */
#define ABS_ETIMEOUT     -6  /* a bounded device-side wait (100 ms) expired */
#define ABS_EDIVERGED    -7  /* a non-finite loss was uploaded; see abs_run_rounds */
#define ABS_ERANGE       -8  /* simulated time left the 2^53 tick range */
#define ABS_ESTALE       -9  /* ABS_RESTART_NONE: an upload older than the staleness bound arrived, i.e. older than
                                the model versions the context keeps; the rounds before it stay valid */

/* model kinds: the sample loss f of Eq. 1 */
#define ABS_LSQ      0  /* f = 1/2 (x.w - y)^2, dims = {d, 1}, no bias */
#define ABS_SOFTMAX  1  /* one affine layer + soft-max cross-entropy */
#define ABS_MLP      2  /* affine layers with ReLU between them + soft-max cross-entropy */
#define ABS_CNN      3  /* the paper's model class (Sec. V-A): two blocks of k x k convolution (stride 1, no padding)
                           + ReLU + 2 x 2 max-pool in front of an ABS_MLP of at least two layers; see `conv` */

/* storage/arithmetic type */
#define ABS_FP32             0  /* fp32 data, fp32 models, fp32 FMA */
#define ABS_BF16_FP32MASTER  1  /* bf16 data, bf16 model versions, activations and deltas;
                                   fp32 accumulation; fp32 master parameters */

#define ABS_K_ADAPTIVE      0   /* K^{t+1} from Eq. 5 */
#define ABS_K_FIXED         1   /* K^t = K0 for all t (K-sync / K-async / ASGD baselines, Sec. II-B) */
#define ABS_BOUND_ADAPTIVE  0   /* threshold from Eq. 4, capped by the staleness bound */
#define ABS_BOUND_FIXED     1   /* threshold = staleness bound in every round (Fig. 1 setting) */
#define ABS_BOUND_OFFSET    2   /* Eq. 4 with the constant a given: max(1, floor(N/K) + bound_offset), capped by
                                   the staleness bound (the sweep over a of Sec. V-B) */

#define ABS_RESTART_ALGORITHM1 0 /* Eq. 6 in the order Algorithm 1 performs it: ages are incremented first, then a
                                   non-selected worker restarts iff its new age exceeds the threshold; consumed
                                   staleness never exceeds the staleness bound */
#define ABS_RESTART_EQ6        1 /* Eq. 6 as printed: the age before the increment is tested, so a worker restarts
                                   one round later and a consumed gradient may be staleness bound + 1 rounds old
                                   (the library then keeps one more model version) */
#define ABS_RESTART_NONE       2 /* no forced restarts at all: AdaSync (with ABS_K_ADAPTIVE) and K-async SGD (with
                                   ABS_K_FIXED), the comparison systems of Sec. II-B and Sec. V.  Staleness is then
                                   unbounded in principle; the library still keeps staleness bound + 1 model
                                   versions, and a run in which an older upload arrives ends with ABS_ESTALE at
                                   that round (choose the bound, at most 255, above the staleness the time law
                                   can produce).  The threshold of Eq. 4 is still computed and reported */

/* execution-time laws (random execution times with stragglers, Sec. V-A) */
#define ABS_T_CONST        0    /* shift */
#define ABS_T_EXP          1    /* Exp(rate) */
#define ABS_T_SHIFTED_EXP  2    /* shift + Exp(rate) */
#define ABS_T_PARETO2      3    /* Pareto, shape 2, minimum `scale` */
#define ABS_T_GAMMA        4    /* shift + Gamma(shape, rate), integer shape in [1, 64]: the sum of `shape`
                                   exponential draws (the law the paper draws execution times from) */

#define ABS_FLAG_NO_TENSOR_CORES 1  /* run the hidden-layer contractions on the FP32-FMA kernels */
#define ABS_FLAG_NO_OVERLAP      2  /* enqueue every kernel on the caller's stream (no side stream for the
                                       server-side kernels of the next round) */
#define ABS_FLAG_NO_BULK_PIPELINE 32 /* bf16 least squares: per-warp 16-byte loads (rows read from HBM, then again
                                       from L2) instead of the bulk-copy pipeline through shared memory */
#define ABS_FLAG_NO_FUSED_BACKWARD 64 /* tensor-core networks: a layer's delta back-propagation and its weight
                                       gradient always get a launch each */
#define ABS_FLAG_NO_PERSISTENT   8  /* small least-squares problems: one kernel launch per step of a round
                                       instead of one persistent kernel that runs all enqueued rounds */

/* kernel classes reported by abs_profile_read */
#define ABS_KC_CTL     0  /* arrival selection + Eq. 4-6 bookkeeping */
#define ABS_KC_GATHER  1  /* minibatch row gather */
#define ABS_KC_FWD     2  /* hidden-layer forward contraction (Eq. 2) */
#define ABS_KC_DGRAD   3  /* hidden-layer delta back-propagation */
#define ABS_KC_WGRAD   4  /* weight gradient summed over the selected workers (Eq. 3) */
#define ABS_KC_OUTPUT  5  /* output layer: forward + loss, its back-propagation and gradient */
#define ABS_KC_LSQ     6  /* least-squares residual + gradient; with local_steps > 1: the workers' local steps
                             (single-layer models), or their set-up, row layouts and copy refreshes (networks) */
#define ABS_KC_UPDATE  7  /* Eq. 3 step + ring write */
#define ABS_KC_ROUNDS  8  /* whole rounds (control step + Eq. 2 + Eq. 3) of a small least-squares problem
                             in one persistent kernel; one launch per abs_enqueue_rounds call */
#define ABS_KC_CONV    9  /* ABS_CNN: the convolution blocks, forward and backward */
#define ABS_KC_COUNT   10

#define ABS_MAX_LAYERS   7
#define ABS_MAX_WORKERS  1024
#define ABS_MAX_BOUND    255

typedef struct abs_ctx abs_ctx;

/* Everything the paper calls f, D, B, eta, w^0 (Sec. II-A). */
typedef struct {
  int kind;                 /* ABS_LSQ | ABS_SOFTMAX | ABS_MLP */
  int n_layers;             /* affine layers; dims has n_layers + 1 entries */
  int dims[ABS_MAX_LAYERS + 1]; /* e.g. {3072,1024,512,10}; LSQ: {d,1}; last dim = classes (<= 64) */
  int conv[6];              /* ABS_CNN only: {H, W, C_in, k, C1, C2}: image size and channels, kernel size, output
                               channels of the two blocks.  Dataset rows are images stored [H][W][C_in]; both
                               convolution outputs must be even-sized; dims[0] must equal the number of features
                               the second block delivers, (rows x columns x C2) of its pooled maps, which are
                               flattened in that order.  Parameter vector: W1[k][k][C_in][C1], b1[C1],
                               W2[k][k][C1][C2], b2[C2], then the affine layers as for ABS_MLP.  A block has at
                               most 4096 parameters; local_steps must be 1 */
  int batch;                /* B of Eq. 2, 1..1024 */
  float lr;                 /* eta, constant */
  int dtype;                /* ABS_FP32 | ABS_BF16_FP32MASTER */
  int local_steps;          /* U of Eq. 2, 1..1024.  U > 1 (local SGD inside a job: the upload is the sum of
                               the U minibatch-gradient sums along the worker's own trajectory, the loss the
                               average of its U minibatch losses) is implemented for ABS_LSQ and ABS_SOFTMAX
                               with <= 16 classes, <= 12288 parameters and batch x classes <= 8192 (the worker's
                               copy lives in shared memory), and for multi-layer ABS_MLP (the selected workers'
                               copies live in the workspace: 8 bytes per parameter and worker, 6 in bf16);
                               in the bf16 configurations
                               each step is evaluated at the bf16 rounding of the fp32 copy */
  int k_mode;               /* ABS_K_* */
  int bound_mode;           /* ABS_BOUND_* */
  int bound_offset;         /* the constant a of Eq. 4 when bound_mode = ABS_BOUND_OFFSET (else ignored);
                               floor(N/K0) + a must not exceed the staleness bound */
  int restart_rule;         /* ABS_RESTART_* */
  int sa_penalty;           /* 0 | 1.  1: staleness-aware step size (Sec. I, Sec. V: "SA"): the step size of a stale
                               gradient is penalised linearly in its delay, i.e. upload k enters the sum of Eq. 3
                               as g_k / max(1, tau_k).  With ABS_RESTART_NONE this is SA-AdaSync */
  int max_rounds;           /* trace capacity: total rounds this context may run */
  int flags;                /* ABS_FLAG_* bits */
  int data_on_host;         /* 0: X, y are device pointers owned by the caller and must outlive
                               the context.  1: X, y are host pointers; abs_init copies them into
                               the workspace (abs_workspace_bytes accounts for the room) */
  const void* X;            /* [n_samples][dims[0]] row-major (ABS_CNN: [n_samples][H*W*C_in]); float (FP32) or
                               bf16 bits (BF16) */
  const void* y;            /* float targets (LSQ) or int32 labels in [0, classes) */
  long long n_samples;      /* M of Eq. 1; worker n owns samples [n*M/N, (n+1)*M/N) */
  const float* w0;          /* host, n_params floats, copied by abs_init */
  void* workspace;          /* device, 256-byte aligned */
  size_t workspace_bytes;
  void* stream;             /* cudaStream_t (0 = default stream) */
} abs_model_desc;

typedef struct {
  int kind;                 /* ABS_T_* */
  double shift, rate, scale;
  int slow_mod, slow_rem;   /* workers with n % slow_mod == slow_rem are slow (slow_mod 0: none) */
  double slow_factor;       /* their durations are multiplied by this */
  int shape;                /* ABS_T_GAMMA: number of exponential draws summed (else ignored) */
} abs_time_dist;

/* Caller-owned host arrays receiving rounds [first_round, first_round + n_rounds).
 * Per-round arrays need n_rounds entries (sel_off/rst_off: n_rounds + 1, offsets into the flat
 * arrays relative to the first returned round).  Flat arrays need cap_sel / cap_rst entries.
 * Any pointer may be NULL to skip that field. */
typedef struct {
  int32_t*  K;          /* K^t */
  int32_t*  n_restart;  /* workers restarted by Eq. 6 after round t */
  int32_t*  theta;      /* threshold used by that restart test (Eq. 4 at K^{t+1}) */
  uint64_t* T_end;      /* tick at which the K^t-th upload arrived */
  float*    loss_mean;  /* estimate of f(w^t): mean uploaded loss */
  uint64_t* comm;       /* cumulative communication rounds (Sec. V-B) after round t */
  int64_t*  sel_off;    /* [n_rounds + 1] */
  int64_t*  rst_off;    /* [n_rounds + 1] */
  int32_t*  sel_id;     /* selected worker ids, arrival order */
  int32_t*  sel_tau;    /* staleness of each consumed gradient */
  float*    sel_loss;   /* each upload's mean minibatch loss */
  int32_t*  rst_id;     /* restarted worker ids, ascending */
  size_t    cap_sel, cap_rst;
} abs_trace;

/* Bytes of device workspace a context needs (Sec. II-A sizes: N workers, ring of S + 1 model
 * versions, activations for N*B rows, trace for max_rounds).  Only kind, dims, batch, dtype,
 * local_steps, flags, max_rounds, data_on_host and n_samples of `model` are read. */
int abs_workspace_bytes(const abs_model_desc* model, int W, int staleness_bound, size_t* out);

/* Algorithm 1, initialisation: K^0, threshold N/K^0 + a := staleness_bound, w^0 broadcast to all
 * workers (every worker starts job 0 at tick 0).  Copies w0 (and the dataset if data_on_host)
 * to the device, enqueues the set-up kernels, synchronises the stream.
 * W in [1, 1024], K0 in [1, W], staleness_bound in [0, 255].
 * First call per process should come before any stream capture. */
int abs_init(abs_ctx** out, const abs_model_desc* model, int W, int K0, int staleness_bound,
             const abs_time_dist* time_dist, unsigned long long seed);

/* Algorithm 1, n iterations of the server loop (Eq. 2-6).  Enqueues n rounds without host
 * synchronisation between them, then synchronises once.  Returns ABS_EDIVERGED if a non-finite
 * loss was uploaded: the round in which it happened and all later ones are not applied, the
 * parameters and the trace stay valid up to the round before.  Errors are sticky. */
int abs_run_rounds(abs_ctx* ctx, int n);

/* Same as abs_run_rounds but returns after enqueueing; the device status is read by the next
 * abs_run_rounds / abs_rounds_done / abs_get_* call.  Used to time the loop with CUDA events. */
int abs_enqueue_rounds(abs_ctx* ctx, int n);

/* Rounds completed so far (synchronises the stream). */
int abs_rounds_done(abs_ctx* ctx, int* rounds);

/* The global model w^t (Eq. 3) as fp32, layout of w0.  dst_host needs n_params floats
 * (cap = its capacity in floats); *d_out receives n_params. */
int abs_get_params(abs_ctx* ctx, float* dst_host, size_t cap, size_t* d_out);

/* Per-round record of Algorithm 1's decisions for rounds [first_round, first_round + n_rounds):
 * K^t, the arrival-ordered selected workers, each gradient's staleness, the restarted workers. */
int abs_get_trace(abs_ctx* ctx, int first_round, int n_rounds, abs_trace* out_host);

/* Checkpoint of the simulation between rounds (Algorithm 1's whole state: the global model and the
 * ring of model versions, every worker's held version, job index and completion tick, K^t, the
 * threshold, f(w^0), the clock, and the trace so far; the Philox streams are counter-based, so
 * nothing of the generators needs saving).  abs_state_bytes: size of the image.  abs_save_state:
 * synchronises the stream and writes the image to dst_host (cap bytes; ABS_ENOSPACE if too small);
 * *written receives its size.  abs_restore_state: loads an image into a context that abs_init
 * created with the same model kind and sizes, batch, step size, dtype, local steps, flags, W, K0,
 * staleness bound, modes, time distribution, seed and max_rounds (ABS_EINVAL otherwise, context
 * unchanged); the context then continues with
 * round `rounds completed in the image`, bit-identically to the context that saved it.  The
 * dataset, w0 and profiling state are not part of the image.  Host memory is the caller's. */
int abs_state_bytes(abs_ctx* ctx, size_t* out);
int abs_save_state(abs_ctx* ctx, void* dst_host, size_t cap, size_t* written);
int abs_restore_state(abs_ctx* ctx, const void* src_host, size_t bytes);

/* Kernels of ours launched on behalf of this context so far (set-up included). */
int abs_launch_count(abs_ctx* ctx, long long* launches);

/* Stand-alone operation: Eq. 2 with U = 1 for n workers of the least-squares model at one model w,
 * and the mean of their uploads (the sum of Eq. 3 divided by n).  Worker i's minibatch is the B
 * sample indices idx[i*B .. i*B+B).  Results: loss_out[i] = mean_b 1/2 (x_b.w - y_b)^2 and
 * g_out[j] = 1/(n B) sum_i sum_b (x_b.w - y_b) x_b[j].
 * All pointers are device memory: X [n_samples][d] and w [d] in the storage type of `dtype`
 * (float, or bf16 for ABS_BF16_FP32MASTER), y float, idx int32 [n*B], g_out float [d], loss_out
 * float [n], scratch float [scratch_floats] with scratch_floats >= n*d (per-worker partial sums,
 * contents undefined afterwards).  n in [1, 1024], B in [1, 1024], d in [1, 2^20].
 * Enqueues on `stream` and returns without synchronising. */
int abs_lsq_gradient(const void* X, const float* y, const void* w, const int* idx, int n, int B, int d,
                     int dtype, float* scratch, size_t scratch_floats, float* g_out, float* loss_out,
                     void* stream);

/* abs_lsq_gradient for callers that must not allocate (the paper has no counterpart; this is a
 * packaging variant of the operation above).  Meant for code that runs where cudaMalloc is off
 * limits: inside a pre-sized memory plan, in a process whose device memory is entirely owned by
 * another component, or on a path where an allocation's implicit synchronisation is not allowed.
 * Same arguments and results as abs_lsq_gradient without the scratch pair: the per-worker
 * partial sums go to a fixed 4 MiB array built into the library (every GPU that loads the
 * library holds it until the process exits), so n*d must not exceed 1048576 floats -- larger
 * requests fail with ABS_ENOSPACE and change nothing.  The function calls no allocator of any
 * kind.  The first call on each device looks up the array's device address (that device must be
 * current); make that first call outside any stream capture.  All calls on a device share the
 * one array and it keeps the previous call's contents (each call overwrites what it reads, so
 * nothing has to be cleared), which means two calls that may overlap on the GPU -- different
 * streams, or different host threads -- race on it: run them on one stream or order them with
 * events. */
int abs_lsq_gradient_noalloc(const void* X, const float* y, const void* w, const int* idx, int n, int B,
                             int d, int dtype, float* g_out, float* loss_out, void* stream);

/* How the context runs (the paper has no counterpart): *partials = number of fp32 partial sums
 * the Eq. 3 step adds up per parameter (0: one per selected worker), *row_block = padding unit of
 * a version group's gradient rows, *rows_cap = row capacity of the activation buffers,
 * path[l] (n_layers entries) = 0 FP32-FMA tiles, 1 tensor cores, 2 narrow output layer.
 * Any pointer may be NULL. */
int abs_get_plan(abs_ctx* ctx, int* partials, int* row_block, int* rows_cap, int* path);

/* Measurement aid (the paper has no counterpart).  After abs_profile_start, every kernel launch
 * of this context is bracketed by a pair of CUDA events on the context's stream until
 * max_launches pairs are used.  abs_profile_read synchronises, adds the elapsed times up per
 * kernel class (ABS_KC_*; both arrays need ABS_KC_COUNT entries), and ends profiling. */
int abs_profile_start(abs_ctx* ctx, int max_launches);
int abs_profile_read(abs_ctx* ctx, long long* launches, double* total_ms);
/* Before abs_profile_read: the recorded launches one by one, in launch order (both streams): kernel
 * class and the times of the two bracketing events in ms since the first recorded launch.  The
 * arrays need `cap` entries; *n_out receives the number filled.  Synchronises. */
int abs_profile_timeline(abs_ctx* ctx, int cap, int* cls, float* start_ms, float* end_ms, int* n_out);

/* Test aid for the failure path of the device-side waits (the paper has no counterpart).  Every wait
 * inside the library's kernels (on an mbarrier or a completion counter) gives up after a time limit,
 * raises the context's device status and lets the kernel return normally.  This call launches a
 * one-warp kernel that waits, with the library's own wait routine and a limit of limit_us
 * microseconds (1 .. 1000000), on a barrier that nothing ever signals, then synchronises.  It is
 * expected to return ABS_ETIMEOUT (abs_last_error names site 900); the context is then in the same
 * sticky state as after a real expiry: no further rounds, while abs_get_params, abs_get_trace and
 * abs_destroy keep working.  Nothing faults, traps or hangs. */
int abs_selftest_wait_timeout(abs_ctx* ctx, int limit_us);

int abs_destroy(abs_ctx* ctx);

/* Text of the last error on this thread ("" if none). */
const char* abs_last_error(void);

#ifdef __cplusplus
}
#endif
#endif
