/*
 * local_adaalter.h — C-ABI of the Local AdaAlter hot-path library (CUDA, sm_100a).
 *
 * The library simulates W data-parallel workers on ONE GPU: every worker owns a
 * replica of a flat fp32 parameter vector x (N coordinates, the concatenation of
 * K tensors) and of the squared-gradient accumulator B^2; one further array holds
 * the accumulator as of the last synchronisation, which Algorithm 3 of
 * arXiv 1911.09030 uses as the (worker-independent) denominator.  All state lives
 * in device memory and every arithmetic step of the method runs in CUDA kernels.
 *
 * Conventions
 *   - Every function returns an int status: LA_OK (0) or a negative LA_E* code.
 *     Nothing throws, aborts or traps.  la_last_error() gives the message of the
 *     most recent failure on a context (or of the last failed la_create*).
 *   - "host" pointers are ordinary CPU memory (pinned or pageable); "device"
 *     pointers are CUDA global memory of the context's device.  Unless stated
 *     otherwise the library copies what it is given and keeps no reference.
 *   - A context is bound to one device and one stream; all kernels are enqueued
 *     on that stream.  One caller thread at a time per context.
 *   - Calls that only enqueue work return before it finishes (la_local_step,
 *     la_sync, la_run, the la_set_* uploads); la_read_state, la_get_stats and
 *     la_destroy synchronise the stream.
 *   - Rounding contract (what "the same result" means): fp32 IEEE-754, one
 *     rounding per written operation, fused multiply-add where stated:
 *       eps2 = eps*eps;  q = (float)t' * eps2;  d = B2stale[j] + q;
 *       r = eta_t / sqrtf(d);  x = fmaf(-r, g, x);  B2 = fmaf(g, g, B2);
 *       mean over workers = adjacent-pair tree sum, then one division by (float)W.
 */
#ifndef LOCAL_ADAALTER_H_
#define LOCAL_ADAALTER_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct la_ctx la_ctx; /* opaque; owned by the library until la_destroy */

enum {
  LA_OK = 0,
  LA_EINVAL = -1, /* bad argument (NULL handle, N=0, W=0, H=0, eps<=0, non-finite eta, ...) */
  LA_ENOMEM = -2, /* device or host allocation failed, or caller arena too small */
  LA_ECUDA = -3,  /* a CUDA runtime call failed; message in la_last_error */
  LA_ESTATE = -4, /* call not valid in the context's current configuration */
  LA_ETOOBIG = -5, /* size exceeds a fixed capacity (la_replica_means_static) */
  LA_EBOUNDS = -6  /* checked build only: a kernel computed an address outside its ranges (skipped, reported) */
};

enum { LA_F32 = 0, LA_BF16 = 1 };               /* gradient dtype */
enum { LA_FUSE_NONE = 0, LA_FUSE_STEP_SYNC = 1, /* la_run: step t'=H and its sync in one pass */
       LA_FUSE_SYNC_STEP = 2,                   /* la_run: sync folded into the following step */
       LA_FUSE_PERIOD = 3,                      /* la_run: up to 8 consecutive local steps (and the sync
                                                   that closes the period) in one pass over HBM; for the
                                                   generated gradients, whose noise lives in registers */
       LA_FUSE_MEAN_ONCE = 4 };                 /* la_run: a synchronisation makes all replicas equal, so its
                                                   result is stored once: the step t'=H writes only the sums of
                                                   its y, A^2 over the workers (into replica 0's rows) and the
                                                   step t'=1 that follows reads that one copy; per period one
                                                   write and one read of W-1 replicas fewer than LA_FUSE_STEP_SYNC.
                                                   la_run (generated gradients) and la_step_grads (supplied
                                                   ones), Local AdaAlter, H >= 2 (otherwise it behaves as
                                                   LA_FUSE_STEP_SYNC).  Between the two steps, also
                                                   across calls, the means are pending; every call that looks
                                                   at or changes the state completes them first. */
enum { LA_RULE_ADAALTER = 0,  /* Algorithm 3, Local AdaAlter (default) */
       LA_RULE_LOCAL_SGD = 1, /* Algorithm 2: y = x - eta G, x averaged every H steps, no accumulator */
       LA_RULE_ADAGRAD = 2 }; /* Algorithm 1: gradients averaged every step, B^2 += G o G, updated B^2 divides */
#define LA_H_NEVER 0xFFFFFFFFu                  /* H = +infinity: never synchronise */
#define LA_MAX_WORKERS 64u                      /* every W up to 16, and 32 and 64, has kernels of its own;
                                                   other counts run kernels that take W at run time
                                                   (same results, the passes that average 10-25 % slower) */

/* Extended creation parameters.  Zero-initialise, then fill. */
typedef struct la_config {
  uint32_t K;            /* number of tensors (>= 1) */
  const uint64_t* sizes; /* host, K entries, each >= 1; tensors are packed back to back, N = sum */
  uint64_t j_base;       /* global index of coordinate 0 (multiple of 4); the noise of coordinate j
                            is keyed on j_base + j, so a job can be sharded by coordinate range */
  uint32_t W;            /* workers / replicas, 1..LA_MAX_WORKERS */
  uint32_t H;            /* synchronisation period (Algorithm 3), >= 1; LA_H_NEVER = never */
  float eta;             /* learning rate (finite) */
  float eps;             /* epsilon (> 0); the algorithm uses eps^2 */
  float b0sq;            /* b_0^2 >= 0, initial value of every accumulator (Algorithm 3, init) */
  void* dev_arena;       /* device; optional caller-owned state memory (256-byte aligned), or NULL */
  uint64_t arena_bytes;  /* size of dev_arena; must be >= la_arena_bytes() */
  void* stream;          /* a cudaStream_t, or NULL for the legacy default stream */
  int32_t device;        /* CUDA device ordinal, or -1 for the current device */
} la_config;

typedef struct la_stats {
  uint64_t launches_local;  /* K1: local step (gradient + update + accumulate), Algorithm 3 body */
  uint64_t launches_sync;   /* K2: stand-alone synchronisation */
  uint64_t launches_fused;  /* every pass that holds a step AND a synchronisation, or several steps */
  uint64_t launches_other;  /* fills, scatter/gather of state */
  double ms_local, ms_sync, ms_fused; /* device time per class; only while profiling is on */
  double bytes_local, bytes_sync, bytes_fused; /* algorithmic HBM bytes issued per class */
  /* the fused class split by kernel (exchange-fused steps of the by-worker path are in
   * launches_fused only) */
  uint64_t launches_step_sync; /* K3: step t'=H and its synchronisation */
  uint64_t launches_sync_step; /* K4: synchronisation folded into the step t'=1 that follows */
  uint64_t launches_period;    /* temporal blocking: several local steps (and the closing sync) */
  double ms_step_sync, ms_sync_step, ms_period;
  double bytes_step_sync, bytes_sync_step, bytes_period;
} la_stats;

/* ---- creation / destruction ------------------------------------------------
 * Algorithm 3, initialisation line: x_{i,0} = x_0, B^2_{i,0} = b_0^2 * 1.
 * la_create: one tensor of N coordinates, x_0 = 0, b_0^2 = 0, device memory
 * allocated (and later freed) by the library, current device, default stream. */
int la_create(la_ctx** out, uint64_t N, uint32_t W, float eta, float eps, uint32_t H);
int la_create_ex(la_ctx** out, const la_config* cfg);
/* Bytes of device memory a context with this configuration needs (state only). */
int la_arena_bytes(const la_config* cfg, uint64_t* bytes);
/* Frees library-owned memory only; a caller arena is left untouched.  NULL is allowed. */
void la_destroy(la_ctx* ctx);
/* Message of the last error; ctx may be NULL (then: last failed creation in this thread). */
const char* la_last_error(const la_ctx* ctx);

/* ---- configuration ---------------------------------------------------------
 * Re-initialise the state: every replica gets x0 (host, N floats; NULL = zeros), every
 * accumulator and the stale accumulator get b0sq; counters return to zero. */
int la_set_init(la_ctx* ctx, const float* x0_host, float b0sq);
/* Synthetic stochastic gradient (stands in for G_{i,t} = grad f(x_{i,t-1}; z_{i,t}) of
 * Algorithm 3): g = s_j * xi, xi ~ N(0,1) from a counter-based generator keyed on
 * (seed, worker, step, global coordinate).  s_host: N floats or NULL for s == 1. */
int la_set_grad_noise(la_ctx* ctx, uint64_t seed, const float* s_host);
/* Noisy diagonal quadratic f = 1/2 sum a_j (x_j - c_j)^2: g = a_j (x - c_j) + sigma * xi,
 * evaluated at the worker's own iterate.  a_host, c_host: N floats each. */
int la_set_grad_quadratic(la_ctx* ctx, uint64_t seed, const float* a_host, const float* c_host,
                          float sigma);
/* Deterministic gradient g = s_j on every worker and step (s_host NULL = 1); for closed-form tests. */
int la_set_grad_constant(la_ctx* ctx, const float* s_host);
/* LA_BF16: round every generated gradient to bfloat16 (nearest-even) and widen, in registers. */
int la_set_grad_dtype(la_ctx* ctx, int dtype);
/* Test switch: all workers draw worker 0's noise (then replicas stay bitwise equal). */
int la_set_identical_workers(la_ctx* ctx, int on);
/* Warm-up of Section 6.2: eta_t = eta * min(1, t / warm_up_steps); 0 switches it off. */
int la_set_warmup(la_ctx* ctx, uint32_t warm_up_steps);
/* Baseline update rules of the paper in the same sweep (LA_RULE_*): Local SGD (Algorithm 2) and
 * Distributed AdaGrad (Algorithm 1), for fp32 generated gradients and for supplied gradient
 * tables (la_local_step_grads, la_step_grads).  Only legal while t' == 0.
 * AdaGrad keeps ONE shared iterate (all workers see x_{t-1}); W only sets how many gradients are
 * averaged per step; la_read_state returns that iterate for any worker, la_sync is LA_ESTATE,
 * and n_sync counts one gradient exchange per iteration. */
int la_set_rule(la_ctx* ctx, int rule);
/* How la_run realises the synchronisation (LA_FUSE_*); results are bitwise the same. */
int la_set_fusion(la_ctx* ctx, int mode);
/* Tuning knob: the sweep kernels run as a grid-stride loop over at most
 * blocks_per_sm * (number of SMs) blocks of 256 threads; 0 restores the built-in
 * per-kernel defaults (16 per replica, between 32 and 96, for kernels that take a step, 768 for the
 * temporal-blocking kernel, unbounded for the pure sync). */
int la_set_launch_shape(la_ctx* ctx, int blocks_per_sm);
/* Launch-bound regime (small N, e.g. a 2 MB state where a step takes a few microseconds): let
 * la_run replay whole periods of H iterations from a captured CUDA graph instead of launching
 * every kernel.  The kernels then read the global step from a device-resident counter, so one
 * graph serves all periods; results are bitwise unchanged.  Needs a context on a non-default
 * stream (LA_ESTATE otherwise); allocates 8 bytes on first use; ignored while profiling, for the
 * AdaGrad rule, for LA_FUSE_SYNC_STEP, and for runs that start inside a period. */
int la_set_graph(la_ctx* ctx, int on);
/* Record CUDA events around every launch and accumulate device time per class. */
int la_set_profiling(la_ctx* ctx, int on);

/* ---- the hot path ------------------------------------------------------------
 * One iteration of Algorithm 3 WITHOUT its synchronisation branch, for every worker:
 * t += 1, t' += 1; G at the worker's own x; y = x - eta_t G / sqrt(B2stale + t' eps^2);
 * A^2 = B^2 + G o G; both committed locally. */
int la_local_step(la_ctx* ctx);
/* Same, with G_{i,t} supplied by the caller: device pointer to [W][N] gradients, worker-major,
 * dtype LA_F32 (4 bytes) or LA_BF16 (2 bytes, widened exactly).  16-byte aligned. Not retained
 * beyond the kernel; the caller must keep it alive until the stream reaches that point. */
int la_local_step_grads(la_ctx* ctx, const void* g_dev, int dtype);
/* One COMPLETE iteration of Algorithm 3 with caller-supplied gradients (same table as above):
 * the local step and, when it makes t' reach H, the synchronisation branch — in the same pass
 * over memory unless the fusion mode is LA_FUSE_NONE.  This is the call a trainer makes once per
 * optimizer step after back-propagation. */
int la_step_grads(la_ctx* ctx, const void* g_dev, int dtype);
/* Synchronisation branch of Algorithm 3: x and B^2 of every worker are replaced by the means
 * over workers; the mean B^2 becomes the stale denominator; t' = 0; n_sync += 1.  Legal at any
 * time (outside la_run it need not fall on a multiple of H). */
int la_sync(la_ctx* ctx);
/* T iterations of Algorithm 3: repeat { local step; if t' == H: synchronise }.  May use fused
 * kernels; the state afterwards is bitwise that of the unfused sequence. */
int la_run(la_ctx* ctx, uint64_t T);

/* A whole job from and to host memory in one call, pipelined: equivalent to
 *   la_set_init(x0_host, b0sq as last set); the la_set_grad_* upload of the arrays given here;
 *   la_run(T); la_read_state(worker, x_host, b2_host, bs_host)
 * with the same bits in the outputs, in the device state and in the counters afterwards, but the
 * coordinates are cut into `chunks` ranges (0 = 16) and the upload of one range, the T iterations
 * of the previous one and the download of the one before overlap on three streams.  This is legal
 * because Algorithm 3 has only coordinate-wise operations and a per-coordinate mean over workers.
 * Host buffers hold N floats each and should be pinned (page-locked) for the copies to overlap.
 *   x0_host              initial iterate, or NULL for zeros
 *   a_host, c_host       quadratic gradient source: both or neither (NULL keeps the arrays on the device)
 *   s_host               scale array of the noise / constant sources, or NULL (keeps what is there)
 *   worker               whose x and B^2 are read back
 *   x_host, b2_host, bs_host   outputs, any may be NULL
 * The gradient source, its seed and sigma, the rule, the fusion mode and H are those of the
 * context.  Returns after the outputs are complete.  Two copy streams and 2 * chunks events are
 * created on the first call and live until la_destroy. */
typedef struct la_stream_io {
  const float* x0_host;
  const float* a_host;
  const float* c_host;
  const float* s_host;
  uint32_t worker;
  float* x_host;
  float* b2_host;
  float* bs_host;
} la_stream_io;
int la_run_streamed(la_ctx* ctx, uint64_t T, const la_stream_io* io, uint32_t chunks);

/* ---- state access (synchronises the stream) ------------------------------------
 * Copy worker `worker`'s x and B^2 and the shared stale accumulator to host buffers of N floats
 * each, in packed tensor order.  Any pointer may be NULL. */
int la_read_state(la_ctx* ctx, uint32_t worker, float* x_host, float* b2_host, float* bs_host);
/* The reverse (checkpoint restore).  Any pointer may be NULL. */
int la_write_state(la_ctx* ctx, uint32_t worker, const float* x_host, const float* b2_host,
                   const float* bs_host);
/* Read coordinates [j0, j0+n) only. */
int la_read_range(la_ctx* ctx, uint32_t worker, uint64_t j0, uint64_t n, float* x_host,
                  float* b2_host, float* bs_host);
/* Offset (in coordinates) and size of tensor k inside the packed vector. */
int la_tensor_range(const la_ctx* ctx, uint32_t k, uint64_t* offset, uint64_t* size);
/* t = local steps since creation, t_prime = local steps since the last synchronisation,
 * n_sync = synchronisations so far.  (Algorithm 3's t' of the NEXT step is t_prime + 1.) */
int la_get_counters(const la_ctx* ctx, uint64_t* t, uint32_t* t_prime, uint64_t* n_sync);
int la_set_counters(la_ctx* ctx, uint64_t t, uint32_t t_prime, uint64_t n_sync);
/* Launch counts, algorithmic bytes and (when profiling) device milliseconds per kernel class.
 * reset != 0 clears the counters after reading. */
int la_get_stats(la_ctx* ctx, la_stats* out, int reset);

/* Diagnostics, off the hot path (synchronises the stream; its first call allocates 16 bytes of
 * device memory).  With x-bar the mean iterate over workers (the auxiliary sequence of Section 5):
 *   objective      = 1/2 sum_j a_j (x-bar_j - c_j)^2, the noisy-quadratic objective at x-bar
 *                    (NaN unless the quadratic gradient source is set)
 *   replica_spread = (1/W) sum_i ||x_i - x-bar||^2, the drift of the replicas since the last
 *                    synchronisation (the quantity Appendix A bounds through H); 0 right after a sync
 * Accumulated in double.  Either pointer may be NULL. */
int la_diagnostics(la_ctx* ctx, double* objective, double* replica_spread);

/* ---- sharding BY WORKER across GPUs (one process per GPU) -----------------------------------
 * The layout of the paper: the workers of Algorithm 3 sit on different devices and exchange x
 * and B^2 every H steps (Section 4.2).  A rank holds W (local) replicas out of W_total.
 * The synchronisation is three enqueued phases around a library-owned exchange buffer
 * [2][stride] (sums of x, sums of B^2); the HOST orders them (la_stream_sync + a barrier across
 * ranks between phases); no kernel ever waits for another rank:
 *   la_comm_export   buffer <- adjacent-pair tree sum over the local replicas
 *   la_comm_combine  this rank's coordinate slice: adjacent-pair tree over all ranks' buffers in
 *                    rank order (plain peer loads), total stored into EVERY rank's buffer
 *                    (alternatively the caller all-reduces the buffer itself, e.g. with NCCL)
 *   la_comm_import   x, B^2 of every local replica <- total / W_total; stale <- mean B^2;
 *                    t' = 0; n_sync += 1
 * With W a power of two the result equals the single-GPU la_sync over W_total replicas bit for
 * bit (a caller-side all-reduce gives the same means up to its summation order).  Local
 * AdaAlter rule only. */
/* Global index of local replica 0 and the total worker count: the noise of local replica i is
 * that of worker worker_base + i.  W_total = 0 returns to the unsharded numbering. */
int la_set_worker_range(la_ctx* ctx, uint32_t worker_base, uint32_t W_total);
/* Allocate the exchange buffer (freed by la_destroy) and fix this context's rank.  If no worker
 * range was set: worker_base = rank * W, W_total = world * W.  With world > 1 the local worker
 * count W must be a power of two (LA_EINVAL otherwise): only then is "local tree, then tree over
 * ranks" the adjacent-pair tree over all workers. */
int la_comm_create(la_ctx* ctx, uint32_t rank, uint32_t world);
/* Device pointer and size of the exchange buffer (2 * stride floats). */
int la_comm_buffer(la_ctx* ctx, void** dev_ptr, uint64_t* bytes);
/* 64-byte CUDA IPC handle of the exchange buffer, to be sent to the other ranks (host buffer). */
int la_comm_ipc_handle(la_ctx* ctx, void* handle64_host);
/* Attach rank peer_rank's exchange buffer: from its IPC handle (another process), or as a raw
 * device pointer that is already valid here (same process).  Mappings are closed by la_destroy. */
int la_comm_open_peer(la_ctx* ctx, uint32_t peer_rank, const void* handle64_host);
int la_comm_set_peer(la_ctx* ctx, uint32_t peer_rank, void* dev_ptr);
int la_comm_export(la_ctx* ctx);
int la_comm_combine(la_ctx* ctx);
int la_comm_import(la_ctx* ctx);
/* The local steps next to a synchronisation, fused with the exchange, so that the
 * synchronisation costs no pass over the replicas of its own:
 *   la_comm_step_export        the local step of Algorithm 3 (generated gradients) that completes a
 *                              period; its y and A^2 are not stored (the means will replace them),
 *                              only their tree sums go to the exchange buffer.  t += 1, t' += 1.
 *                              Until the import the replicas hold the PREVIOUS step's values.
 *   la_comm_step_grads_export  the same with caller-supplied gradients (table as for
 *                              la_local_step_grads)
 *   la_comm_import_step        la_comm_import and the first local step of the next period in one
 *                              pass: every replica starts from total / W_total.  n_sync += 1,
 *                              t += 1, t' = 1.  (With H = 1 use la_comm_import instead.)
 * Sequence: step_export, exchange (la_comm_combine between barriers, or an all-reduce of the
 * buffer), then import_step or import.  Results are bitwise those of the unfused calls. */
int la_comm_step_export(la_ctx* ctx);
int la_comm_step_grads_export(la_ctx* ctx, const void* g_dev, int dtype);
int la_comm_import_step(la_ctx* ctx);
/* la_comm_import_step with caller-supplied gradients for the step t' = 1 (table as for
 * la_local_step_grads): together with la_comm_step_grads_export a trainer's synchronisation
 * costs no pass over the replicas of its own. */
int la_comm_import_step_grads(la_ctx* ctx, const void* g_dev, int dtype);
/* Verification aid for the synthetic gradient source (not part of the paper's method): the two
 * building blocks of the normal draw, exactly as the sweep kernels evaluate them, over their whole
 * 24-bit domains, so that they can be compared element by element with another implementation:
 *   radius_dev[k-1] = sqrt(-2 ln(k 2^-24)), k = 1..2^24
 *   cos_dev[q], sin_dev[q] = cos, sin(2 pi q 2^-24), q = 0..2^24-1
 * Each pointer is device memory for 2^24 floats, or NULL to skip that table.  Enqueued on
 * `stream` (a cudaStream_t, NULL = default) of the current device; needs no context. */
int la_noise_tables(float* radius_dev, float* cos_dev, float* sin_dev, void* stream);
/* Block until the context's stream is idle. */
int la_stream_sync(la_ctx* ctx);

/* ---- checked build ----------------------------------------------------------------------------
 * (No counterpart in the paper: a development aid.)  liblocal_adaalter_debug.so is the same
 * library compiled with -DLA_DEBUG.  Its kernels test every global-memory address they form
 * against the byte ranges the pass may touch (state arena, caller's gradient table, exchange
 * buffer) and the running row pointers against base + (replica * stride + coordinate) * 4.  An
 * offending access is skipped (a load yields 0) and counted; nothing traps or asserts.  The next
 * synchronising call (la_stream_sync, la_read_state / la_read_range, la_get_stats) then returns
 * LA_EBOUNDS with the first offending address in la_last_error, and clears the count.  The
 * arithmetic is unchanged (results stay bitwise equal to the normal library); it is slower and is
 * never the library that is timed.  The kernel that combines the ranks' exchange buffers
 * (la_comm_combine) is not range-checked.
 * la_debug_build: 1 in the checked library, 0 in the normal one.
 * la_debug_narrow: test knob of the checked library (LA_ESTATE in the normal one): the kernels
 * treat the last `bytes` bytes of the state arena as foreign, so that in-bounds accesses there are
 * reported and skipped — a way to see the report without forming a bad address.  0 restores. */
int la_debug_build(void);
int la_debug_narrow(la_ctx* ctx, uint64_t bytes);

/* ---- for callers that must not allocate ------------------------------------------------------
 * (The paper has no counterpart: this is a deployment variant of the replica average that
 * la_comm_export / la_comm_import compute.)
 * Who needs it: programs that gave the whole GPU to their own allocator at start-up and have
 * nothing left for cudaMalloc (the caller-arena mode of la_create_ex is for them), and services
 * that ban cudaMalloc/cudaFree once running because both stall the device.  This call makes no
 * allocation of any kind: its intermediate sums live in a fixed array inside the library image,
 * 2 * LA_STATIC_SCRATCH_MAX_COORDS floats (8 MiB) on every GPU that loads the library, until
 * the process exits.
 *   x_dev, b2_dev    device, [W][stride] floats, 16-byte aligned: the W replicas (read only)
 *   n, stride        coordinates, and floats between replicas (n <= stride, stride % 4 == 0,
 *                    stride <= LA_STATIC_SCRATCH_MAX_COORDS, else LA_ETOOBIG)
 *   x_mean_dev,      device, n floats each: adjacent-pair tree sum over the replicas divided
 *   b2_mean_dev      by (float)W — the same bits la_sync would put into every replica
 *   stream           a cudaStream_t (NULL = default); the work is only enqueued
 * The first call on a device looks up the array's device address (cudaGetSymbolAddress) with
 * that device current; make that first call outside any stream capture.  Under CUDA's default
 * lazy module loading that first call is also when the driver sets the 8 MiB aside on that
 * device (not when the library is loaded), so make it during start-up, before your own
 * allocator takes what is left of the GPU, or run with CUDA_MODULE_LOADING=EAGER.  If it fails
 * the call returns LA_ECUDA, leaves no sticky CUDA error behind and may simply be repeated.  All calls share the
 * one array: it is fully rewritten for [0, n) by each call (nothing needs to start at zero, and
 * it keeps the last call's sums afterwards), so two calls that overlap on the GPU — different
 * streams, or different threads — race; run them in stream order. */
#define LA_STATIC_SCRATCH_MAX_COORDS 1048576u
int la_replica_means_static(const float* x_dev, const float* b2_dev, uint32_t W, uint64_t n, uint64_t stride,
                            float* x_mean_dev, float* b2_mean_dev, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* LOCAL_ADAALTER_H_ */
