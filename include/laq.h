/*
 * laq.h -- C ABI of the B200 (sm_100a) LAQ library.
 *
 * LAQ = Lazily Aggregated Quantized gradients (Sun, Chen, Giannakis, Yang, NeurIPS 2019).
 * The library runs Algorithm 2 of the paper for M workers simulated on ONE GPU.  One iteration is
 *   1. every worker's local gradient g_m = grad f_m(theta^k)                       (Algorithm 2, worker step)
 *   2. the b-bit innovation quantizer: R_m = ||g_m - Q_m(theta_hat^{k-1})||_inf,
 *      tau = 1/(2^b-1), codes q = floor((g_m - Q_prev + R_m)/(2 tau R_m) + 1/2)     (Sec. 2.1, Eq. (5))
 *      and the innovation dQ_m = 2 tau R_m q - R_m 1                               (Sec. 2.1, Eq. (6))
 *   3. the squared norms ||dQ_m||^2 and ||eps_m||^2, eps_m = g_m - (Q_prev + dQ_m)  (Sec. 2.1, Sec. 2.2)
 *   4. the skip rule (7a) with the staleness clock (7b)                            (Sec. 2.2, Eq. (7a), (7b))
 *   5. grad^k = grad^{k-1} + sum_{uploading m} dQ_m ; theta^{k+1} = theta^k - alpha grad^k   (Eq. (4))
 * All five steps run in CUDA kernels; there is no CPU fallback.
 *
 * Conventions
 *   - Every pointer is marked HOST or DEVICE.  The caller owns every buffer, including the device
 *     workspace and the CUDA stream; the library owns only the laq_ctx it returns.
 *   - All device work is enqueued on the stream given to laq_init.
 *   - No function throws, aborts or traps the device.  Every fallible function returns a laq_status;
 *     laq_last_error() gives a text for the most recent failure on that context.
 *   - Conditions detected on the device freeze the state at the iteration where they occurred and are
 *     reported by the next call that synchronises (laq_step with a trace, laq_get_state, laq_get_worker,
 *     laq_sync): a non-finite gradient or radius as LAQ_ENONFINITE, a bounded wait that ran out as
 *     LAQ_ETIMEOUT.  No kernel waits without a limit, and none traps.  laq_set_state clears the condition.
 *   - Floating point: theta, gradients and quantizer state are fp32; each quantizer operation is one
 *     IEEE round-to-nearest operation in the order  d = g - Q_prev ; R = max|d| ; s = (2 tau) R ;
 *     t = (d + R)/s + 1/2 (IEEE division) ; q = floor t ; dQ = s q - R (multiply, then subtract) ;
 *     Q_new = Q_prev + dQ ; eps = g - Q_new, with no fused multiply-add (kernels may reach q by a cheaper
 *     route where they can prove that it gives the same integer); codes, dQ, Q_new and eps are therefore
 *     reproducible bit for bit.  Squared norms are fp64 sums of exact fp32 products, except that the sweep over
 *     rows generated in the kernel (LAQ_MODEL_SYNTH) and over rows of 2^20 or more coordinates read from memory
 *     first sums runs of 32 products in fp32 (relative error of a run below 2^-19; of a whole row typically
 *     1e-9); the skip rule is evaluated in fp64.
 *   - Code stream of worker m (the paper's b p-bit part of the upload message): code i occupies bits
 *     [i b, (i+1) b) of the stream, bit j of the stream being bit (j mod 32) of 32-bit word floor(j / 32)
 *     (least significant first; for b = 3 a code may straddle two words).
 *   - Readings where the paper is silent: initial Q_m = 0, ||eps_hat_m||^2 = 0, grad^0 = 0, the D stored
 *     squared parameter differences start at 0, clocks start at t_bar + 1 (every worker uploads at
 *     k = 1); R_m = 0 yields q = 0, dQ = 0; ||theta^{k+1}-theta^k||^2 is taken as ||alpha grad^k||^2.
 */
#ifndef LAQ_B200_H
#define LAQ_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct laq_ctx laq_ctx;

typedef enum {
  LAQ_OK = 0,
  LAQ_EINVAL = 1,      /* bad argument or unsupported configuration */
  LAQ_EWORKSPACE = 2,  /* workspace pointer null, misaligned (256 B) or too small */
  LAQ_ECUDA = 3,       /* a CUDA runtime call failed */
  LAQ_ENONFINITE = 4,  /* a gradient or radius was inf/nan; state frozen at that iteration */
  LAQ_ESTATE = 5,      /* call not valid in the context's current state (e.g. shards missing) */
  LAQ_ETIMEOUT = 6     /* a bounded wait inside a kernel (on an asynchronous copy or a tensor-core stage) ran out;
                          the kernel gave up, the state is frozen at that iteration, the CUDA context stays usable */
} laq_status;

/* Which f_m the workers hold (supplement, "Simulation details"; global loss f = (1/N) sum_m f_m,
 * every sample loss carries (lambda/2)||theta||^2, so worker m adds (N_m/N) lambda theta). */
typedef enum {
  LAQ_MODEL_LOGREG_BIN = 0, /* z = x.theta, loss softplus(z) - y z, y in {0,1}; p = n_features (<= 256) */
  LAQ_MODEL_SOFTMAX = 1,    /* softmax(theta x), theta [n_classes x n_features] row-major; p = C F */
  LAQ_MODEL_MLP2 = 2,       /* ReLU network F-H-C; theta = W1[H x F], b1[H], W2[C x H], b2[C];
                               the products X W1^T and dH^T X take bf16 operands, fp32 accumulation */
  LAQ_MODEL_SYNTH = 3,      /* no data: g_m^k[i] generated in the kernels from (seed, m, i, k), see below */
  LAQ_MODEL_EXTERNAL = 4    /* the caller supplies g (M x p) before every step with laq_set_gradients */
} laq_model;

/* LAQ_MODEL_SYNTH stream (fp32; coordinates in groups of four, group v = i / 4, e = i mod 4):
 *   fmix32(x): x ^= x>>16; x *= 0x85ebca6b; x ^= x>>13; x *= 0xc2b2ae35; x ^= x>>16
 *   key_m = fmix32(seed_lo ^ fmix32(seed_hi + 0x9e3779b9 (m+1)))
 *   h0 = fmix32((uint32) v ^ key_m);  h1 = h0 * 0x9e3779b1;  h1 ^= h1 >> 15
 *   for a word with bytes b0..b3 (b0 lowest): S = b0+b1+b2+b3-510, A = b0-b1+b2-b3
 *   z_0 = S(h0), z_1 = A(h0), z_2 = S(h1), z_3 = A(h1)
 *   cz = fp32(synth_sigma / sqrt(21845)), eta_m = fp32(synth_eta0 (m+1)/M)
 *   g_m^k[i] = fma(fl(k eta_m), z_{e xor 2}, z_e) * cz,  k = 1, 2, ...   (requires p < 2^32) */

enum {
  LAQ_FLAG_QUANT_OFF = 1u,  /* no quantizer: an upload carries the innovation g_m - Q_m(theta_hat^{k-1}) itself,
                               32 bits per coordinate, eps = 0 in (7a): the lazily aggregated gradient baseline
                               (LAG) of Sec. 4.  R is still reported; no codes are written (they stay zero) */
  LAQ_FLAG_TRIGGER_OFF = 2u,/* every worker uploads every iteration: Algorithm 1 (QGD); with LAQ_FLAG_QUANT_OFF
                               as well: gradient descent, Eq. (2) */
  LAQ_FLAG_SPARSE_X = 8u,   /* LAQ_MODEL_SOFTMAX only (2..10 classes, at most 896 features): laq_load_shards also
                               makes a compressed copy of the shard (its non-zeros by rows and by columns, in tiles
                               of 128 rows) and step 1 runs over the non-zeros only.  Same gradient up to the order
                               of the fp32 sums.  The copies may take as many entries (6 bytes each) as the shard has
                               elements; a denser shard makes laq_load_shards return LAQ_EWORKSPACE */
  LAQ_FLAG_STORE_G = 4u     /* LAQ_MODEL_SYNTH only: step 1 writes the M x p gradients of the iteration to the
                               workspace (as a gradient kernel does, Algorithm 2's worker step) and steps 2-5 read
                               them from memory instead of regenerating them; same values, same results */
};

typedef struct {
  int32_t model;            /* laq_model */
  int32_t M;                /* number of workers, 1..1024 */
  int64_t p;                /* dimension of theta, 1..2^32-1 (checked against the model shape) */
  const int64_t* N;         /* HOST, length M: samples per worker {N_m}; ignored for SYNTH / EXTERNAL */
  int32_t n_features;       /* F */
  int32_t n_classes;        /* C (SOFTMAX: 2..16, MLP2) */
  int32_t n_hidden;         /* H (MLP2) */
  float alpha;              /* step size */
  float lambda;             /* l2 regulariser */
  int32_t b;                /* bits per coordinate: 1, 2, 3, 4, 8 or 16 */
  int32_t D;                /* number of stored parameter differences, 1..64; the paper requires D <= t_bar */
  const float* xi;          /* HOST, length D: weights xi_1..xi_D of (7a), finite and >= 0; xi[0] pairs with the
                               newest difference */
  int32_t tbar;             /* staleness bound of (7b), -1 .. 2^31 - 3 (with -1 the clock test always fails:
                               nobody ever skips).  The paper asks for D <= t_bar; smaller values are accepted,
                               the rule (7a) then looks further back than a copy can be stale */
  int32_t clock_mode;       /* 0: Algorithm 2 as printed, skip allowed while t_m <= t_bar;
                               1: strict, skip needs t_m + 2 <= t_bar (t_bar = 1 never skips) */
  uint32_t flags;           /* LAQ_FLAG_* */
  uint64_t seed;            /* SYNTH stream and minibatch windows */
  float synth_sigma;        /* SYNTH only */
  float synth_eta0;         /* SYNTH only */
  int32_t trace_capacity;   /* per-iteration records kept on the device for laq_step's trace (0 = none) */
  int32_t batch;            /* 0: full local gradients.  > 0 (models with samples): the minibatch variant of the
                               Sec. 4 stochastic tests.  At iteration k = 1, 2, .. worker m uses the B_m =
                               min(batch, N_m) samples (o + j) mod N_m, j < B_m, a cyclic window starting at
                               o = fmix32(fmix32(seed_lo + (uint32) k) ^ (seed_hi + 0x9e3779b9 (m+1))) mod N_m, and
                               g_m = (N_m / B_m)(1/N) sum_window grad l_i + (N_m/N) lambda theta; the reported loss
                               is the same estimate of f */
  int32_t world;            /* 0 or 1: all M workers live in this context.  > 1: the workers are spread over `world`
                               contexts (one per GPU), round robin: this context runs steps 1-4 for the workers
                               m = rank, rank + world, ... and holds their Q_m; every context holds theta, grad and
                               the stored differences, and applies every upload (the server's side of Fig. 2 is
                               replicated).  M, N and p keep their global meaning.  Needs the quantizer
                               (no LAQ_FLAG_QUANT_OFF) and M >= world; driven with laq_step_local,
                               laq_local_uploads, laq_apply_uploads instead of laq_step */
  int32_t rank;             /* 0 .. world-1 */
} laq_config;

/* Per-iteration report of laq_step.  All pointers HOST, each may be NULL; n = n_iters of that call.
 * Row j describes the j-th iteration of the call. */
typedef struct {
  uint8_t* skip;     /* [n][M]  1 = worker skipped the upload, 0 = uploaded */
  float* R;          /* [n][M]  radius R_m^k */
  double* n_dq;      /* [n][M]  ||dQ_m^k||^2 */
  double* n_eps;     /* [n][M]  ||eps_m^k||^2 */
  double* rhs;       /* [n][M]  right-hand side of (7a) */
  double* dtheta2;   /* [n]     ||theta^{k+1}-theta^k||^2 */
  double* loss;      /* [n]     f(theta^k) (model workloads; 0 for SYNTH / EXTERNAL) */
  int32_t* uploads;  /* [n]     |M^k| */
} laq_trace;

/* Explicit state for laq_get_state / laq_set_state.  All pointers HOST, each may be NULL (skipped).
 * Together with the configuration and the shards, the fields marked (S) determine every later
 * iteration; the others are read-only views of the last iteration. */
typedef struct {
  float* theta;       /* (S) [p]        theta^k */
  float* agg;         /* (S) [p]        grad^{k-1}, the server's lazily aggregated gradient */
  float* qprev;       /* (S) [M][p]     Q_m(theta_hat_m^{k-1}); per-worker arrays of this struct have one row per LOCAL
                                        worker when laq_config.world > 1 */
  double* n_eps_hat;  /* (S) [M]        ||eps_hat_m||^2, the error at worker m's last upload */
  int32_t* clock;     /* (S) [M]        t_m */
  double* ring;       /* (S) [D]        stored squared differences, newest first */
  int64_t* counters;  /* (S) [3]        iterations done, uploads so far, bits so far (uploads x (32 + b p)) */
  float* g;           /*     [M][p]     last local gradients (SYNTH: only with LAQ_FLAG_STORE_G) */
  uint32_t* codes;    /*     [M][W]     last code streams, W = ceil(p b / 32) words per worker */
  float* R;           /*     [M]        last radii */
  double* n_dq;       /*     [M]        last ||dQ_m||^2 */
  double* n_eps;      /*     [M]        last ||eps_m||^2 */
  uint8_t* skip;      /*     [M]        last skip mask */
} laq_state;

/* Device memory the caller must provide for this configuration (bytes).  0 if the configuration is
 * invalid.  Holds theta, grad, Q_prev, g, code streams, the resident shards and kernel scratch. */
size_t laq_workspace_bytes(const laq_config* cfg /* HOST */);

/* Create a context (Algorithm 2, "Initialize").  d_workspace: DEVICE, 256-byte aligned, at least
 * laq_workspace_bytes(cfg) bytes, owned by the caller and kept alive until laq_destroy.
 * theta0: HOST, length p, or NULL for zeros.  cuda_stream: a cudaStream_t (NULL = default stream).
 * The configuration (including N and xi) is copied.  Returns LAQ_EINVAL / LAQ_EWORKSPACE / LAQ_ECUDA. */
laq_status laq_init(laq_ctx** out, const laq_config* cfg, void* d_workspace, size_t workspace_bytes,
                    const float* theta0, void* cuda_stream);

/* Make worker m's shard resident (Eq. (1): the N_m samples of f_m).  X: [N_m][n_features] fp32
 * row-major, y: [N_m] int32 labels (0/1 for LOGREG_BIN, 0..C-1 otherwise); both HOST if
 * on_device == 0, DEVICE otherwise.  The data is copied into the workspace.  N_m must equal cfg.N[m]. */
laq_status laq_load_shards(laq_ctx* ctx, int32_t m, const float* X, const int32_t* y, int64_t N_m,
                           int32_t on_device);

/* LAQ_MODEL_EXTERNAL: provide the M x p local gradients of the next iteration (row m = g_m).
 * HOST if on_device == 0, DEVICE otherwise; copied into the workspace. */
laq_status laq_set_gradients(laq_ctx* ctx, const float* g, int32_t on_device);

/* Run n_iters iterations of Algorithm 2 (for EXTERNAL: n_iters must be 1).  With trace == NULL the
 * call only enqueues work on the stream and returns.  With a trace (n_iters <= trace_capacity) it
 * synchronises once at the end, fills the HOST arrays and reports device-detected errors.
 * Calls of four or more iterations replay the iteration's kernels as CUDA graphs (captured once per context on
 * a stream of the library's own, launched into the context's stream; plain launches if capture is not possible,
 * while per-stage timing is on, or after laq_tune(ctx, "graphs", 0)). */
laq_status laq_step(laq_ctx* ctx, int32_t n_iters, const laq_trace* trace);

/* One iteration in two halves, for workers spread over several contexts (laq_config.world > 1; also valid for
 * world <= 1, where the two halves together equal laq_step(ctx, 1, NULL) bit for bit).
 *
 * laq_step_local enqueues steps 1-4 of Algorithm 2 for this context's workers: local gradients, quantizer, norms,
 * skip rule and clocks.  Every uploading worker's message (Eq. (6) and the text after it: the radius, 32 bits, and
 * the b p-bit code stream) is then ready in this context: the radius through laq_local_uploads, the code stream in
 * the workspace at byte offset  codes_offset_bytes + l code_row_bytes  for the l-th local worker (laq_query).
 *
 * laq_local_uploads synchronises and returns the local uploaders of the iteration in flight: *n of them, their
 * GLOBAL worker indices m[0..*n) in ascending order and radii R[0..*n).  m, R: HOST, room for the local worker count.
 *
 * laq_apply_uploads enqueues step 5, the server's update, with ALL uploads of the iteration, local and remote:
 * n uploaders, global indices m[] ascending, radii R[] (HOST).  Before the call the caller must have put the code
 * stream of every REMOTE uploader m into this context's mailbox, at byte offset
 * mailbox_offset_bytes + m code_row_bytes of the workspace (laq_query), ordered before this call on the context's
 * stream.  Uploads are applied in ascending worker order, as laq_step does; Q_m is updated for local uploaders.
 * The upload and bit counters count all n uploads, so they agree on every context. */
laq_status laq_step_local(laq_ctx* ctx);
laq_status laq_local_uploads(laq_ctx* ctx, int32_t* n, int32_t* m, float* R);
laq_status laq_apply_uploads(laq_ctx* ctx, int32_t n, const int32_t* m, const float* R);

/* Wait for the stream and report device-detected errors. */
laq_status laq_sync(laq_ctx* ctx);

/* Copy state to HOST buffers (synchronises).  The buffers are filled even when the state is frozen; the call
 * then returns LAQ_ENONFINITE or LAQ_ETIMEOUT. */
laq_status laq_get_state(laq_ctx* ctx, const laq_state* out);

/* One worker's rows after the last iteration (synchronises): qprev [p] = Q_m(theta_hat_m), g [p] = its
 * last local gradient (not for SYNTH), and the upload message of Eq. (6): the radius R (one float) and the
 * code stream codes [ceil(p b / 32)] words.  All HOST, each may be NULL. */
laq_status laq_get_worker(laq_ctx* ctx, int32_t m, float* qprev, float* g, uint32_t* codes, float* R);

/* Overwrite the (S) fields that are non-NULL (resume from a saved state; synchronises). */
laq_status laq_set_state(laq_ctx* ctx, const laq_state* in);

/* Number of kernels the library has launched on this context so far. */
int64_t laq_kernel_launches(const laq_ctx* ctx);

/* Launch-shape override for measurement sweeps: key "sweep_threads", "sweep_blocks_per_sm",
 * "agg_threads", "agg_blocks_per_sm", "grad_blocks_per_worker", and "graphs" (0: laq_step uses plain launches
 * only; 1, the default: graph replay).  Values outside the documented limits return LAQ_EINVAL and change
 * nothing.
 * Key "starve_copies" (0 or 1, default 0) exists for testing the LAQ_ETIMEOUT path without disturbing the device:
 * while it is 1, one warp of the quantize sweep over generated rows (LAQ_MODEL_SYNTH), and the loader of one block
 * of the network's tensor-core kernels (LAQ_MODEL_MLP2), issue none of their asynchronous copies and poll with a
 * short limit, so their consumers' waits run out with nothing in flight. */
laq_status laq_tune(laq_ctx* ctx, const char* key, int32_t value);

/* Read-only facts about the launch plan, for tests and reports: key "sweep_blocks_per_worker", "sweep_threads",
 * "sweep_tile_groups" (16-byte groups per staged tile of the quantize sweep over generated or stored rows),
 * "aggregate_blocks", "grad_blocks_per_worker", "local_workers" (workers whose steps 1-4 run in this context),
 * "codes_offset_bytes", "code_row_bytes", "mailbox_offset_bytes" (see laq_step_local).  Unknown keys return
 * LAQ_EINVAL. */
laq_status laq_query(const laq_ctx* ctx, const char* key, int64_t* value /* HOST */);

/* Per-kernel device timing for measurement.  While enabled, laq_step brackets every stage of an iteration
 * with CUDA events on the context's stream (up to 512 iterations per call are recorded).
 * laq_kernel_times synchronises and returns, summed since the last call to it, the milliseconds and the
 * launch counts of the four stages: [0] local gradient, [1] radius, [2] quantize + norms + trigger,
 * [3] lazy aggregate + theta step.  ms and launches: HOST arrays of 4. */
laq_status laq_set_profiling(laq_ctx* ctx, int32_t enabled);
laq_status laq_kernel_times(laq_ctx* ctx, double* ms, int64_t* launches);

/* (The paper has no counterpart for this entry point; it exists for hosts that must not allocate.)
 * The quantizer of ONE worker -- radius, packed codes and the two squared norms, exactly as steps 2-3 of
 * laq_step compute them -- without a context and without any allocation: no cudaMalloc/cudaFree, no
 * workspace.  It is meant for callers that cannot allocate device memory themselves: a host program that
 * has given the whole GPU to its own memory pool, or a latency-critical loop in which allocation calls are
 * banned because they synchronise the device.  The kernels' reduction scratch (33 024 bytes: running
 * maximum, per-block partial sums, a ticket) is a __device__ array inside the library; every GPU that
 * loads the library holds it until the process exits.
 *   d_g, d_qprev : DEVICE, [p] fp32, the gradient and the stored quantized copy (inputs, unchanged)
 *   d_codes      : DEVICE, [ceil(p b / 32)] words, the code stream (output)
 *   d_R          : DEVICE, one float, the radius (output)
 *   d_norms      : DEVICE, two doubles, ||dQ||^2 and ||eps||^2 (output)
 *   errbuf       : HOST, optional buffer for an error text (errbuf_len bytes), may be NULL
 * Limits: b in {1, 2, 4, 8, 16}; 1 <= p <= 2^31, larger p is rejected with LAQ_EINVAL and a message.
 * The call is asynchronous on cuda_stream.  All calls on one GPU share the scratch, which still holds the
 * previous call's values (the call clears what must start at zero): calls whose kernels overlap on the same
 * GPU race with each other, so keep them on one stream or otherwise serialised.  The first call on each
 * device looks up the scratch's device address (and loads the module); make that call during start-up,
 * before any stream capture.  The device that holds the buffers must be the current device of the calling thread
 * (checked: LAQ_EINVAL otherwise).  The looked-up address is cached per device and does not survive a
 * cudaDeviceReset.  A non-finite input yields a non-finite *d_R, zero norms and untouched codes. */
laq_status laq_quantize_worker_static(const float* d_g, const float* d_qprev, int64_t p, int32_t b,
                                      uint32_t* d_codes, float* d_R, double* d_norms, void* cuda_stream,
                                      char* errbuf, size_t errbuf_len);

/* Text of the last failure on this context ("" if none).  Valid until the next call on ctx. */
const char* laq_last_error(const laq_ctx* ctx);

/* Free the context (not the workspace).  Waits for the stream first.  NULL is allowed. */
void laq_destroy(laq_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* LAQ_B200_H */
