// Host side of the C ABI declared in laq.h: configuration checks, carving of the caller's device
// workspace, and the per-iteration launch plan of Algorithm 2.  No arithmetic of the method runs
// on the host; every step of the iteration is a kernel (laq_sweeps.cu, laq_grad_*.cu).
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "laq_internal.cuh"

using namespace laq;

struct laq_ctx {
  laq_config cfg;                      // cfg.M and cfg.N describe the LOCAL workers (all of them unless world > 1)
  int world = 1, rank = 0, M_total = 0;
  int32_t* d_up_m_in = nullptr;        // device staging of laq_apply_uploads' arguments
  float* d_up_R_in = nullptr;
  std::vector<int64_t> N;
  std::vector<float> xi;
  Params P;
  LaunchShape ls;
  cudaStream_t st = nullptr;
  int64_t launches = 0;
  std::string err;
  std::vector<char> shard_loaded;
  bool ext_g_set = false;
  int gbpw = 1, gbpw_cap = 1;
  char* ws = nullptr;
  size_t ws_bytes = 0;
  std::vector<const float*> Xptr;
  std::vector<const int32_t*> yptr;
  std::vector<void*> sp_region;        // LAQ_FLAG_SPARSE_X: where each worker's compressed copies go
  MlpPlan mlp;
  // optional per-stage timing
  bool profiling = false;
  std::vector<cudaEvent_t> ev;        // kProfIters x 5 events
  int ev_used = 0;                    // iterations recorded and not yet read
  double stage_ms[4] = {0, 0, 0, 0};
  int64_t stage_launches[4] = {0, 0, 0, 0};
  // the kernels of one iteration (and of kGraphIters iterations) as executable graphs, replayed by laq_step
  bool graphs_enabled = true, graphs_failed = false;
  cudaStream_t cap_stream = nullptr;   // capture happens here, never on the caller's stream
  cudaGraphExec_t graph_one = nullptr, graph_many = nullptr;
  int64_t launches_per_iter = 0;
  std::vector<char> trace_host;        // short per-iteration reports land here in one copy
};

namespace {

constexpr size_t kAlign = 256;
constexpr int kMaxAggBlocks = kNumSMs * 32;
constexpr int kGradBlocksCap = 64;
constexpr int kProfIters = 512;
constexpr size_t kTraceSpanMax = 64 * 1024;   // reports up to this size come back in one copy

size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

bool valid_b(int b) { return b == 1 || b == 2 || b == 3 || b == 4 || b == 8 || b == 16; }

long long model_p(const laq_config& c) {
  switch (c.model) {
    case LAQ_MODEL_LOGREG_BIN: return c.n_features;
    case LAQ_MODEL_SOFTMAX: return (long long)c.n_classes * c.n_features;
    case LAQ_MODEL_MLP2:
      return (long long)c.n_hidden * c.n_features + c.n_hidden + (long long)c.n_classes * c.n_hidden + c.n_classes;
    default: return c.p;
  }
}

const char* check_config(const laq_config* c) {
  if (!c) return "config is null";
  if (c->model < 0 || c->model > LAQ_MODEL_EXTERNAL) return "unknown model";
  if (c->M < 1 || c->M > kMaxWorkers) return "M must be in 1..1024";
  if (c->p < 1 || c->p >= (1ll << 32)) return "p must be in 1..2^32-1";
  if (!valid_b(c->b)) return "b must be 1, 2, 3, 4, 8 or 16";
  if (c->D < 1 || c->D > kMaxD) return "D must be in 1..64";
  if (!c->xi) return "xi is null";
  for (int d = 0; d < c->D; ++d)
    if (!std::isfinite(c->xi[d]) || c->xi[d] < 0.f) return "every xi_d must be finite and >= 0";
  if (c->tbar < -1 || c->tbar > 0x7fffffff - 2) return "tbar must be in -1..2^31-3";
  if (!(c->alpha > 0.f) || !std::isfinite(c->alpha)) return "alpha must be positive and finite";
  if (c->clock_mode != 0 && c->clock_mode != 1) return "clock_mode must be 0 or 1";
  if (c->trace_capacity < 0) return "trace_capacity must be >= 0";
  if (c->flags & ~(uint32_t)(LAQ_FLAG_TRIGGER_OFF | LAQ_FLAG_QUANT_OFF | LAQ_FLAG_STORE_G | LAQ_FLAG_SPARSE_X)) return "unknown flag";
  if ((c->flags & LAQ_FLAG_SPARSE_X) && (c->model != LAQ_MODEL_SOFTMAX || !sparse_shape_ok(c->n_features, c->n_classes)))
    return "LAQ_FLAG_SPARSE_X needs LAQ_MODEL_SOFTMAX with 2..10 classes and at most 896 features";
  if ((c->flags & LAQ_FLAG_STORE_G) && c->model != LAQ_MODEL_SYNTH) return "LAQ_FLAG_STORE_G needs LAQ_MODEL_SYNTH";
  if (c->batch < 0) return "batch must be >= 0";
  if (c->world < 0 || c->world > kMaxWorkers) return "world must be in 0..1024";
  if (c->world > 1) {
    if (c->rank < 0 || c->rank >= c->world) return "rank must be in 0..world-1";
    if (c->M < c->world) return "world > 1 needs at least one worker per context (M >= world)";
    if (c->flags & LAQ_FLAG_QUANT_OFF) return "world > 1 needs the quantizer (the upload is the coded message)";
  } else if (c->rank != 0) {
    return "rank must be 0 unless world > 1";
  }
  if (c->batch > 0 && (c->model == LAQ_MODEL_SYNTH || c->model == LAQ_MODEL_EXTERNAL))
    return "batch > 0 needs a model with samples";
  const bool data = c->model == LAQ_MODEL_LOGREG_BIN || c->model == LAQ_MODEL_SOFTMAX || c->model == LAQ_MODEL_MLP2;
  if (data) {
    if (!c->N) return "N is null";
    for (int m = 0; m < c->M; ++m)
      if (c->N[m] < 1 || c->N[m] > (1ll << 31) - 1) return "every N_m must be in 1..2^31-1";
    if (c->n_features < 1) return "n_features must be positive";
    if (model_p(*c) != c->p) return "p does not match the model shape";
    if (!std::isfinite(c->lambda) || c->lambda < 0.f) return "lambda must be finite and >= 0";
  }
  if (c->model == LAQ_MODEL_LOGREG_BIN && c->n_features > 256) return "LOGREG_BIN supports n_features <= 256";
  if (c->model == LAQ_MODEL_SOFTMAX) {
    if (!softmax_classes_supported(c->n_classes)) return "SOFTMAX supports 2..16 classes";
    if (c->n_features > 1024) return "SOFTMAX supports n_features <= 1024";
  }
  if (c->model == LAQ_MODEL_MLP2) {
    const char* e = mlp_check_shape(c->n_features, c->n_hidden, c->n_classes);
    if (e) return e;
  }
  if (c->model == LAQ_MODEL_SYNTH) {
    if (!std::isfinite(c->synth_sigma) || !std::isfinite(c->synth_eta0)) return "synth parameters must be finite";
  }
  return nullptr;
}

// The workers of this context: all M, or (world > 1) the global workers rank, rank + world, ...
int local_workers(const laq_config& c) {
  return c.world > 1 ? (c.M - c.rank + c.world - 1) / c.world : c.M;
}

// The configuration as the rest of this file uses it: M and N describe the local workers.  Nl receives the local
// shard sizes; *n_total the number of samples of ALL workers (the 1/N of the global loss).
laq_config localize(const laq_config& c, std::vector<int64_t>& Nl, long long* n_total) {
  laq_config l = c;
  const bool data = c.model == LAQ_MODEL_LOGREG_BIN || c.model == LAQ_MODEL_SOFTMAX || c.model == LAQ_MODEL_MLP2;
  const int Ml = local_workers(c), stride = c.world > 1 ? c.world : 1, first = c.world > 1 ? c.rank : 0;
  Nl.assign(Ml, 0);
  long long tot = 0;
  if (data && c.N) {
    for (int m = 0; m < c.M; ++m) tot += c.N[m];
    for (int i = 0; i < Ml; ++i) Nl[i] = c.N[first + stride * i];
  }
  if (n_total) *n_total = tot;
  l.M = Ml;
  l.N = Nl.data();
  return l;
}

struct Plan {
  size_t total = 0;
  size_t mailbox = 0, up_q = 0, up_in_m = 0, up_in_R = 0;
  size_t sc, theta, agg, qp, g, codes, Rbits, norms, n_epshat, clock, skip, up_m, up_R, up_s, ring, xi, loss_m,
      part_q, part_d, part_t, t_skip, t_R, t_ndq, t_neps, t_rhs, t_d2, t_loss, t_up, Xptr, yptr, Ndev, cnt_grad,
      gpart, lpart, state_end, mlp;
  std::vector<size_t> X, y, sp;
  size_t sp_desc = 0;
  long long ps, nv, cw;
  int gbpw_cap;
};

int default_gbpw(const laq_config& c) {
  // one wave of resident blocks (shared memory decides how many fit on an SM)
  int g = (grad_blocks_per_sm(c.model, c.n_features, c.n_classes) * kNumSMs) / c.M;
  if (g > kGradBlocksCap) g = kGradBlocksCap;
  return g < 1 ? 1 : g;
}

// c: the localized configuration; M_total: all workers (= c.M unless the workers are spread over contexts)
Plan make_plan(const laq_config& c, int M_total) {
  Plan pl;
  const size_t M = (size_t)c.M, Mt = (size_t)M_total;
  const bool spread = M_total != c.M;
  pl.ps = (c.p + 15) / 16 * 16;
  pl.nv = pl.ps / 4;
  pl.cw = ((pl.ps * c.b + 31) / 32 + 3) / 4 * 4;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    off = align_up(off + bytes);
    return o;
  };
  const size_t cap = (size_t)c.trace_capacity;
  const bool data = c.model == LAQ_MODEL_LOGREG_BIN || c.model == LAQ_MODEL_SOFTMAX || c.model == LAQ_MODEL_MLP2;
  pl.sc = take(sizeof(DevScalars));
  pl.theta = take(pl.ps * 4);
  pl.agg = take(pl.ps * 4);
  pl.qp = take(M * pl.ps * 4);
  pl.g = (c.model == LAQ_MODEL_SYNTH && !(c.flags & LAQ_FLAG_STORE_G)) ? off : take(M * pl.ps * 4);
  // local code rows, then (workers spread over contexts) one mailbox row per global worker for received messages
  pl.codes = take((M + (spread ? Mt : 0)) * pl.cw * 4);
  pl.mailbox = pl.codes + M * pl.cw * 4;
  pl.Rbits = take(2 * M * 4);
  pl.norms = take(3 * M * 8);
  pl.n_epshat = take(M * 8);
  pl.clock = take(M * 4);
  pl.skip = take(M);
  pl.up_m = take(Mt * 4);
  pl.up_q = take(Mt * 4);
  pl.up_R = take(Mt * 4);
  pl.up_s = take(Mt * 4);
  pl.up_in_m = take(Mt * 4);
  pl.up_in_R = take(Mt * 4);
  pl.ring = take((size_t)c.D * 8);
  pl.xi = take((size_t)c.D * 4);
  pl.loss_m = take(M * 8);
  pl.part_q = take(M * kMaxSweepBlocksPerWorker * 2 * 8);
  pl.part_d = take((size_t)kMaxAggBlocks * 8);
  pl.part_t = take((size_t)kMaxAggBlocks * 8);
  pl.t_skip = take(cap * M);
  pl.t_R = take(cap * M * 4);
  pl.t_ndq = take(cap * M * 8);
  pl.t_neps = take(cap * M * 8);
  pl.t_rhs = take(cap * M * 8);
  pl.t_d2 = take(cap * 8);
  pl.t_loss = take(cap * 8);
  pl.t_up = take(cap * 4);
  pl.Xptr = take(M * 8);
  pl.yptr = take(M * 8);
  pl.Ndev = take(M * 8);
  pl.cnt_grad = take(M * 4);
  pl.state_end = off;  // everything up to here is zero-filled by laq_init
  pl.gbpw_cap = 1;
  pl.gpart = pl.lpart = pl.mlp = off;
  if (data) {
    pl.gbpw_cap = kGradBlocksCap;
    if (c.model != LAQ_MODEL_MLP2) {
      pl.gpart = take(M * (size_t)pl.gbpw_cap * pl.ps * 4);
      pl.lpart = take(M * (size_t)pl.gbpw_cap * 8);
    } else {
      pl.mlp = take(mlp_scratch_bytes(c));
    }
    for (size_t m = 0; m < M; ++m) {
      pl.X.push_back(take((size_t)c.N[m] * c.n_features * 4));
      pl.y.push_back(take((size_t)c.N[m] * 4));
    }
    if (c.flags & LAQ_FLAG_SPARSE_X) {
      pl.sp_desc = take(M * sizeof(SparseShard));
      for (size_t m = 0; m < M; ++m) pl.sp.push_back(take(sparse_region_bytes(c.N[m], c.n_features)));
    }
  }
  pl.total = off;
  return pl;
}

laq_status fail(laq_ctx* ctx, laq_status s, const std::string& msg) {
  if (ctx) ctx->err = msg;
  return s;
}

laq_status cuda_fail(laq_ctx* ctx, cudaError_t e, const char* what) {
  return fail(ctx, LAQ_ECUDA, std::string(what) + ": " + cudaGetErrorString(e));
}

#define LAQ_CUDA(ctx, call)                                  \
  do {                                                       \
    cudaError_t e_ = (call);                                 \
    if (e_ != cudaSuccess) return cuda_fail(ctx, e_, #call); \
  } while (0)

bool needs_shards(const laq_ctx* c) {
  return c->cfg.model == LAQ_MODEL_LOGREG_BIN || c->cfg.model == LAQ_MODEL_SOFTMAX || c->cfg.model == LAQ_MODEL_MLP2;
}

// What the device error word says (bit 0: non-finite gradient or radius; any other bit: a bounded wait ran out).
laq_status status_of_error_word(laq_ctx* ctx, uint32_t err) {
  if (err & 1u)
    return fail(ctx, LAQ_ENONFINITE, "a gradient or radius was not finite; the state is frozen at that iteration");
  if (err & ~1u)
    return fail(ctx, LAQ_ETIMEOUT, "a bounded wait on an asynchronous copy or tensor-core stage ran out; the state is frozen at that iteration");
  return LAQ_OK;
}

// Reads the device error word after a synchronisation.
laq_status check_device_error(laq_ctx* ctx) {
  uint32_t err = 0;
  LAQ_CUDA(ctx, cudaMemcpyAsync(&err, &ctx->P.sc->err, 4, cudaMemcpyDeviceToHost, ctx->st));
  LAQ_CUDA(ctx, cudaStreamSynchronize(ctx->st));
  return status_of_error_word(ctx, err);
}

}  // namespace

namespace {

constexpr int kGraphIters = 8;       // iterations per replay of the larger graph
constexpr int kGraphMinIters = 4;    // shorter calls go out as plain launches

// The kernels of one iteration on stream st; ev (5 events) brackets the four stages when profiling.
void enqueue_iteration(laq_ctx* ctx, cudaStream_t st, cudaEvent_t* ev, bool first_half = false) {
  const laq_config& c = ctx->cfg;
  const Params& P = ctx->P;
  if (ev) cudaEventRecord(ev[0], st);
  const int64_t l0 = ctx->launches;
  // small problems: steps 2-5 (and, when cheap, the combination of the gradient kernels' block partials)
  // run in one single-block kernel
  const bool small = small_iteration_applies(P) && !first_half;   // the single-block kernel runs steps 2-5 as one
  const bool linear = c.model == LAQ_MODEL_LOGREG_BIN || c.model == LAQ_MODEL_SOFTMAX;
  const bool fuse_finalize = small && linear && ctx->gbpw <= 64;
  // mid-size linear models: the kernel that combines the gradient partials also takes the quantizer's radius
  const bool fuse_radius = linear && !small && !(c.flags & LAQ_FLAG_QUANT_OFF);
  switch (c.model) {
    case LAQ_MODEL_LOGREG_BIN:
      ctx->launches += launch_grad_logreg(P, ctx->ls, ctx->gbpw, st);
      if (!fuse_finalize) ctx->launches += launch_grad_finalize(P, ctx->gbpw, &P.sc->theta_sq, fuse_radius, st);
      break;
    case LAQ_MODEL_SOFTMAX:
      ctx->launches += (c.flags & LAQ_FLAG_SPARSE_X) ? launch_grad_softmax_sparse(P, ctx->gbpw, st)
                                                     : launch_grad_softmax(P, ctx->ls, ctx->gbpw, st);
      if (!fuse_finalize) ctx->launches += launch_grad_finalize(P, ctx->gbpw, &P.sc->theta_sq, fuse_radius, st);
      break;
    case LAQ_MODEL_MLP2:
      ctx->launches += mlp_launch_gradients(ctx->mlp, P, &P.sc->theta_sq, st);
      break;
    case LAQ_MODEL_SYNTH:
      if (c.flags & LAQ_FLAG_STORE_G) ctx->launches += launch_synth_fill(P, st);
      break;
    default: break;
  }
  if (ev) {
    cudaEventRecord(ev[1], st);
    ctx->stage_launches[0] += ctx->launches - l0;
  }
  if (small) {
    if (ev) {
      cudaEventRecord(ev[2], st);
      cudaEventRecord(ev[3], st);
    }
    ctx->launches += launch_small_iteration(P, fuse_finalize ? ctx->gbpw : 0, st);
  } else {
    if (c.flags & LAQ_FLAG_QUANT_OFF) {
      // no quantizer: one sweep gives the radius, the norm and the skip decisions (the radius slot stays empty)
      if (ev) cudaEventRecord(ev[2], st);
      ctx->launches += launch_innovation_trigger(P, ctx->ls, st);
    } else {
      if (!fuse_radius) ctx->launches += launch_radius(P, ctx->ls, st);
      if (ev) cudaEventRecord(ev[2], st);
      ctx->launches += launch_quantize_trigger(P, ctx->ls, st);
    }
    if (ev) cudaEventRecord(ev[3], st);
    if (!first_half) ctx->launches += launch_aggregate(P, ctx->ls, st);
  }
  if (ev) {
    cudaEventRecord(ev[4], st);
    for (int s = 1; s < 4; ++s) ctx->stage_launches[s] += (s == 1 && (small || fuse_radius || (c.flags & LAQ_FLAG_QUANT_OFF))) ? 0 : 1;
  }
}

bool graphs_usable(const laq_ctx* ctx) {
  return ctx->graphs_enabled && !ctx->graphs_failed && !ctx->profiling && ctx->cfg.model != LAQ_MODEL_EXTERNAL;
}

void drop_graphs(laq_ctx* ctx) {
  if (ctx->graph_one) cudaGraphExecDestroy(ctx->graph_one);
  if (ctx->graph_many) cudaGraphExecDestroy(ctx->graph_many);
  ctx->graph_one = ctx->graph_many = nullptr;
}

// Captures n iterations on the library's own capture stream (the caller's stream may be the legacy default
// stream, which cannot capture) and instantiates them; null on any failure.
cudaGraphExec_t capture_iterations(laq_ctx* ctx, int n) {
  cudaGraph_t graph = nullptr;
  cudaGraphExec_t exec = nullptr;
  if (cudaStreamBeginCapture(ctx->cap_stream, cudaStreamCaptureModeRelaxed) != cudaSuccess) return nullptr;
  const int64_t l0 = ctx->launches;
  for (int i = 0; i < n; ++i) enqueue_iteration(ctx, ctx->cap_stream, nullptr);
  ctx->launches_per_iter = (ctx->launches - l0) / n;
  ctx->launches = l0;                                  // nothing ran: the replays are counted when they are launched
  const cudaError_t e = cudaStreamEndCapture(ctx->cap_stream, &graph);
  if (e == cudaSuccess && graph) {
    if (cudaGraphInstantiate(&exec, graph, 0) != cudaSuccess) exec = nullptr;
    cudaGraphDestroy(graph);
  }
  return exec;
}

void build_graphs(laq_ctx* ctx) {
  if (!ctx->cap_stream && cudaStreamCreateWithFlags(&ctx->cap_stream, cudaStreamNonBlocking) != cudaSuccess) {
    ctx->graphs_failed = true;
    return;
  }
  ctx->graph_one = capture_iterations(ctx, 1);
  ctx->graph_many = ctx->graph_one ? capture_iterations(ctx, kGraphIters) : nullptr;
  if (!ctx->graph_one || !ctx->graph_many) {
    drop_graphs(ctx);
    ctx->graphs_failed = true;    // plain launches from now on
    cudaGetLastError();
  }
}

}  // namespace

extern "C" {

size_t laq_workspace_bytes(const laq_config* cfg) {
  if (check_config(cfg)) return 0;
  std::vector<int64_t> Nl;
  const laq_config l = localize(*cfg, Nl, nullptr);
  return make_plan(l, cfg->M).total;
}

laq_status laq_init(laq_ctx** out, const laq_config* cfg, void* d_workspace, size_t workspace_bytes,
                    const float* theta0, void* cuda_stream) {
  if (!out) return LAQ_EINVAL;
  *out = nullptr;
  laq_ctx* ctx = new (std::nothrow) laq_ctx();
  if (!ctx) return LAQ_EINVAL;
  *out = ctx;  // returned even on failure so that laq_last_error can be read; free with laq_destroy
  std::memset(&ctx->P, 0, sizeof(Params));
  std::memset(&ctx->cfg, 0, sizeof(laq_config));
  if (const char* e = check_config(cfg)) return fail(ctx, LAQ_EINVAL, e);
  long long n_total = 0;
  ctx->cfg = localize(*cfg, ctx->N, &n_total);
  ctx->xi.assign(cfg->xi, cfg->xi + cfg->D);
  ctx->cfg.xi = ctx->xi.data();
  ctx->cfg.N = ctx->N.data();
  ctx->world = cfg->world > 1 ? cfg->world : 1;
  ctx->rank = cfg->world > 1 ? cfg->rank : 0;
  ctx->M_total = cfg->M;
  ctx->st = (cudaStream_t)cuda_stream;
  const Plan pl = make_plan(ctx->cfg, ctx->M_total);
  if (!d_workspace) return fail(ctx, LAQ_EWORKSPACE, "workspace is null");
  if ((uintptr_t)d_workspace % kAlign) return fail(ctx, LAQ_EWORKSPACE, "workspace must be 256-byte aligned");
  if (workspace_bytes < pl.total) return fail(ctx, LAQ_EWORKSPACE, "workspace is smaller than laq_workspace_bytes(cfg)");
  cudaPointerAttributes attr;
  if (cudaPointerGetAttributes(&attr, d_workspace) != cudaSuccess ||
      (attr.type != cudaMemoryTypeDevice && attr.type != cudaMemoryTypeManaged)) {
    cudaGetLastError();
    return fail(ctx, LAQ_EWORKSPACE, "workspace is not device memory");
  }
  char* ws = (char*)d_workspace;
  ctx->ws = ws;
  ctx->ws_bytes = workspace_bytes;
  Params& P = ctx->P;
  const laq_config& c = ctx->cfg;
  P.M = c.M; P.b = c.b; P.D = c.D; P.tbar = c.tbar; P.clock_mode = c.clock_mode; P.model = c.model;
  P.M_total = ctx->M_total; P.m_first = ctx->rank; P.m_stride = ctx->world;
  P.flags = c.flags;
  P.F = c.n_features; P.C = c.n_classes; P.H = c.n_hidden;
  P.p = c.p; P.ps = pl.ps; P.nv = pl.nv; P.cw = pl.cw;
  P.alpha = c.alpha; P.lambda = c.lambda;
  {
    const double a = (double)c.alpha;
    P.trig_c = (a * a) * ((double)ctx->M_total * (double)ctx->M_total);   // (7a) divides by alpha^2 M^2, M = all workers
  }
  P.sc = (DevScalars*)(ws + pl.sc);
  P.theta = (float*)(ws + pl.theta);
  P.agg = (float*)(ws + pl.agg);
  P.qp = (float*)(ws + pl.qp);
  P.g = (c.model == LAQ_MODEL_SYNTH && !(c.flags & LAQ_FLAG_STORE_G)) ? nullptr : (float*)(ws + pl.g);
  P.codes = (uint32_t*)(ws + pl.codes);
  P.Rbits = (uint32_t*)(ws + pl.Rbits);
  P.norms = (double*)(ws + pl.norms);
  P.n_epshat = (double*)(ws + pl.n_epshat);
  P.clock = (int32_t*)(ws + pl.clock);
  P.skip = (uint8_t*)(ws + pl.skip);
  P.up_m = (int32_t*)(ws + pl.up_m);
  P.up_q = (int32_t*)(ws + pl.up_q);
  ctx->d_up_m_in = (int32_t*)(ws + pl.up_in_m);
  ctx->d_up_R_in = (float*)(ws + pl.up_in_R);
  P.up_R = (float*)(ws + pl.up_R);
  P.up_s = (float*)(ws + pl.up_s);
  P.ring = (double*)(ws + pl.ring);
  P.xi = (float*)(ws + pl.xi);
  P.loss_m = (double*)(ws + pl.loss_m);
  P.part_q = (double*)(ws + pl.part_q);
  P.part_d = (double*)(ws + pl.part_d);
  P.part_t = (double*)(ws + pl.part_t);
  P.trace_cap = c.trace_capacity;
  P.t_skip = (uint8_t*)(ws + pl.t_skip);
  P.t_R = (float*)(ws + pl.t_R);
  P.t_ndq = (double*)(ws + pl.t_ndq);
  P.t_neps = (double*)(ws + pl.t_neps);
  P.t_rhs = (double*)(ws + pl.t_rhs);
  P.t_d2 = (double*)(ws + pl.t_d2);
  P.t_loss = (double*)(ws + pl.t_loss);
  P.t_up = (int32_t*)(ws + pl.t_up);
  P.seed_lo = (uint32_t)(c.seed & 0xffffffffull);
  P.seed_hi = (uint32_t)(c.seed >> 32);
  P.batch = c.batch;
  P.zero = 0u;
  P.starve = 0u;
  P.cz = (float)((double)c.synth_sigma / std::sqrt(21845.0));
  P.eta0 = c.synth_eta0;
  P.X = (const float* const*)(ws + pl.Xptr);
  P.y = (const int32_t* const*)(ws + pl.yptr);
  P.N = (const long long*)(ws + pl.Ndev);
  P.cnt_grad = (uint32_t*)(ws + pl.cnt_grad);
  P.gpart = (float*)(ws + pl.gpart);
  P.lpart = (double*)(ws + pl.lpart);
  P.Ntot = n_total;      // samples of ALL workers: f = (1/N) sum_m f_m
  P.Nloc = 0;
  for (int m = 0; m < c.M; ++m) P.Nloc += ctx->N[m];
  P.sp = (const SparseShard*)(ws + pl.sp_desc);
  for (size_t m = 0; m < pl.sp.size(); ++m) ctx->sp_region.push_back(ws + pl.sp[m]);
  ctx->gbpw_cap = pl.gbpw_cap;
  ctx->gbpw = default_gbpw(c);
  if (c.flags & LAQ_FLAG_SPARSE_X) {
    ctx->gbpw = sparse_blocks_per_worker((const long long*)ctx->N.data(), c.M);
    if (ctx->gbpw > kGradBlocksCap) ctx->gbpw = kGradBlocksCap;
  }
  if ((c.model == LAQ_MODEL_LOGREG_BIN || c.model == LAQ_MODEL_SOFTMAX) && !(c.flags & LAQ_FLAG_SPARSE_X)) {
    long long n_max = 1;
    for (int m = 0; m < c.M; ++m) n_max = ctx->N[m] > n_max ? ctx->N[m] : n_max;
    const int tiles = grad_tiles_per_worker(c.model, c.n_features, c.n_classes, n_max);
    if (ctx->gbpw > tiles) ctx->gbpw = tiles;
  }

  LAQ_CUDA(ctx, cudaMemsetAsync(ws, 0, pl.state_end, ctx->st));
  if (needs_shards(ctx)) {
    ctx->shard_loaded.assign(c.M, 0);
    ctx->Xptr.resize(c.M);
    ctx->yptr.resize(c.M);
    for (int m = 0; m < c.M; ++m) {
      ctx->Xptr[m] = (const float*)(ws + pl.X[m]);
      ctx->yptr[m] = (const int32_t*)(ws + pl.y[m]);
    }
    LAQ_CUDA(ctx, cudaMemcpyAsync(ws + pl.Xptr, ctx->Xptr.data(), 8 * (size_t)c.M, cudaMemcpyHostToDevice, ctx->st));
    LAQ_CUDA(ctx, cudaMemcpyAsync(ws + pl.yptr, ctx->yptr.data(), 8 * (size_t)c.M, cudaMemcpyHostToDevice, ctx->st));
    LAQ_CUDA(ctx, cudaMemcpyAsync(ws + pl.Ndev, ctx->N.data(), 8 * (size_t)c.M, cudaMemcpyHostToDevice, ctx->st));
    if (c.model == LAQ_MODEL_MLP2) {
      laq_status s = mlp_setup(ctx->mlp, P, (const long long*)ctx->N.data(), ws + pl.mlp, ctx->st);
      if (s == LAQ_OK) s = mlp_set_row_offsets(ctx->mlp, (const long long*)ctx->N.data(), c.M, ctx->st);
      if (s == LAQ_OK) s = mlp_setup_tensor_path(ctx->mlp, P, ctx->st);
      if (s != LAQ_OK) return fail(ctx, s, "network scratch set-up failed");
      // tensor-core path: the theta step keeps the bf16 copy of W1 current (H F is a multiple of 4 there)
      P.w1b = (uint16_t*)mlp_w1_copy(ctx->mlp);
      P.w1b_n = P.w1b ? (long long)c.n_hidden * c.n_features : 0;
    }
  }
  std::vector<int32_t> clocks(c.M, c.tbar + 1);  // every worker uploads at k = 1
  LAQ_CUDA(ctx, cudaMemcpyAsync(P.clock, clocks.data(), 4 * (size_t)c.M, cudaMemcpyHostToDevice, ctx->st));
  LAQ_CUDA(ctx, cudaMemcpyAsync(P.xi, ctx->xi.data(), 4 * (size_t)c.D, cudaMemcpyHostToDevice, ctx->st));
  if (theta0) {
    LAQ_CUDA(ctx, cudaMemcpyAsync(P.theta, theta0, 4 * (size_t)c.p, cudaMemcpyHostToDevice, ctx->st));
    ctx->launches += launch_theta_sq(P, ctx->st);        // ||theta^0||^2 for the regulariser term of the loss
  }
  if (c.model == LAQ_MODEL_MLP2) ctx->launches += mlp_refresh_w1_copy(ctx->mlp, P, ctx->st);   // theta^0 (or zeros)
  LAQ_CUDA(ctx, cudaStreamSynchronize(ctx->st));  // the host vectors above go out of scope
  return LAQ_OK;
}

laq_status laq_load_shards(laq_ctx* ctx, int32_t m, const float* X, const int32_t* y, int64_t N_m,
                           int32_t on_device) {
  if (!ctx || !ctx->ws) return LAQ_EINVAL;
  if (!needs_shards(ctx)) return fail(ctx, LAQ_ESTATE, "this model holds no data shards");
  if (m < 0 || m >= ctx->cfg.M) return fail(ctx, LAQ_EINVAL, "worker index out of range");
  if (!X || !y) return fail(ctx, LAQ_EINVAL, "X or y is null");
  if (N_m != ctx->N[m]) return fail(ctx, LAQ_EINVAL, "N_m differs from the configured value");
  const cudaMemcpyKind kind = on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice;
  LAQ_CUDA(ctx, cudaMemcpyAsync((void*)ctx->Xptr[m], X, (size_t)N_m * ctx->cfg.n_features * 4, kind, ctx->st));
  LAQ_CUDA(ctx, cudaMemcpyAsync((void*)ctx->yptr[m], y, (size_t)N_m * 4, kind, ctx->st));
  if (ctx->cfg.model == LAQ_MODEL_MLP2) {
    long long row_offset = 0;
    for (int i = 0; i < m; ++i) row_offset += ctx->N[i];
    ctx->launches += mlp_convert_shard(ctx->mlp, ctx->P, m, ctx->Xptr[m], N_m, row_offset, ctx->st);
  }
  if (ctx->cfg.flags & LAQ_FLAG_SPARSE_X) {
    std::string why;
    const laq_status s = sparse_build(m, ctx->Xptr[m], N_m, ctx->cfg.n_features, ctx->sp_region[m],
                                      const_cast<SparseShard*>(ctx->P.sp), ctx->st, &why);
    if (s != LAQ_OK) return fail(ctx, s, why);
    ctx->launches += 2;
  }
  LAQ_CUDA(ctx, cudaStreamSynchronize(ctx->st));  // the caller may reuse its buffers on return
  ctx->shard_loaded[m] = 1;
  return LAQ_OK;
}

laq_status laq_set_gradients(laq_ctx* ctx, const float* g, int32_t on_device) {
  if (!ctx || !ctx->ws) return LAQ_EINVAL;
  if (ctx->cfg.model != LAQ_MODEL_EXTERNAL) return fail(ctx, LAQ_ESTATE, "model is not LAQ_MODEL_EXTERNAL");
  if (!g) return fail(ctx, LAQ_EINVAL, "g is null");
  const cudaMemcpyKind kind = on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice;
  const Params& P = ctx->P;
  LAQ_CUDA(ctx, cudaMemcpy2DAsync(P.g, (size_t)P.ps * 4, g, (size_t)P.p * 4, (size_t)P.p * 4, (size_t)P.M, kind,
                                  ctx->st));
  if (!on_device) LAQ_CUDA(ctx, cudaStreamSynchronize(ctx->st));
  ctx->ext_g_set = true;
  return LAQ_OK;
}

laq_status laq_step(laq_ctx* ctx, int32_t n_iters, const laq_trace* trace) {
  if (!ctx || !ctx->ws) return LAQ_EINVAL;
  if (n_iters < 0) return fail(ctx, LAQ_EINVAL, "n_iters must be >= 0");
  const laq_config& c = ctx->cfg;
  const Params& P = ctx->P;
  if (needs_shards(ctx))
    for (int m = 0; m < c.M; ++m)
      if (!ctx->shard_loaded[m]) return fail(ctx, LAQ_ESTATE, "laq_load_shards has not been called for every worker");
  if (c.model == LAQ_MODEL_EXTERNAL) {
    if (n_iters > 1) return fail(ctx, LAQ_EINVAL, "LAQ_MODEL_EXTERNAL steps one iteration per call");
    if (n_iters == 1 && !ctx->ext_g_set) return fail(ctx, LAQ_ESTATE, "laq_set_gradients has not been called");
  }
  if (trace && n_iters > c.trace_capacity) return fail(ctx, LAQ_EINVAL, "n_iters exceeds trace_capacity");
  if (ctx->world > 1 && n_iters > 0)
    return fail(ctx, LAQ_ESTATE, "workers are spread over contexts: use laq_step_local, laq_local_uploads, laq_apply_uploads");
  LAQ_CUDA(ctx, cudaMemsetAsync(&P.sc->trace_pos, trace ? 0 : 0xff, 4, ctx->st));  // 0xffffffff = tracing off
  int it = 0;
  if (graphs_usable(ctx) && n_iters >= kGraphMinIters) {
    // the first iteration of a context goes out as plain launches (it also sets the kernels' attributes); the
    // graphs are then captured once and replayed: fewer host calls and shorter gaps between dependent kernels
    if (!ctx->graph_one) {
      enqueue_iteration(ctx, ctx->st, nullptr);
      it = 1;
      build_graphs(ctx);
    }
    if (ctx->graph_one) {
      for (; it + kGraphIters <= n_iters; it += kGraphIters) {
        LAQ_CUDA(ctx, cudaGraphLaunch(ctx->graph_many, ctx->st));
        ctx->launches += ctx->launches_per_iter * kGraphIters;
      }
      for (; it < n_iters; ++it) {
        LAQ_CUDA(ctx, cudaGraphLaunch(ctx->graph_one, ctx->st));
        ctx->launches += ctx->launches_per_iter;
      }
    }
  }
  for (; it < n_iters; ++it) {
    cudaEvent_t* ev = nullptr;
    if (ctx->profiling && ctx->ev_used < kProfIters) {
      ev = &ctx->ev[(size_t)ctx->ev_used * 5];
      ctx->ev_used += 1;
    }
    enqueue_iteration(ctx, ctx->st, ev);
  }
  LAQ_CUDA(ctx, cudaGetLastError());
  if (c.model == LAQ_MODEL_EXTERNAL && n_iters == 1) ctx->ext_g_set = false;
  if (!trace) return LAQ_OK;
  const size_t n = (size_t)n_iters, M = (size_t)c.M;
  // The eight report arrays lie one after the other in the workspace.  Short reports come back as ONE copy of that
  // span into a host buffer of the context and are handed out from there: a call that steps one iteration and reads
  // its report pays for one transfer instead of eight.  Long reports are copied array by array, rows used only.
  const char* span0 = (const char*)P.t_skip;
  const size_t span = (size_t)((const char*)P.t_up + (size_t)c.trace_capacity * 4 - span0);
  if (span <= kTraceSpanMax) {
    if (ctx->trace_host.size() < span) ctx->trace_host.resize(span);
    LAQ_CUDA(ctx, cudaMemcpyAsync(ctx->trace_host.data(), span0, span, cudaMemcpyDeviceToHost, ctx->st));
    const laq_status status = check_device_error(ctx);     // synchronises
    auto hand = [&](void* dst, const void* src, size_t bytes) {
      if (dst && bytes) std::memcpy(dst, ctx->trace_host.data() + ((const char*)src - span0), bytes);
    };
    hand(trace->skip, P.t_skip, n * M);
    hand(trace->R, P.t_R, n * M * 4);
    hand(trace->n_dq, P.t_ndq, n * M * 8);
    hand(trace->n_eps, P.t_neps, n * M * 8);
    hand(trace->rhs, P.t_rhs, n * M * 8);
    hand(trace->dtheta2, P.t_d2, n * 8);
    hand(trace->loss, P.t_loss, n * 8);
    hand(trace->uploads, P.t_up, n * 4);
    return status;
  }
  auto pull = [&](void* dst, const void* src, size_t bytes) -> cudaError_t {
    if (!dst || !bytes) return cudaSuccess;
    return cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToHost, ctx->st);
  };
  LAQ_CUDA(ctx, pull(trace->skip, P.t_skip, n * M));
  LAQ_CUDA(ctx, pull(trace->R, P.t_R, n * M * 4));
  LAQ_CUDA(ctx, pull(trace->n_dq, P.t_ndq, n * M * 8));
  LAQ_CUDA(ctx, pull(trace->n_eps, P.t_neps, n * M * 8));
  LAQ_CUDA(ctx, pull(trace->rhs, P.t_rhs, n * M * 8));
  LAQ_CUDA(ctx, pull(trace->dtheta2, P.t_d2, n * 8));
  LAQ_CUDA(ctx, pull(trace->loss, P.t_loss, n * 8));
  LAQ_CUDA(ctx, pull(trace->uploads, P.t_up, n * 4));
  return check_device_error(ctx);
}

laq_status laq_step_local(laq_ctx* ctx) {
  if (!ctx || !ctx->ws) return LAQ_EINVAL;
  const laq_config& c = ctx->cfg;
  if (c.flags & LAQ_FLAG_QUANT_OFF) return fail(ctx, LAQ_ESTATE, "the split iteration needs the quantizer");
  if (needs_shards(ctx))
    for (int m = 0; m < c.M; ++m)
      if (!ctx->shard_loaded[m]) return fail(ctx, LAQ_ESTATE, "laq_load_shards has not been called for every worker");
  if (c.model == LAQ_MODEL_EXTERNAL && !ctx->ext_g_set) return fail(ctx, LAQ_ESTATE, "laq_set_gradients has not been called");
  LAQ_CUDA(ctx, cudaMemsetAsync(&ctx->P.sc->trace_pos, 0xff, 4, ctx->st));   // no per-iteration report
  enqueue_iteration(ctx, ctx->st, nullptr, /*first_half=*/true);
  LAQ_CUDA(ctx, cudaGetLastError());
  ctx->ext_g_set = false;
  return LAQ_OK;
}

laq_status laq_local_uploads(laq_ctx* ctx, int32_t* n, int32_t* m, float* R) {
  if (!ctx || !ctx->ws) return LAQ_EINVAL;
  if (!n || !m || !R) return fail(ctx, LAQ_EINVAL, "null pointer");
  const Params& P = ctx->P;
  DevScalars sc;
  LAQ_CUDA(ctx, cudaMemcpyAsync(&sc, P.sc, sizeof(sc), cudaMemcpyDeviceToHost, ctx->st));
  LAQ_CUDA(ctx, cudaStreamSynchronize(ctx->st));
  *n = 0;
  if (const laq_status st = status_of_error_word(ctx, sc.err)) return st;
  if ((int)sc.n_up > P.M) return fail(ctx, LAQ_ESTATE, "laq_local_uploads must follow laq_step_local");
  LAQ_CUDA(ctx, cudaMemcpyAsync(m, P.up_m, 4 * (size_t)sc.n_up, cudaMemcpyDeviceToHost, ctx->st));
  LAQ_CUDA(ctx, cudaMemcpyAsync(R, P.up_R, 4 * (size_t)sc.n_up, cudaMemcpyDeviceToHost, ctx->st));
  LAQ_CUDA(ctx, cudaStreamSynchronize(ctx->st));
  for (uint32_t u = 0; u < sc.n_up; ++u) m[u] = ctx->rank + ctx->world * m[u];   // local row -> global worker index
  *n = (int32_t)sc.n_up;
  return LAQ_OK;
}

laq_status laq_apply_uploads(laq_ctx* ctx, int32_t n, const int32_t* m, const float* R) {
  if (!ctx || !ctx->ws) return LAQ_EINVAL;
  if (n < 0 || n > ctx->M_total || (n > 0 && (!m || !R))) return fail(ctx, LAQ_EINVAL, "bad upload list");
  for (int u = 0; u < n; ++u)
    if (m[u] < 0 || m[u] >= ctx->M_total || (u > 0 && m[u] <= m[u - 1]))
      return fail(ctx, LAQ_EINVAL, "upload list must hold distinct global worker indices in ascending order");
  if (n > 0) {
    LAQ_CUDA(ctx, cudaMemcpyAsync(ctx->d_up_m_in, m, 4 * (size_t)n, cudaMemcpyHostToDevice, ctx->st));
    LAQ_CUDA(ctx, cudaMemcpyAsync(ctx->d_up_R_in, R, 4 * (size_t)n, cudaMemcpyHostToDevice, ctx->st));
    LAQ_CUDA(ctx, cudaStreamSynchronize(ctx->st));      // m and R are the caller's pageable host memory
  }
  ctx->launches += launch_merge_uploads(ctx->P, n, ctx->d_up_m_in, ctx->d_up_R_in, ctx->st);
  ctx->launches += launch_aggregate(ctx->P, ctx->ls, ctx->st);
  LAQ_CUDA(ctx, cudaGetLastError());
  return LAQ_OK;
}

laq_status laq_sync(laq_ctx* ctx) {
  if (!ctx || !ctx->ws) return LAQ_EINVAL;
  return check_device_error(ctx);
}

laq_status laq_get_state(laq_ctx* ctx, const laq_state* out) {
  if (!ctx || !ctx->ws) return LAQ_EINVAL;
  if (!out) return fail(ctx, LAQ_EINVAL, "state is null");
  const Params& P = ctx->P;
  const size_t M = (size_t)P.M, p = (size_t)P.p;
  DevScalars sc;
  LAQ_CUDA(ctx, cudaMemcpyAsync(&sc, P.sc, sizeof(sc), cudaMemcpyDeviceToHost, ctx->st));
  LAQ_CUDA(ctx, cudaStreamSynchronize(ctx->st));
  auto pull = [&](void* dst, const void* src, size_t bytes) -> cudaError_t {
    if (!dst || !bytes) return cudaSuccess;
    return cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToHost, ctx->st);
  };
  auto pull2d = [&](void* dst, size_t dpitch, const void* src, size_t spitch, size_t width, size_t rows) -> cudaError_t {
    if (!dst) return cudaSuccess;
    return cudaMemcpy2DAsync(dst, dpitch, src, spitch, width, rows, cudaMemcpyDeviceToHost, ctx->st);
  };
  LAQ_CUDA(ctx, pull(out->theta, P.theta, p * 4));
  LAQ_CUDA(ctx, pull(out->agg, P.agg, p * 4));
  LAQ_CUDA(ctx, pull2d(out->qprev, p * 4, P.qp, (size_t)P.ps * 4, p * 4, M));
  if (out->g) {
    if (!P.g) return fail(ctx, LAQ_EINVAL, "g is not stored for LAQ_MODEL_SYNTH");
    LAQ_CUDA(ctx, pull2d(out->g, p * 4, P.g, (size_t)P.ps * 4, p * 4, M));
  }
  const size_t W = (p * (size_t)P.b + 31) / 32;
  LAQ_CUDA(ctx, pull2d(out->codes, W * 4, P.codes, (size_t)P.cw * 4, W * 4, M));
  LAQ_CUDA(ctx, pull(out->n_eps_hat, P.n_epshat, M * 8));
  LAQ_CUDA(ctx, pull(out->clock, P.clock, M * 4));
  LAQ_CUDA(ctx, pull(out->skip, P.skip, M));
  std::vector<double> ring(P.D), norms(3 * M);
  std::vector<uint32_t> Rb(2 * M);
  LAQ_CUDA(ctx, pull(ring.data(), P.ring, (size_t)P.D * 8));
  LAQ_CUDA(ctx, pull(norms.data(), P.norms, 3 * M * 8));
  LAQ_CUDA(ctx, pull(Rb.data(), P.Rbits, 2 * M * 4));
  LAQ_CUDA(ctx, cudaStreamSynchronize(ctx->st));
  if (out->ring)
    for (int d = 0; d < P.D; ++d) out->ring[d] = ring[(sc.ring_head + d) % P.D];
  for (size_t m = 0; m < M; ++m) {
    if (out->n_dq) out->n_dq[m] = norms[3 * m];
    if (out->n_eps) out->n_eps[m] = norms[3 * m + 1];
    if (out->R) {
      const uint32_t bits = sc.k ? Rb[((sc.k - 1) & 1ull) * M + m] : 0u;
      std::memcpy(&out->R[m], &bits, 4);
    }
  }
  if (out->counters) {
    out->counters[0] = (int64_t)sc.k;
    out->counters[1] = (int64_t)sc.uploads;
    out->counters[2] = (int64_t)sc.bits;
  }
  return status_of_error_word(ctx, sc.err);
}

laq_status laq_get_worker(laq_ctx* ctx, int32_t m, float* qprev, float* g, uint32_t* codes, float* R) {
  if (!ctx || !ctx->ws) return LAQ_EINVAL;
  const Params& P = ctx->P;
  if (m < 0 || m >= P.M) return fail(ctx, LAQ_EINVAL, "worker index out of range");
  if (g && !P.g) return fail(ctx, LAQ_EINVAL, "g is not stored for LAQ_MODEL_SYNTH");
  const size_t p = (size_t)P.p, W = (p * (size_t)P.b + 31) / 32;
  DevScalars sc;
  LAQ_CUDA(ctx, cudaMemcpyAsync(&sc, P.sc, sizeof(sc), cudaMemcpyDeviceToHost, ctx->st));
  LAQ_CUDA(ctx, cudaStreamSynchronize(ctx->st));
  if (qprev) LAQ_CUDA(ctx, cudaMemcpyAsync(qprev, P.qp + (size_t)m * P.ps, p * 4, cudaMemcpyDeviceToHost, ctx->st));
  if (g) LAQ_CUDA(ctx, cudaMemcpyAsync(g, P.g + (size_t)m * P.ps, p * 4, cudaMemcpyDeviceToHost, ctx->st));
  if (codes) LAQ_CUDA(ctx, cudaMemcpyAsync(codes, P.codes + (size_t)m * P.cw, W * 4, cudaMemcpyDeviceToHost, ctx->st));
  if (R) {
    *R = 0.f;
    if (sc.k)
      LAQ_CUDA(ctx, cudaMemcpyAsync(R, P.Rbits + ((sc.k - 1) & 1ull) * P.M + m, 4, cudaMemcpyDeviceToHost, ctx->st));
  }
  LAQ_CUDA(ctx, cudaStreamSynchronize(ctx->st));
  return status_of_error_word(ctx, sc.err);
}

laq_status laq_set_state(laq_ctx* ctx, const laq_state* in) {
  if (!ctx || !ctx->ws) return LAQ_EINVAL;
  if (!in) return fail(ctx, LAQ_EINVAL, "state is null");
  const Params& P = ctx->P;
  const size_t M = (size_t)P.M, p = (size_t)P.p;
  DevScalars sc;
  LAQ_CUDA(ctx, cudaMemcpyAsync(&sc, P.sc, sizeof(sc), cudaMemcpyDeviceToHost, ctx->st));
  LAQ_CUDA(ctx, cudaStreamSynchronize(ctx->st));
  auto push = [&](void* dst, const void* src, size_t bytes) -> cudaError_t {
    if (!src || !bytes) return cudaSuccess;
    return cudaMemcpyAsync(dst, src, bytes, cudaMemcpyHostToDevice, ctx->st);
  };
  LAQ_CUDA(ctx, push(P.theta, in->theta, p * 4));
  LAQ_CUDA(ctx, push(P.agg, in->agg, p * 4));
  if (in->qprev)
    LAQ_CUDA(ctx, cudaMemcpy2DAsync(P.qp, (size_t)P.ps * 4, in->qprev, p * 4, p * 4, M, cudaMemcpyHostToDevice, ctx->st));
  LAQ_CUDA(ctx, push(P.n_epshat, in->n_eps_hat, M * 8));
  LAQ_CUDA(ctx, push(P.clock, in->clock, M * 4));
  if (in->ring) {
    LAQ_CUDA(ctx, push(P.ring, in->ring, (size_t)P.D * 8));
    sc.ring_head = 0;
  }
  if (in->counters) {
    if (in->counters[0] < 0 || in->counters[1] < 0 || in->counters[2] < 0) return fail(ctx, LAQ_EINVAL, "negative counter");
    sc.k = (unsigned long long)in->counters[0];
    sc.uploads = (unsigned long long)in->counters[1];
    sc.bits = (unsigned long long)in->counters[2];
  }
  sc.err = 0;
  sc.cnt_quant = sc.cnt_agg = 0;
  LAQ_CUDA(ctx, cudaMemsetAsync(P.Rbits, 0, 2 * M * 4, ctx->st));
  LAQ_CUDA(ctx, cudaMemcpyAsync(P.sc, &sc, sizeof(sc), cudaMemcpyHostToDevice, ctx->st));
  if (in->theta) ctx->launches += launch_theta_sq(P, ctx->st);   // after the scalars: it overwrites theta_sq
  if (in->theta && ctx->cfg.model == LAQ_MODEL_MLP2) ctx->launches += mlp_refresh_w1_copy(ctx->mlp, P, ctx->st);
  LAQ_CUDA(ctx, cudaStreamSynchronize(ctx->st));
  return LAQ_OK;
}

int64_t laq_kernel_launches(const laq_ctx* ctx) { return ctx ? ctx->launches : 0; }

laq_status laq_tune(laq_ctx* ctx, const char* key, int32_t value) {
  if (!ctx || !ctx->ws || !key) return LAQ_EINVAL;
  const std::string k(key);
  auto pow2_threads = [](int v) { return v == 64 || v == 128 || v == 256 || v == 512; };
  if (k == "sweep_threads" && pow2_threads(value)) ctx->ls.sweep_threads = value;
  else if (k == "sweep_blocks_per_sm" && value >= 1 && value <= 128) ctx->ls.sweep_blocks_per_sm = value;
  else if (k == "agg_threads" && pow2_threads(value) && value <= 256) ctx->ls.agg_threads = value;
  else if (k == "agg_blocks_per_sm" && value >= 1 && value <= 32) ctx->ls.agg_blocks_per_sm = value;
  else if (k == "grad_blocks_per_worker" && value >= 1 && value <= ctx->gbpw_cap) ctx->gbpw = value;
  else if (k == "graphs" && (value == 0 || value == 1)) ctx->graphs_enabled = value != 0;
  else if (k == "starve_copies" && (value == 0 || value == 1)) ctx->P.starve = (uint32_t)value;
  else return fail(ctx, LAQ_EINVAL, "unknown tuning key or value outside its limits");
  drop_graphs(ctx);     // captured launch shapes are stale
  return LAQ_OK;
}

laq_status laq_query(const laq_ctx* ctx, const char* key, int64_t* value) {
  if (!ctx || !ctx->ws || !key || !value) return LAQ_EINVAL;
  const std::string k(key);
  if (k == "sweep_blocks_per_worker") *value = sweep_blocks_per_worker(ctx->P, ctx->ls);
  else if (k == "sweep_threads") *value = ctx->ls.sweep_threads;
  else if (k == "sweep_tile_groups") *value = sweep_tile_groups();
  else if (k == "aggregate_blocks") *value = aggregate_blocks(ctx->P, ctx->ls);
  else if (k == "grad_blocks_per_worker") *value = ctx->gbpw;
  else if (k == "local_workers") *value = ctx->P.M;
  else if (k == "codes_offset_bytes") *value = (int64_t)((const char*)ctx->P.codes - ctx->ws);
  else if (k == "code_row_bytes") *value = (int64_t)ctx->P.cw * 4;
  else if (k == "mailbox_offset_bytes")
    *value = ctx->M_total != ctx->P.M ? (int64_t)((const char*)(ctx->P.codes + (size_t)ctx->P.M * ctx->P.cw) - ctx->ws) : -1;
  else return LAQ_EINVAL;
  return LAQ_OK;
}

laq_status laq_set_profiling(laq_ctx* ctx, int32_t enabled) {
  if (!ctx || !ctx->ws) return LAQ_EINVAL;
  if (enabled && ctx->ev.empty()) {
    ctx->ev.resize((size_t)kProfIters * 5);
    for (auto& e : ctx->ev) LAQ_CUDA(ctx, cudaEventCreate(&e));
  }
  ctx->profiling = enabled != 0;
  return LAQ_OK;
}

laq_status laq_kernel_times(laq_ctx* ctx, double* ms, int64_t* launches) {
  if (!ctx || !ctx->ws) return LAQ_EINVAL;
  LAQ_CUDA(ctx, cudaStreamSynchronize(ctx->st));
  for (int i = 0; i < ctx->ev_used; ++i) {
    cudaEvent_t* ev = &ctx->ev[(size_t)i * 5];
    for (int s = 0; s < 4; ++s) {
      float t = 0.f;
      LAQ_CUDA(ctx, cudaEventElapsedTime(&t, ev[s], ev[s + 1]));
      ctx->stage_ms[s] += (double)t;
    }
  }
  ctx->ev_used = 0;
  for (int s = 0; s < 4; ++s) {
    if (ms) ms[s] = ctx->stage_ms[s];
    if (launches) launches[s] = ctx->stage_launches[s];
    ctx->stage_ms[s] = 0.0;
    ctx->stage_launches[s] = 0;
  }
  return LAQ_OK;
}

const char* laq_last_error(const laq_ctx* ctx) { return ctx ? ctx->err.c_str() : "context is null"; }

void laq_destroy(laq_ctx* ctx) {
  if (!ctx) return;
  if (ctx->ws) cudaStreamSynchronize(ctx->st);
  mlp_teardown(ctx->mlp);
  drop_graphs(ctx);
  if (ctx->cap_stream) cudaStreamDestroy(ctx->cap_stream);
  for (auto& e : ctx->ev) cudaEventDestroy(e);
  delete ctx;
}

}  // extern "C"
