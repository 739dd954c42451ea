// Internal declarations shared by the library's translation units (not part of the public ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <string>

#include "laq.h"

namespace laq {

constexpr int kMaxWorkers = 1024;   // M limit: the trigger stage runs in one block
constexpr int kMaxD = 64;           // D limit
constexpr int kMaxSweepBlocksPerWorker = 256;
constexpr int kNumSMs = 148;        // B200

// Scalars that live on the device so that an iteration needs no host round trip.
struct DevScalars {
  uint32_t err;         // 0 = ok; bit 0 = non-finite gradient/radius (state frozen)
  uint32_t ring_head;   // slot of the newest stored squared parameter difference
  uint32_t trace_pos;   // next trace row
  uint32_t n_up;        // |M^k| of the iteration in flight
  uint32_t cnt_quant;   // "last block done" tickets
  uint32_t cnt_agg;
  uint32_t pad0, pad1;
  unsigned long long k;        // iterations done
  unsigned long long uploads;  // sum_k |M^k|
  unsigned long long bits;     // uploads x (32 + b p)
  double theta_sq;             // ||theta^k||^2 (for the regulariser term of the reported loss)
};

// A worker's shard in compressed form (LAQ_FLAG_SPARSE_X), see laq_grad_sparse.cu.
struct SparseShard {
  const float* val;          // values of both copies
  const uint16_t* idx;       // feature index (copy by rows) or row in tile (copy by columns)
  const long long* off_r;    // [tiles + 1] first entry of each tile's copy by rows
  const long long* off_c;    // [tiles + 1] first entry of each tile's copy by columns
  int tiles;
};

// Everything a kernel needs, passed by value.
struct Params {
  int M, b, D, tbar, clock_mode, model;   // M: workers whose rows live in this context
  int M_total, m_first, m_stride;         // all workers; local worker m is global worker m_first + m_stride m
  uint32_t flags;
  int F, C, H;               // model shape
  long long p, ps, nv, cw;   // coordinates, padded row stride (floats), ps/4, code words per row
  float alpha, lambda;
  double trig_c;             // alpha^2 M^2 (fp64)
  // state
  float* theta;
  float* agg;
  float* qp;        // [M][ps]
  float* g;         // [M][ps]   (null for SYNTH)
  uint32_t* codes;  // [M][cw]
  uint32_t* Rbits;  // [2][M]   radius as float bits, double-buffered by iteration parity
  double* norms;    // [M][3]   n_dq, n_eps, rhs of the last iteration
  double* n_epshat; // [M]
  int32_t* clock;   // [M]
  uint8_t* skip;    // [M]
  int32_t* up_m;    // [M_total] uploaders in ascending order: row of the code buffer that holds the message
  int32_t* up_q;    // [M_total] row of Q_prev to update, -1 for an uploader whose Q_m lives in another context
  float* up_R;      // [M_total] their radii
  float* up_s;      // [M] their grid steps 2 tau R
  double* ring;     // [D] circular
  float* xi;        // [D]
  double* loss_m;   // [M]
  DevScalars* sc;
  // scratch for the fixed-order two-stage reductions
  double* part_q;   // [M][kMaxSweepBlocksPerWorker][2]
  double* part_d;   // [agg blocks]  partial ||alpha grad||^2
  double* part_t;   // [agg blocks]  partial ||theta^{k+1}||^2
  // trace (rows = iterations of the current laq_step call)
  int trace_cap;
  uint8_t* t_skip;
  float* t_R;
  double *t_ndq, *t_neps, *t_rhs, *t_d2, *t_loss;
  int32_t* t_up;
  // synthetic gradient stream
  uint32_t seed_lo, seed_hi;
  int batch;                 // 0: full local gradients; > 0: minibatch size per worker
  uint32_t zero;             // always 0; opaque to the compiler (used to order a store after a load)
  uint32_t starve;           // test hook (laq_tune "starve_copies"): one loader issues no copies, see laq.h
  float cz, eta0;
  // shards
  long long Ntot;            // samples of ALL workers (the 1/N of the global loss)
  long long Nloc;            // samples resident in this context (= Ntot unless the workers are spread over contexts)
  const float* const* X;     // device array of M device pointers
  const int32_t* const* y;   // device array of M device pointers
  const long long* N;        // device [M]
  // model scratch
  float* gpart;              // gradient partials [M][gbpw][ps]
  double* lpart;             // loss partials [M][gbpw]
  uint32_t* cnt_grad;        // [M] tickets
  const SparseShard* sp;     // device [M], LAQ_FLAG_SPARSE_X only
  uint16_t* w1b;             // network, tensor-core path: bf16 copy of theta's first w1b_n coordinates (W1), kept up
  long long w1b_n;           // to date by the theta step (null / 0 otherwise)
};

#ifdef __CUDACC__
// 32-bit finalizer of MurmurHash3 (public domain)
__device__ __forceinline__ uint32_t fmix32(uint32_t x) {
  x ^= x >> 16;
  x *= 0x85ebca6bu;
  x ^= x >> 13;
  x *= 0xc2b2ae35u;
  x ^= x >> 16;
  return x;
}

// Packed fp32 pairs: sm_100 executes two fused multiply-adds per lane in one instruction.
__device__ __forceinline__ unsigned long long ffma2(unsigned long long a, unsigned long long b, unsigned long long c) {
  unsigned long long d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ void unpack2(unsigned long long v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ unsigned long long pack2(float lo, float hi) {
  unsigned long long v;
  asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "f"(lo), "f"(hi));
  return v;
}

// ---- bulk asynchronous copies global -> shared, completion counted in bytes on an mbarrier ---------------------
// Source, destination and size are multiples of 16 bytes.  Every wait is bounded: after kRingWaitLimit polls it
// returns false; the caller records kErrRingWait in DevScalars::err, stops using the ring, and gives the copies
// still in flight the same bounded time to land before it leaves.
constexpr uint32_t kRingWaitLimit = 1u << 22;
constexpr uint32_t kStarvedWaitLimit = 1u << 10;   // polls of a consumer whose loader was told to issue nothing
constexpr uint32_t kErrRingWait = 16u;             // bit of DevScalars::err: a wait on a staged tile ran out

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void ring_bar_init(uint32_t bar) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void ring_expect(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void ring_copy(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
// one copy that is the whole content of a stage
__device__ __forceinline__ void ring_fetch(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  ring_expect(bar, bytes);
  ring_copy(dst, src, bytes, bar);
}
__device__ __forceinline__ bool ring_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded: false once the limit is reached (the caller records it and stops using the ring).
__device__ __forceinline__ bool ring_wait(uint32_t bar, uint32_t parity, uint32_t limit = kRingWaitLimit) {
  for (uint32_t it = 0; it < limit; ++it) {
    if (ring_try_wait(bar, parity)) return true;
    if (it > 64) __nanosleep(64);
  }
  return false;
}

// Rows of worker m that enter the local gradient of the iteration in progress: all N_m rows, or (minibatch
// variant of Sec. 4) the cyclic window of B_m = min(batch, N_m) consecutive rows whose start is drawn from
// (seed, m, k): rows [start, start + len_a) followed by rows [0, len_b).
struct RowWindow {
  long long start, len_a, len_b;
  long long tiles_a = 0;   // set by tiles(): tiles of the first piece (a 64-bit division, done once per kernel)
  __device__ __forceinline__ long long tiles(int rows) {
    tiles_a = (len_a + rows - 1) / rows;
    return tiles_a + (len_b + rows - 1) / rows;
  }
  // tile t of `rows` rows -> first row and number of rows (tiles never straddle the wrap); tiles(rows) comes first
  __device__ __forceinline__ void tile(long long t, int rows, long long& r0, int& nr) const {
    long long left;
    if (t < tiles_a) {
      r0 = start + t * rows;
      left = len_a - t * rows;
    } else {
      t -= tiles_a;
      r0 = t * rows;
      left = len_b - t * rows;
    }
    nr = (int)(left < rows ? left : rows);
  }
  __device__ __forceinline__ bool contains(long long r) const {
    return (r >= start && r < start + len_a) || r < len_b;
  }
};

__device__ __forceinline__ RowWindow row_window(const Params& P, int m) {
  const long long n = P.N[m];
  RowWindow w;
  if (P.batch <= 0 || P.batch >= n) {
    w.start = 0;
    w.len_a = n;
    w.len_b = 0;
    return w;
  }
  const uint32_t k = (uint32_t)(P.sc->k + 1ull);
  const uint32_t gid = (uint32_t)(P.m_first + P.m_stride * m);   // the worker's global index
  const uint32_t h = fmix32(fmix32(P.seed_lo + k) ^ (P.seed_hi + 0x9e3779b9u * (gid + 1u)));
  w.start = (long long)(h % (uint32_t)n);
  const long long to_end = n - w.start;
  w.len_a = P.batch < to_end ? P.batch : to_end;
  w.len_b = P.batch - w.len_a;
  return w;
}

// N_m / B_m: what the sum over the window is scaled by so that it estimates the sum over the shard
__device__ __forceinline__ double batch_scale(const Params& P, int m) {
  const long long n = P.N[m];
  return (P.batch <= 0 || P.batch >= n) ? 1.0 : (double)n / (double)P.batch;
}
#endif

struct LaunchShape {
  int sweep_threads = 128;
  int sweep_blocks_per_sm = 64;    // many small blocks: the last partial wave costs a few percent at most
  int agg_threads = 256;
  int agg_blocks_per_sm = 32;
  int grad_blocks_per_worker = 0;  // 0 = automatic
};

// kernels' host-side launchers (each returns the number of kernels it launched)
bool generated_in_sweeps(const Params& P);
int launch_synth_fill(const Params& P, cudaStream_t st);
int launch_radius(const Params& P, const LaunchShape& ls, cudaStream_t st);
bool small_iteration_applies(const Params& P);
int launch_small_iteration(const Params& P, int gbpw_finalize, cudaStream_t st);
int launch_innovation_trigger(const Params& P, const LaunchShape& ls, cudaStream_t st);
int launch_quantize_trigger(const Params& P, const LaunchShape& ls, cudaStream_t st);
int launch_aggregate(const Params& P, const LaunchShape& ls, cudaStream_t st);
int launch_merge_uploads(const Params& P, int n, const int32_t* d_m, const float* d_R, cudaStream_t st);
int launch_grad_logreg(const Params& P, const LaunchShape& ls, int gbpw, cudaStream_t st);
int launch_grad_softmax(const Params& P, const LaunchShape& ls, int gbpw, cudaStream_t st);
int launch_grad_finalize(const Params& P, int gbpw, const double* theta_sq, bool with_radius, cudaStream_t st);
bool softmax_classes_supported(int C);
bool sparse_shape_ok(int F, int C);
size_t sparse_region_bytes(long long n, int F);
int sparse_blocks_per_worker(const long long* N, int M);
int launch_grad_softmax_sparse(const Params& P, int gbpw, cudaStream_t st);
int grad_tiles_per_worker(int model, int F, int C, long long n_max);
int grad_blocks_per_sm(int model, int F, int C);

// one-hidden-layer ReLU network (laq_grad_mlp.cu)
struct MlpPlan {
  void* scratch = nullptr;
  int ready = 0;
};
const char* mlp_check_shape(int F, int H, int C);   // null if supported, else the reason
size_t mlp_scratch_bytes(const laq_config& c);
laq_status mlp_setup(MlpPlan& mp, const Params& P, const long long* N_host, void* scratch, cudaStream_t st);
laq_status mlp_set_row_offsets(MlpPlan& mp, const long long* N_host, int M, cudaStream_t st);
laq_status mlp_setup_tensor_path(MlpPlan& mp, const Params& P, cudaStream_t st);
int mlp_convert_shard(MlpPlan& mp, const Params& P, int m, const float* X, long long n, long long row_offset,
                      cudaStream_t st);
int mlp_launch_gradients(MlpPlan& mp, const Params& P, const double* theta_sq, cudaStream_t st);
void* mlp_w1_copy(const MlpPlan& mp);   // the bf16 copy of W1 that the tensor-core path reads (null: plain path)
int mlp_refresh_w1_copy(MlpPlan& mp, const Params& P, cudaStream_t st);   // after theta was set from outside
void mlp_teardown(MlpPlan& mp);
laq_status sparse_build(int m, const float* X, long long n, int F, void* region, SparseShard* desc_dev, cudaStream_t st,
                        std::string* err);
int sweep_blocks_per_worker(const Params& P, const LaunchShape& ls);
int sweep_tile_groups();
int launch_theta_sq(const Params& P, cudaStream_t st);
int aggregate_blocks(const Params& P, const LaunchShape& ls);

}  // namespace laq
