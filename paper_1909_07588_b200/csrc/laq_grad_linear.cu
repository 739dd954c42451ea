// Step 1 of the LAQ iteration for the two linear models of the paper's supplement
// ("Simulation details"): worker m's gradient of f_m at theta^k over its resident shard,
//   g_m = (1/N) sum_n grad CE(x_{m,n}; theta) + (N_m/N) lambda theta,
// as a skinny contraction that reads every sample once: a block stages a tile of consecutive rows
// (contiguous in memory) in shared memory, computes the residuals (sigma(z) - y, or softmax - onehot)
// and accumulates residual^T x in registers across its tiles.  Block partials are combined in a
// fixed order by grad_finalize_kernel, which also adds the regulariser share (and takes the quantizer's radius).
#include <cuda_pipeline.h>

#include "laq_internal.cuh"

namespace laq {

namespace {

__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_sum_f(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Copy `count` consecutive floats global -> shared; where alignment allows as asynchronous 16-byte copies, so
// that every thread has all of its copies in flight at once.  Ends with the copies complete for this thread;
// the caller's __syncthreads() makes them visible to the block.
__device__ __forceinline__ void stage_rows(const float* __restrict__ src, float* dst, int count) {
  if ((reinterpret_cast<uintptr_t>(src) & 15u) == 0) {
    const int n4 = count >> 2;
    for (int i = threadIdx.x; i < n4; i += blockDim.x) __pipeline_memcpy_async(dst + 4 * i, src + 4 * i, 16);
    __pipeline_commit();
    for (int i = (n4 << 2) + threadIdx.x; i < count; i += blockDim.x) dst[i] = __ldg(src + i);
    __pipeline_wait_prior(0);
  } else {
    for (int i = threadIdx.x; i < count; i += blockDim.x) dst[i] = __ldg(src + i);
  }
}

// ------------------------------------------------------------------------------------------------
// binary logistic regression, F <= 256
// ------------------------------------------------------------------------------------------------
constexpr int kLrThreads = 256;
constexpr int kLrMaxRows = 256;   // rows per tile: at most one per thread, fewer for wide rows

__global__ void __launch_bounds__(kLrThreads) grad_logreg_kernel(const Params P, int gbpw, int rows) {
  extern __shared__ __align__(16) float smem[];
  const int F = P.F, m = blockIdx.y, t = threadIdx.x;
  float* xs = smem;                          // [rows][F]
  float* ths = xs + rows * F;                // [F]
  float* rs = ths + ((F + 3) & ~3);          // [rows]
  float* red = rs + kLrMaxRows;              // [kLrThreads]
  __shared__ double shd[32];
  const float* __restrict__ X = P.X[m];
  const int32_t* __restrict__ y = P.y[m];
  for (int f = t; f < F; f += blockDim.x) ths[f] = P.theta[f];
  const int S = kLrThreads / F;              // row slices handled in parallel in the second phase
  const bool active = t < S * F;
  const int f_own = t % F, slice = t / F;
  float acc = 0.f;
  double loss = 0.0;
  RowWindow win = row_window(P, m);
  const long long ntiles = win.tiles(rows);
  for (long long tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
    long long r0;
    int nr;
    win.tile(tile, rows, r0, nr);
    __syncthreads();
    stage_rows(X + r0 * F, xs, nr * F);
    __syncthreads();
    if (t < nr) {
      const float* xr = xs + t * F;
      float z = 0.f;
      for (int f = 0; f < F; ++f) z = fmaf(xr[f], ths[f], z);
      const float yv = (float)y[r0 + t];
      float sig, sp;
      if (z >= 0.f) {
        const float e = expf(-z);
        sig = 1.0f / (1.0f + e);
        sp = z + log1pf(e);
      } else {
        const float e = expf(z);
        sig = e / (1.0f + e);
        sp = log1pf(e);
      }
      rs[t] = sig - yv;
      loss += (double)(sp - yv * z);
    }
    __syncthreads();
    if (active)
      for (int r = slice; r < nr; r += S) acc = fmaf(rs[r], xs[r * F + f_own], acc);  // address = (r-slice) F + t
  }
  __syncthreads();
  red[t] = active ? acc : 0.f;
  __syncthreads();
  if (t < F) {
    float s = 0.f;
    for (int sl = 0; sl < S; ++sl) s += red[sl * F + t];
    P.gpart[((long long)m * gbpw + blockIdx.x) * P.ps + t] = s;
  }
  loss = warp_sum_d(loss);
  if ((t & 31) == 0) shd[t >> 5] = loss;
  __syncthreads();
  if (t == 0) {
    double l = 0.0;
    for (int i = 0; i < kLrThreads / 32; ++i) l += shd[i];
    P.lpart[(long long)m * gbpw + blockIdx.x] = l;
  }
}

// Issue the copies of `count` consecutive floats global -> shared without waiting for them (the caller commits the
// group and waits later); sources that are not 16-byte aligned are copied with plain loads.
__device__ __forceinline__ void stage_rows_async(const float* __restrict__ src, float* dst, int count) {
  if ((reinterpret_cast<uintptr_t>(src) & 15u) == 0) {
    const int n4 = count >> 2;
    for (int i = threadIdx.x; i < n4; i += blockDim.x) __pipeline_memcpy_async(dst + 4 * i, src + 4 * i, 16);
    for (int i = (n4 << 2) + threadIdx.x; i < count; i += blockDim.x) dst[i] = __ldg(src + i);
  } else {
    for (int i = threadIdx.x; i < count; i += blockDim.x) dst[i] = __ldg(src + i);
  }
}

// The same for an even number of features.  Tiles of 128 rows in a two-deep ring of shared-memory buffers (the next
// tile arrives while the current one is worked on); 8-byte reads (rows start 8-byte aligned); two threads per row in
// the first phase (each half of the features, joined through shared memory), two features per thread in the second, so that a
// residual read from shared memory feeds two multiply-adds.  About a third of the instructions of the kernel above.
constexpr int kLr2Rows = 128;

// FT > 0 fixes the feature count at compile time (54 and 22, the shapes of the paper's two logistic-regression
// tests): offsets become immediates, the score loop is straight-line code and its half of theta sits in registers.
// FT = 0 reads the count from the parameters.  The arithmetic and its order are the same in both forms.
template <int FT>
__global__ void __launch_bounds__(kLrThreads) grad_logreg_pair_kernel(const Params P, int gbpw) {
  extern __shared__ __align__(16) float smem[];
  const int F = FT > 0 ? FT : P.F, F2 = F >> 1, m = blockIdx.y, t = threadIdx.x;
  float* xs0 = smem;                         // [2][128][F]
  float* ths = xs0 + 2 * kLr2Rows * F;       // [F]
  float* rs = ths + ((F + 3) & ~3);          // [128]
  float* red = rs + kLr2Rows;                // [2][kLrThreads]
  __shared__ double shd[32];
  __shared__ float zpart[kLr2Rows];
  const float* __restrict__ X = P.X[m];
  const int32_t* __restrict__ y = P.y[m];
  const int S = kLrThreads / F2;             // row slices handled in parallel in the second phase
  const bool active = t < S * F2;
  const int j_own = t % F2, slice = t / F2;
  const int row = t & (kLr2Rows - 1), half = t >> 7, fh = (F2 + 1) >> 1;   // first phase: half of the features of a row
  const int f_lo = half * fh, f_hi = half ? F2 : fh;
  constexpr int kHalfPairs = FT > 0 ? (FT / 2 + 1) / 2 : 1;
  float2 thr[kHalfPairs];                    // FT > 0: this thread's half of theta, as pairs
  if constexpr (FT > 0) {
#pragma unroll
    for (int i = 0; i < kHalfPairs; ++i)
      thr[i] = f_lo + i < f_hi ? __ldg(reinterpret_cast<const float2*>(P.theta) + f_lo + i) : make_float2(0.f, 0.f);
  } else {
    for (int f = t; f < F; f += blockDim.x) ths[f] = P.theta[f];
  }
  float acc0 = 0.f, acc1 = 0.f;
  double loss = 0.0;
  RowWindow win = row_window(P, m);
  const long long ntiles = win.tiles(kLr2Rows);
  auto stage = [&](long long tile, float* xs) {
    long long r0;
    int nr;
    win.tile(tile, kLr2Rows, r0, nr);
    stage_rows_async(X + r0 * F, xs, nr * F);
  };
  int buf = 0;
  if ((long long)blockIdx.x < ntiles) stage(blockIdx.x, xs0);
  __pipeline_commit();
  for (long long tile = blockIdx.x; tile < ntiles; tile += gridDim.x, buf ^= 1) {
    long long r0;
    int nr;
    win.tile(tile, kLr2Rows, r0, nr);
    float* xs = xs0 + buf * kLr2Rows * F;
    __syncthreads();                                  // everybody is done with the buffer refilled below
    // the row's label, asked for now and used after the scores
    const int y_row = (half == 0 && row < nr) ? __ldg(y + r0 + row) : 0;
    if (tile + gridDim.x < ntiles) stage(tile + gridDim.x, xs0 + (buf ^ 1) * kLr2Rows * F);
    __pipeline_commit();
    __pipeline_wait_prior(1);                         // this tile's copies (the older group) have landed
    __syncthreads();
    {
      float z = 0.f;
      if (row < nr) {
        const float2* xr = reinterpret_cast<const float2*>(xs + row * F);
        if constexpr (FT > 0) {
          const float2* xh = xr + f_lo;
#pragma unroll
          for (int i = 0; i < kHalfPairs; ++i)
            if (i + 1 < kHalfPairs || f_lo + i < f_hi) {   // only the last pair of the second half can be missing
              const float2 x = xh[i];
              z = fmaf(x.x, thr[i].x, z);
              z = fmaf(x.y, thr[i].y, z);
            }
        } else {
          const float2* th2 = reinterpret_cast<const float2*>(ths);
#pragma unroll 4
          for (int f = f_lo; f < f_hi; ++f) {
            const float2 x = xr[f], th = th2[f];
            z = fmaf(x.x, th.x, z);
            z = fmaf(x.y, th.y, z);
          }
        }
      }
      if (half) zpart[row] = z;                       // warps 4-7: second half of the features
      __syncthreads();
      if (half == 0 && row < nr) {                    // warps 0-3: join the halves, residual and loss
        z = z + zpart[row];
        const float yv = (float)y_row;
        float sig, sp;
        if (z >= 0.f) {
          const float e = expf(-z);
          sig = 1.0f / (1.0f + e);
          sp = z + log1pf(e);
        } else {
          const float e = expf(z);
          sig = e / (1.0f + e);
          sp = log1pf(e);
        }
        rs[row] = sig - yv;
        loss += (double)(sp - yv * z);
      }
    }
    __syncthreads();
    if (active) {
      const float* px = xs + slice * F + 2 * j_own;
      const int step = S * F;
#pragma unroll 4
      for (int r = slice; r < nr; r += S, px += step) {
        const float2 x = *reinterpret_cast<const float2*>(px);
        const float rv = rs[r];
        acc0 = fmaf(rv, x.x, acc0);
        acc1 = fmaf(rv, x.y, acc1);
      }
    }
  }
  __pipeline_wait_prior(0);
  __syncthreads();
  red[t] = active ? acc0 : 0.f;
  red[kLrThreads + t] = active ? acc1 : 0.f;
  __syncthreads();
  if (t < F) {
    const float* rp = red + (t & 1) * kLrThreads + (t >> 1);
    float s = 0.f;
    for (int sl = 0; sl < S; ++sl) s += rp[sl * F2];
    P.gpart[((long long)m * gbpw + blockIdx.x) * P.ps + t] = s;
  }
  loss = warp_sum_d(loss);
  if ((t & 31) == 0) shd[t >> 5] = loss;
  __syncthreads();
  if (t == 0) {
    double l = 0.0;
    for (int i = 0; i < kLrThreads / 32; ++i) l += shd[i];
    P.lpart[(long long)m * gbpw + blockIdx.x] = l;
  }
}

// ------------------------------------------------------------------------------------------------
// Binary logistic regression with F = 54 or 22 features (the shapes of the paper's two logistic tests; F / 2 odd).
// A block is one loader warp and eight worker warps around a ring of kLwStages shared-memory stages of 128
// consecutive rows.  The loader asks the copy engine for a whole tile with ONE request (cp.async.bulk, 128 F floats,
// completion counted in bytes on the stage's "full" mbarrier); few large requests matter: an SM starts a bulk copy
// only about every 100 ns.  A worker warp waits for the stage, works on its 16 rows of the tile and arrives on the
// stage's "empty" mbarrier, on which the loader waits before it refills the stage: no block-wide barrier in the
// loop, every wait bounded.
//   scores     lane = (row, half): 8-byte reads of half of its row (row pitch F floats: the 16 lanes of a half warp
//              hit 32 different banks), that half of theta in registers; the halves meet by one shuffle;
//   gradient   lane = feature pair: acc += residual[row] x[row][pair] over the warp's 16 rows, the residual fetched
//              by a shuffle, the pair by one conflict-free 8-byte read.
// Rows start 8-byte aligned (F even).  A tile that starts 8 bytes past a 16-byte boundary (minibatch windows that
// begin at an odd row) is placed 8 bytes into its stage, so that the bulk copy runs between 16-byte boundaries on
// both sides; its first two floats, and the up to three floats that follow the last whole 16 bytes of a tile (the
// last rows of a shard), are copied by lanes of the loader warp with plain loads before the request goes out.
// ------------------------------------------------------------------------------------------------
constexpr int kLwWarps = 8;                       // worker warps
constexpr int kLwThreads = 32 * (kLwWarps + 1);
constexpr int kLwRows = 128;                      // rows per tile
constexpr int kLwWarpRows = kLwRows / kLwWarps;   // 16
constexpr int kLwStages = 3;

static size_t logreg_warp_smem(int F) { return (size_t)kLwStages * (kLwRows * F + 4) * sizeof(float); }
static bool logreg_warp_path(int F) { return F == 54 || F == 22; }

template <int FT>
__global__ void __launch_bounds__(kLwThreads) grad_logreg_ring_kernel(const Params P, int gbpw) {
  static_assert((FT & 3) == 2 && FT <= 64, "F / 2 must be odd and fit one lane per feature pair");
  constexpr int F2 = FT / 2, FH = (F2 + 1) / 2;    // pairs per row; pairs of the first half
  constexpr uint32_t kTileFloats = kLwRows * FT + 4;   // 16 bytes of slack: a tile may sit 8 bytes into its stage
  extern __shared__ __align__(128) float smem[];
  __shared__ __align__(8) unsigned long long bars[2 * kLwStages];
  __shared__ float red[kLwWarps][FT];
  __shared__ double shd[kLwWarps];
  const int m = blockIdx.y, t = threadIdx.x, lane = t & 31, w = t >> 5;
  const float* __restrict__ X = P.X[m];
  const int32_t* __restrict__ y = P.y[m];
  const uint32_t full_a = smem_addr(bars), empty_a = full_a + 8 * kLwStages;
  if (t == 0) {
    for (int st = 0; st < kLwStages; ++st) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(full_a + 8 * st) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(empty_a + 8 * st), "r"(kLwWarps) : "memory");
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  RowWindow win = row_window(P, m);
  const int ntiles = (int)win.tiles(kLwRows);                    // N_m < 2^31
  const int n_my = ntiles > (int)blockIdx.x ? (ntiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
  float acc0 = 0.f, acc1 = 0.f;
  double loss = 0.0;
  if (w == kLwWarps) {
    // ---- loader warp
    uint32_t st = 0, round = 0;
    for (int i = 0; i < n_my; ++i) {
      long long r0;
      int nr;
      win.tile((long long)blockIdx.x + (long long)i * gridDim.x, kLwRows, r0, nr);
      // the workers are done with what the stage held (passes at once in the first round)
      if (!__all_sync(0xffffffffu, ring_wait(empty_a + 8 * st, (round & 1u) ^ 1u))) {
        if (lane == 0) atomicOr(&P.sc->err, kErrRingWait);
        break;
      }
      const float* src = X + r0 * FT;
      const int total = nr * FT;                                             // floats of the tile
      const int shift = (int)((reinterpret_cast<uintptr_t>(src) & 15u) >> 2);   // 0 or 2 floats
      float* dst = smem + st * kTileFloats + shift;                          // row 0 of the tile in the stage
      const int head = shift ? 2 : 0;                                        // floats before the first 16-byte boundary
      const int body = (total - head) & ~3;                                  // whole 16-byte units
      if (lane < head) dst[lane] = __ldg(src + lane);
      if (lane >= 8 && lane - 8 < total - head - body) dst[head + body + lane - 8] = __ldg(src + head + body + lane - 8);
      __syncwarp();
      if (lane == 0) {
        if (body > 0) {
          ring_fetch(smem_addr(dst + head), src + head, (uint32_t)body * 4u, full_a + 8 * st);
        } else {
          asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(full_a + 8 * st) : "memory");
        }
      }
      if (++st == (uint32_t)kLwStages) {
        st = 0;
        ++round;
      }
    }
  } else {
    // ---- worker warps
    const int row = lane & 15, half = lane >> 4;
    constexpr int kMaxHalf = FH;                   // the second half has F2 - FH = FH - 1 pairs
    float2 thr[kMaxHalf];
#pragma unroll
    for (int j = 0; j < kMaxHalf; ++j)
      thr[j] = (half == 0 || j < F2 - FH) ? __ldg(reinterpret_cast<const float2*>(P.theta) + half * FH + j) : make_float2(0.f, 0.f);
    uint32_t st = 0, round = 0;
    for (int i = 0; i < n_my; ++i) {
      long long r0;
      int nr;
      win.tile((long long)blockIdx.x + (long long)i * gridDim.x, kLwRows, r0, nr);
      const int wr0 = w * kLwWarpRows;               // this warp's rows of the tile: wr0 .. wr0 + 15
      const int wnr = nr - wr0 < kLwWarpRows ? (nr - wr0 > 0 ? nr - wr0 : 0) : kLwWarpRows;
      const int y_row = (half == 0 && row < wnr) ? __ldg(y + r0 + wr0 + row) : 0;   // asked for now, used after the scores
      if (!__all_sync(0xffffffffu, ring_wait(full_a + 8 * st, round & 1u))) {
        if (lane == 0) atomicOr(&P.sc->err, kErrRingWait);
        break;
      }
      const int shift = (int)((reinterpret_cast<uintptr_t>(X + r0 * FT) & 15u) >> 2);   // as the loader placed the tile
      const float* xs = smem + st * kTileFloats + shift + wr0 * FT;
      // ---- scores: lane = (row, half of the features)
      float res = 0.f;
      {
        float z0 = 0.f, z1 = 0.f;
        if (row < wnr) {
          const float2* xr = reinterpret_cast<const float2*>(xs + row * FT) + half * FH;
#pragma unroll
          for (int j = 0; j < kMaxHalf; ++j)
            if (j < F2 - FH || half == 0) {          // only the last pair of the second half is missing
              const float2 a = xr[j];
              z0 = fmaf(a.x, thr[j].x, z0);
              z1 = fmaf(a.y, thr[j].y, z1);
            }
        }
        float z = z0 + z1;
        z += __shfl_xor_sync(0xffffffffu, z, 16);    // both halves now hold the row's score (same sum in both)
        if (half == 0 && row < wnr) {
          const float yv = (float)y_row;
          float sig, sp;
          if (z >= 0.f) {
            const float e = expf(-z);
            sig = 1.0f / (1.0f + e);
            sp = z + log1pf(e);
          } else {
            const float e = expf(z);
            sig = e / (1.0f + e);
            sp = log1pf(e);
          }
          res = sig - yv;
          loss += (double)(sp - yv * z);
        }
      }
      // ---- gradient: lane = feature pair (rows beyond a short tile are skipped: the stage may hold anything there)
      {
        const float2* xc = reinterpret_cast<const float2*>(xs) + (lane < F2 ? lane : 0);
        float a0 = 0.f, a1 = 0.f, b0 = 0.f, b1 = 0.f;
        if (wnr == kLwWarpRows) {
#pragma unroll
          for (int r = 0; r < kLwWarpRows; r += 2) {
            const float ra = __shfl_sync(0xffffffffu, res, r), rb = __shfl_sync(0xffffffffu, res, r + 1);
            const float2 xa = xc[r * F2], xb = xc[(r + 1) * F2];
            a0 = fmaf(ra, xa.x, a0);
            a1 = fmaf(ra, xa.y, a1);
            b0 = fmaf(rb, xb.x, b0);
            b1 = fmaf(rb, xb.y, b1);
          }
        } else {
          for (int r = 0; r < wnr; ++r) {
            const float ra = __shfl_sync(0xffffffffu, res, r);
            const float2 xa = xc[r * F2];
            a0 = fmaf(ra, xa.x, a0);
            a1 = fmaf(ra, xa.y, a1);
          }
        }
        acc0 += a0 + b0;
        acc1 += a1 + b1;
      }
      __syncwarp();                                  // every lane has read the stage
      if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(empty_a + 8 * st) : "memory");
      if (++st == (uint32_t)kLwStages) {
        st = 0;
        ++round;
      }
    }
    if (lane < F2) {
      red[w][2 * lane] = acc0;
      red[w][2 * lane + 1] = acc1;
    }
    loss = warp_sum_d(loss);
    if (lane == 0) shd[w] = loss;
  }
  // ---- block partial: the warps' sums in warp order.  If a wait ran out some warps stopped early; the error word
  // is set and nothing of this iteration is used.
  __syncthreads();
  if (t < FT) {
    float sum = red[0][t];
#pragma unroll
    for (int k = 1; k < kLwWarps; ++k) sum += red[k][t];
    P.gpart[((long long)m * gbpw + blockIdx.x) * P.ps + t] = sum;
  }
  if (t == 0) {
    double l = 0.0;
    for (int k = 0; k < kLwWarps; ++k) l += shd[k];
    P.lpart[(long long)m * gbpw + blockIdx.x] = l;
  }
}

// ------------------------------------------------------------------------------------------------
// C-class softmax regression, F <= 1024
// ------------------------------------------------------------------------------------------------
constexpr int kSmThreads = 256;
constexpr int kSmRows = 16;
constexpr int kSmMaxJ = 4;  // features per thread: F <= kSmMaxJ * kSmThreads

template <int C>
__global__ void __launch_bounds__(kSmThreads) grad_softmax_kernel(const Params P, int gbpw) {
  extern __shared__ __align__(16) float smem[];
  const int F = P.F, m = blockIdx.y, t = threadIdx.x, lane = t & 31, w = t >> 5;
  float* xs = smem;                 // [kSmRows][F]
  float* res = xs + kSmRows * F;    // [kSmRows][C]
  __shared__ double shd[32];
  const float* __restrict__ X = P.X[m];
  const int32_t* __restrict__ y = P.y[m];
  const float* __restrict__ theta = P.theta;
  float acc[kSmMaxJ][C];
#pragma unroll
  for (int j = 0; j < kSmMaxJ; ++j)
#pragma unroll
    for (int c = 0; c < C; ++c) acc[j][c] = 0.f;
  double loss = 0.0;
  RowWindow win = row_window(P, m);
  const long long ntiles = win.tiles(kSmRows);
  for (long long tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
    long long r0;
    int nr;
    win.tile(tile, kSmRows, r0, nr);
    __syncthreads();
    stage_rows(X + r0 * F, xs, nr * F);
    __syncthreads();
    // phase 1: a warp per row computes the C scores, the softmax and the residual
    for (int r = w; r < nr; r += kSmThreads / 32) {
      float z[C];
#pragma unroll
      for (int c = 0; c < C; ++c) z[c] = 0.f;
      const float* xr = xs + r * F;
      for (int f = lane; f < F; f += 32) {
        const float x = xr[f];
#pragma unroll
        for (int c = 0; c < C; ++c) z[c] = fmaf(x, __ldg(theta + c * F + f), z[c]);
      }
#pragma unroll
      for (int c = 0; c < C; ++c) z[c] = warp_sum_f(z[c]);
      float zmax = z[0];
#pragma unroll
      for (int c = 1; c < C; ++c) zmax = fmaxf(zmax, z[c]);
      float e[C], sum = 0.f;
#pragma unroll
      for (int c = 0; c < C; ++c) {
        e[c] = expf(z[c] - zmax);
        sum += e[c];
      }
      const int yv = y[r0 + r];
      const float inv = 1.0f / sum;
      float zy = 0.f;
#pragma unroll
      for (int c = 0; c < C; ++c) {
        if (c == yv) zy = z[c];
        if (lane == 0) res[r * C + c] = e[c] * inv - (c == yv ? 1.f : 0.f);
      }
      if (lane == 0) loss += (double)((zmax + logf(sum)) - zy);
    }
    __syncthreads();
    // phase 2: thread t owns features t, t + 256, ...; residuals are broadcast from shared memory
    for (int r = 0; r < nr; ++r) {
      float rr[C];
#pragma unroll
      for (int c = 0; c < C; ++c) rr[c] = res[r * C + c];
#pragma unroll
      for (int j = 0; j < kSmMaxJ; ++j) {
        const int f = t + j * kSmThreads;
        if (f < F) {
          const float x = xs[r * F + f];
#pragma unroll
          for (int c = 0; c < C; ++c) acc[j][c] = fmaf(rr[c], x, acc[j][c]);
        }
      }
    }
  }
  float* gp = P.gpart + ((long long)m * gbpw + blockIdx.x) * P.ps;
#pragma unroll
  for (int j = 0; j < kSmMaxJ; ++j) {
    const int f = t + j * kSmThreads;
    if (f < F) {
#pragma unroll
      for (int c = 0; c < C; ++c) gp[c * F + f] = acc[j][c];
    }
  }
  loss = warp_sum_d(loss);
  __syncthreads();
  if (lane == 0) shd[w] = loss;
  __syncthreads();
  if (t == 0) {
    double l = 0.0;
    for (int i = 0; i < kSmThreads / 32; ++i) l += shd[i];
    P.lpart[(long long)m * gbpw + blockIdx.x] = l;
  }
}

// ------------------------------------------------------------------------------------------------
// C-class softmax regression, fast path: F a multiple of 4, F <= 896, C <= 12.
// 224 threads (7 warps), tiles of 8 rows in a two-deep ring of shared-memory buffers filled by asynchronous
// 16-byte copies (the next tile arrives while the current one is worked on); rows are padded to an odd number of
// 16-byte units so that 16-byte reads down a column of rows are conflict free; theta sits in shared memory too.
//   phase 1  lane = (row, feature group mod 4), warp = slice of the feature axis: scores from 16-byte reads of x
//            and broadcast 16-byte reads of theta; the 28 partials per (row, class) are summed through shared
//            memory, one thread per row then does softmax, residual and loss;
//   phase 2  thread = four consecutive features: acc[4][C] += residual[r][c] * x[r][f] over the tile's rows,
//            one 16-byte read of x and the broadcast residuals per row.
// Two blocks fit on an SM.
// ------------------------------------------------------------------------------------------------
constexpr int kS2Threads = 224;
constexpr int kS2Warps = 7;
constexpr int kS2Rows = 8;
constexpr int kS2Parts = 4 * kS2Warps;   // partial scores per (row, class)

// FT > 0 fixes the feature count at compile time (784, the 28 x 28 inputs of the paper's tests): every row and
// class offset is then an immediate and the loops have known trip counts; FT = 0 reads it from the parameters.
template <int C, int FT>
__global__ void __launch_bounds__(kS2Threads, 2) grad_softmax_tile_kernel(const Params P, int gbpw) {
  extern __shared__ __align__(16) float smem[];
  const int F = FT > 0 ? FT : P.F, F4 = F >> 2, FP4 = F4 | 1, FP = FP4 << 2;      // padded row stride (floats)
  const int m = blockIdx.y, t = threadIdx.x, lane = t & 31, w = t >> 5;
  float* xs0 = smem;                                 // [2][8][FP]
  float* ths = xs0 + 2 * kS2Rows * FP;               // [C][F]      theta
  float* plog = ths + C * F;                         // [28][8][C]  partial scores
  float* res = plog + kS2Parts * kS2Rows * C;        // [8][12][2]  residuals, each stored twice (packed pairs)
  __shared__ double shd[8];
  __shared__ float zs[kS2Rows * 12];                 // [8][C]      scores
  static_assert(kS2Rows * C <= kS2Threads, "one thread per (row, class)");
  const float* __restrict__ X = P.X[m];
  const int32_t* __restrict__ y = P.y[m];
  for (int i = t; i < C * F4; i += kS2Threads)
    reinterpret_cast<float4*>(ths)[i] = __ldg(reinterpret_cast<const float4*>(P.theta) + i);
  const int kw = (F4 + kS2Warps - 1) / kS2Warps;     // 16-byte groups of features per warp in phase 1
  const int row1 = lane & 7, par = lane >> 3;
  const int k_lo = w * kw + par, k_hi = min(F4, w * kw + kw);
  const bool owner = t < F4;                         // phase 2: thread t owns features 4t .. 4t+3
  unsigned long long acc01[C], acc23[C];            // packed pairs (features 4t, 4t+1) and (4t+2, 4t+3)
#pragma unroll
  for (int c = 0; c < C; ++c) acc01[c] = acc23[c] = 0ull;
  double loss = 0.0;
  RowWindow win = row_window(P, m);
  const long long ntiles = win.tiles(kS2Rows);

  // asynchronous staging of one tile: contiguous rows in global memory -> padded rows in shared memory
  auto stage = [&](long long tile, float* xs) {
    long long r0;
    int nr;
    win.tile(tile, kS2Rows, r0, nr);
    const float4* src = reinterpret_cast<const float4*>(X + r0 * F);
    const int cnt = nr * F4;
    int r = t / F4, k = t - r * F4;
    for (int i = t; i < kS2Rows * F4; i += kS2Threads) {
      float* dst = xs + r * FP + 4 * k;
      if (i < cnt)
        __pipeline_memcpy_async(dst, src + i, 16);
      else
        *reinterpret_cast<float4*>(dst) = make_float4(0.f, 0.f, 0.f, 0.f);
      k += kS2Threads;
      while (k >= F4) {
        k -= F4;
        ++r;
      }
    }
  };

  int buf = 0;
  if ((long long)blockIdx.x < ntiles) stage(blockIdx.x, xs0);
  __pipeline_commit();
  for (long long tile = blockIdx.x; tile < ntiles; tile += gridDim.x, buf ^= 1) {
    long long r0;
    int nr;
    win.tile(tile, kS2Rows, r0, nr);
    float* xs = xs0 + buf * kS2Rows * FP;
    __syncthreads();                                  // everybody is done with the buffer refilled below
    if (tile + gridDim.x < ntiles) stage(tile + gridDim.x, xs0 + (buf ^ 1) * kS2Rows * FP);
    __pipeline_commit();
    __pipeline_wait_prior(1);                         // this tile's copies (the older group) have landed
    __syncthreads();
    {  // phase 1 (packed pairs: the two halves of a score are added at the end)
      unsigned long long z2[C];
#pragma unroll
      for (int c = 0; c < C; ++c) z2[c] = 0ull;
      const ulonglong2* xr = reinterpret_cast<const ulonglong2*>(xs + row1 * FP);
      const ulonglong2* th2 = reinterpret_cast<const ulonglong2*>(ths);
      for (int k = k_lo; k < k_hi; k += 4) {
        const ulonglong2 x = xr[k];
#pragma unroll
        for (int c = 0; c < C; ++c) {
          const ulonglong2 th = th2[c * F4 + k];
          z2[c] = ffma2(x.x, th.x, z2[c]);
          z2[c] = ffma2(x.y, th.y, z2[c]);
        }
      }
#pragma unroll
      for (int c = 0; c < C; ++c) {
        float lo, hi;
        unpack2(z2[c], lo, hi);
        plog[((4 * w + par) * kS2Rows + row1) * C + c] = lo + hi;
      }
    }
    __syncthreads();
    if (t < kS2Rows * C) {  // one thread per (row, class): sum the 28 partial scores in a fixed order
      float s = 0.f;
#pragma unroll
      for (int ww = 0; ww < kS2Parts; ++ww) s += plog[ww * kS2Rows * C + t];
      zs[t] = s;
    }
    __syncthreads();
    if (t < kS2Rows) {  // one thread per row: softmax, residual, loss
      float z[C];
#pragma unroll
      for (int c = 0; c < C; ++c) z[c] = zs[t * C + c];
      float zmax = z[0];
#pragma unroll
      for (int c = 1; c < C; ++c) zmax = fmaxf(zmax, z[c]);
      float e[C], sum = 0.f;
#pragma unroll
      for (int c = 0; c < C; ++c) {
        e[c] = expf(z[c] - zmax);
        sum += e[c];
      }
      const bool live = t < nr;
      const int yv = live ? y[r0 + t] : -1;
      const float inv = 1.0f / sum;
      float zy = 0.f;
#pragma unroll
      for (int c = 0; c < C; ++c) {
        if (c == yv) zy = z[c];
        const float rv = live ? (e[c] * inv - (c == yv ? 1.f : 0.f)) : 0.f;
        res[(t * 12 + c) * 2] = rv;
        res[(t * 12 + c) * 2 + 1] = rv;
      }
      if (live) loss += (double)((zmax + logf(sum)) - zy);
    }
    __syncthreads();
    if (owner) {  // phase 2
      const float* xc = xs + 4 * t;
#pragma unroll 2
      for (int r = 0; r < kS2Rows; ++r) {             // rows beyond the shard hold zero residuals
        const ulonglong2 x = *reinterpret_cast<const ulonglong2*>(xc + r * FP);
        const ulonglong2* rp = reinterpret_cast<const ulonglong2*>(res + r * 24);
#pragma unroll
        for (int c = 0; c < C; c += 2) {
          const ulonglong2 rr = rp[c >> 1];           // (r_c, r_c), (r_c+1, r_c+1)
          acc01[c] = ffma2(rr.x, x.x, acc01[c]);
          acc23[c] = ffma2(rr.x, x.y, acc23[c]);
          if (c + 1 < C) {
            acc01[c + 1] = ffma2(rr.y, x.x, acc01[c + 1]);
            acc23[c + 1] = ffma2(rr.y, x.y, acc23[c + 1]);
          }
        }
      }
    }
  }
  __pipeline_wait_prior(0);
  float* gp = P.gpart + ((long long)m * gbpw + blockIdx.x) * P.ps;
  if (owner) {
#pragma unroll
    for (int c = 0; c < C; ++c) {
      float4 v;
      unpack2(acc01[c], v.x, v.y);
      unpack2(acc23[c], v.z, v.w);
      *reinterpret_cast<float4*>(gp + c * F + 4 * t) = v;
    }
  }
  loss = warp_sum_d(loss);
  __syncthreads();
  if (lane == 0) shd[w] = loss;
  __syncthreads();
  if (t == 0) {
    double l = 0.0;
    for (int i = 0; i < kS2Warps; ++i) l += shd[i];
    P.lpart[(long long)m * gbpw + blockIdx.x] = l;
  }
}

}  // namespace

// Combine the block partials of worker blockIdx.y in block order, scale by 1/N and add the
// worker's share (N_m/N) lambda theta of the regulariser; block 0 of each worker also writes the
// worker's loss term.  theta_sq = ||theta^k||^2 comes from the previous theta step.
// RADIUS: the kernel also takes the largest |g_m - Q_prev| of its coordinates (as unsigned bit patterns, which order
// like the floats and put inf and nan on top) into the worker's radius word of this iteration, so that the separate
// radius sweep is not launched: the gradient is in a register here anyway.
template <bool RADIUS>
__global__ void __launch_bounds__(256) grad_finalize_kernel(const Params P, int gbpw, const double* theta_sq) {
  const int m = blockIdx.y;
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const double inv_N = 1.0 / (double)P.Ntot;
  const double share = (double)P.N[m] / (double)P.Ntot;
  uint32_t mx = 0;
  if (i < P.p) {
    const float* gp = P.gpart + (long long)m * gbpw * P.ps + i;
    double s = 0.0;
    for (int blk = 0; blk < gbpw; ++blk) s += (double)gp[(long long)blk * P.ps];
    const double g = s * (inv_N * batch_scale(P, m)) + share * (double)P.lambda * (double)P.theta[i];
    const float gf = (float)g;
    P.g[(long long)m * P.ps + i] = gf;
    if (RADIUS) mx = __float_as_uint(__fsub_rn(gf, P.qp[(long long)m * P.ps + i])) & 0x7fffffffu;
  }
  if (RADIUS) {
    mx = __reduce_max_sync(0xffffffffu, mx);
    if ((threadIdx.x & 31) == 0 && mx != 0u) atomicMax(&P.Rbits[(P.sc->k & 1ull) * P.M + m], mx);   // order independent
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    double l = 0.0;
    for (int blk = 0; blk < gbpw; ++blk) l += P.lpart[(long long)m * gbpw + blk];
    P.loss_m[m] = l * (inv_N * batch_scale(P, m)) + share * 0.5 * (double)P.lambda * (*theta_sq);
  }
}

// ------------------------------------------------------------------------------------------------
// C-class softmax regression, wide path: feature count fixed at compile time (a multiple of 16), C <= 10.
// One block of 256 threads per SM; tiles of 24 rows in two shared-memory stages.  The eighth warp asks the copy
// engine for the next tile (one bulk copy per row into rows padded to an odd number of 16-byte units, completion
// counted in bytes on the stage's mbarrier, bounded waits) while warps 0-6 work on the current one:
//   scores     lane = (row group rg = lane mod 8, phase kp = lane / 8) owns rows rg, rg + 8, rg + 16 and, in each
//              trip, the 16-byte feature group 4 (w + 7 trip) + kp: three 16-byte reads of x, C broadcast reads of
//              theta, 6 C packed multiply-adds; the 28 partial scores per (row, class) go through shared memory;
//   softmax    one thread per (row, class), a row's classes in neighbouring lanes: sum of the partials in a fixed
//              order, maximum and sum of the row by shuffles (the same order in every lane of a row), residual, loss;
//              the row's label is asked for before the score product;
//   gradient   thread = four consecutive features: acc[4][C] += residual[r][c] x[r][f] over the tile's rows, as packed
//              pairs of classes: a row's residuals are read once as they lie (three broadcast reads, 40 bytes) and
//              each of the thread's four samples is doubled in a register.
// Every offset is an immediate and every loop has a known trip count.
// ------------------------------------------------------------------------------------------------
constexpr int kSwThreads = 256;
constexpr int kSwWarps = 7;
#ifndef LAQ_SW_RPL
#define LAQ_SW_RPL 3
#endif
#ifndef LAQ_SW_STAGES
#define LAQ_SW_STAGES 2
#endif
constexpr int kSwRpl = LAQ_SW_RPL;         // rows per lane in the score product
constexpr int kSwRows = 8 * kSwRpl;        // rows per tile
constexpr int kSwStages = LAQ_SW_STAGES;   // tiles in shared memory: one at work, the others on their way
constexpr int kSwParts = 4 * kSwWarps;

template <int C, int FT>
struct SwShape {
  static constexpr int F = FT, F4 = FT / 4, FP4 = F4 | 1, FP = FP4 * 4, QUADS = F4 / 4;
  static constexpr int ITERS = (QUADS + kSwWarps - 1) / kSwWarps;
  static constexpr int RC = kSwRows * C;
  // floats: stages of samples, theta, partial scores, residual pairs
  static constexpr size_t kFloats = kSwStages * (size_t)kSwRows * FP + (size_t)C * F + (size_t)kSwParts * RC + (size_t)kSwRows * 24;
  static_assert(FT % 16 == 0 && F4 <= kSwThreads, "feature groups: a thread per group, four groups per trip");
  static_assert(C >= 2 && C <= 10 && kSwRpl * C <= 32 && kSwThreads == 256, "a warp's lanes = its rows x classes");
};

template <int C, int FT>
__global__ void __launch_bounds__(kSwThreads, 1) grad_softmax_wide_kernel(const Params P, int gbpw) {
  using S = SwShape<C, FT>;
  constexpr int F = S::F, F4 = S::F4, FP = S::FP, RC = S::RC;
  extern __shared__ __align__(128) float smem[];
  float* xs0 = smem;                                  // [stages][rows][FP]
  float* ths = xs0 + kSwStages * kSwRows * FP;        // [C][F]
  float* plog = ths + C * F;                          // [28][24][C]
  float* res = plog + kSwParts * RC;                  // [rows][12] residuals (slots C .. 11 stay zero)
  __shared__ double shd[kSwThreads / 32];
  __shared__ __align__(8) unsigned long long bars[kSwStages];
  const int m = blockIdx.y, t = threadIdx.x, lane = t & 31, w = t >> 5;
  const float* __restrict__ X = P.X[m];
  const int32_t* __restrict__ y = P.y[m];
  const uint32_t bar_a = smem_addr(bars), xs_a = smem_addr(xs0);
  RowWindow win = row_window(P, m);
  const long long ntiles = win.tiles(kSwRows);

  // the producer warp asks for one tile: a copy per row, all counted on the stage's barrier
  auto request = [&](long long tile, int s) {
    long long r0;
    int nr;
    win.tile(tile, kSwRows, r0, nr);
    if (lane == 0) ring_expect(bar_a + 8 * s, (uint32_t)nr * F * 4u);
    __syncwarp();
    if (lane < nr)
      ring_copy(xs_a + (uint32_t)((s * kSwRows + lane) * FP) * 4u, X + (r0 + lane) * F, F * 4u, bar_a + 8 * s);
  };

  if (t == 0) {
    for (int s = 0; s < kSwStages; ++s) ring_bar_init(bar_a + 8 * s);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  for (int i = t; i < C * F4; i += kSwThreads)
    reinterpret_cast<float4*>(ths)[i] = __ldg(reinterpret_cast<const float4*>(P.theta) + i);
  for (int i = t; i < kSwRows * 12; i += kSwThreads) res[i] = 0.f;
  __syncthreads();
  if (w == kSwWarps)   // the first tiles of this block, one per stage but the last
    for (int s = 0; s < kSwStages - 1; ++s)
      if ((long long)blockIdx.x + (long long)s * gridDim.x < ntiles) request(blockIdx.x + (long long)s * gridDim.x, s);

  const bool owner = t < F4;                          // gradient phase: thread t owns features 4t .. 4t+3
  constexpr int CP = (C + 1) / 2;                     // pairs of classes (2k, 2k+1)
  unsigned long long acc[4][CP];                      // [feature][pair of classes]
#pragma unroll
  for (int f = 0; f < 4; ++f)
#pragma unroll
    for (int c = 0; c < CP; ++c) acc[f][c] = 0ull;
  double loss = 0.0;
  const int rg = lane & 7, kp = lane >> 3;
  // softmax phase: warp w owns rows kSwRpl w .. kSwRpl w + kSwRpl - 1, lane = (row within the warp, class)
  constexpr uint32_t kRcMask = (kSwRpl * C >= 32) ? 0xffffffffu : ((1u << (kSwRpl * C)) - 1u);
  const bool rc_lane = lane < kSwRpl * C;
  const int row_rc = kSwRpl * w + lane / C, cls_rc = lane % C;
  bool failed = false;
  int i = 0, s = 0;
  uint32_t parity = 0;
  long long tile = blockIdx.x;
  for (; tile < ntiles; tile += gridDim.x, ++i) {
    long long r0;
    int nr;
    win.tile(tile, kSwRows, r0, nr);
    const bool landed = ring_wait(bar_a + 8 * s, parity);
    // also: everybody is done with the previous tile, whose stage the next request overwrites
    if (!__syncthreads_and(landed ? 1 : 0)) {
      failed = true;
      break;
    }
    // the row's label, asked for now and used after the score product
    const int yv = (rc_lane && row_rc < nr) ? __ldg(y + r0 + row_rc) : -1;
    const long long ahead = tile + (long long)(kSwStages - 1) * gridDim.x;
    if (w == kSwWarps && ahead < ntiles) request(ahead, s == 0 ? kSwStages - 1 : s - 1);
    float* xs = xs0 + s * kSwRows * FP;
    if (nr < kSwRows) {   // rows beyond the window's piece: zeros (block-uniform branch)
      for (int j = t; j < (kSwRows - nr) * F4; j += kSwThreads) {
        const int r = nr + j / F4, k = j - (j / F4) * F4;
        *reinterpret_cast<float4*>(xs + r * FP + 4 * k) = make_float4(0.f, 0.f, 0.f, 0.f);
      }
      __syncthreads();
    }
    if (w < kSwWarps) {  // scores
      unsigned long long z2[kSwRpl][C];
#pragma unroll
      for (int r = 0; r < kSwRpl; ++r)
#pragma unroll
        for (int c = 0; c < C; ++c) z2[r][c] = 0ull;
      const float* xb = xs + rg * FP + 4 * kp;
      const float* tb = ths + 4 * kp;
#pragma unroll
      for (int it = 0; it < S::ITERS; ++it) {
        const int q = w + kSwWarps * it;
        if (S::QUADS % kSwWarps == 0 || q < S::QUADS) {
          ulonglong2 x[kSwRpl];
#pragma unroll
          for (int r = 0; r < kSwRpl; ++r) x[r] = *reinterpret_cast<const ulonglong2*>(xb + 16 * q + 8 * r * FP);
#pragma unroll
          for (int c = 0; c < C; ++c) {
            const ulonglong2 th = *reinterpret_cast<const ulonglong2*>(tb + c * F + 16 * q);
#pragma unroll
            for (int r = 0; r < kSwRpl; ++r) z2[r][c] = ffma2(x[r].x, th.x, z2[r][c]);
#pragma unroll
            for (int r = 0; r < kSwRpl; ++r) z2[r][c] = ffma2(x[r].y, th.y, z2[r][c]);
          }
        }
      }
      float* pl = plog + ((4 * w + kp) * kSwRows + rg) * C;
#pragma unroll
      for (int r = 0; r < kSwRpl; ++r)
#pragma unroll
        for (int c = 0; c < C; ++c) {
          float lo, hi;
          unpack2(z2[r][c], lo, hi);
          pl[8 * r * C + c] = lo + hi;
        }
    }
    __syncthreads();
    if (rc_lane) {  // one thread per (row, class); the classes of a row sit in neighbouring lanes of one warp
      float z = 0.f;
#pragma unroll
      for (int pp = 0; pp < kSwParts; ++pp) z += plog[pp * RC + row_rc * C + cls_rc];   // fixed order
      // every lane of a row reads the row's C values in the same order: identical maximum and sum in all of them
      const int lane0 = lane - cls_rc;
      float zmax = __shfl_sync(kRcMask, z, lane0);
#pragma unroll
      for (int c = 1; c < C; ++c) zmax = fmaxf(zmax, __shfl_sync(kRcMask, z, lane0 + c));
      const float e = expf(z - zmax);
      float sum = 0.f;
#pragma unroll
      for (int c = 0; c < C; ++c) sum += __shfl_sync(kRcMask, e, lane0 + c);
      const float zy = __shfl_sync(kRcMask, z, lane0 + (yv >= 0 ? yv : 0));
      const bool live = row_rc < nr;
      const float inv = 1.0f / sum;
      const float rv = live ? (e * inv - (cls_rc == yv ? 1.f : 0.f)) : 0.f;
      res[row_rc * 12 + cls_rc] = rv;
      if (live && cls_rc == 0) loss += (double)((zmax + logf(sum)) - zy);
    }
    __syncthreads();
    if (owner) {  // gradient
      const float* xc = xs + 4 * t;
#pragma unroll 4
      for (int r = 0; r < kSwRows; ++r) {             // rows beyond the piece hold zero residuals and zero samples
        const float4 x = *reinterpret_cast<const float4*>(xc + r * FP);
        const unsigned long long xx[4] = {pack2(x.x, x.x), pack2(x.y, x.y), pack2(x.z, x.z), pack2(x.w, x.w)};
        unsigned long long rr[6];                     // (r_0, r_1), (r_2, r_3), ...
        {
          const ulonglong2 a = *reinterpret_cast<const ulonglong2*>(res + r * 12);
          rr[0] = a.x;
          rr[1] = a.y;
          if (CP > 2) {
            const ulonglong2 b = *reinterpret_cast<const ulonglong2*>(res + r * 12 + 4);
            rr[2] = b.x;
            rr[3] = b.y;
          }
          if (CP > 4) rr[4] = *reinterpret_cast<const unsigned long long*>(res + r * 12 + 8);
        }
#pragma unroll
        for (int c = 0; c < CP; ++c)
#pragma unroll
          for (int f = 0; f < 4; ++f) acc[f][c] = ffma2(rr[c], xx[f], acc[f][c]);
      }
    }
    if (++s == kSwStages) {
      s = 0;
      parity ^= 1u;
    }
  }
  if (failed) {
    // record the failure and give the requests in flight (the tile waited for and up to kSwStages - 2 after it) the
    // same bounded time once more, so that none lands in the shared memory of a later block
    if (t == 0) atomicOr(&P.sc->err, kErrRingWait);
    for (int j = 0; j < kSwStages - 1 && tile < ntiles; ++j, tile += gridDim.x) {
      ring_wait(bar_a + 8 * s, parity);
      if (++s == kSwStages) {
        s = 0;
        parity ^= 1u;
      }
    }
  }
  float* gp = P.gpart + ((long long)m * gbpw + blockIdx.x) * P.ps;
  if (owner) {
#pragma unroll
    for (int c = 0; c < CP; ++c) {
      float4 lo, hi;                                  // classes 2c and 2c + 1
      unpack2(acc[0][c], lo.x, hi.x);
      unpack2(acc[1][c], lo.y, hi.y);
      unpack2(acc[2][c], lo.z, hi.z);
      unpack2(acc[3][c], lo.w, hi.w);
      *reinterpret_cast<float4*>(gp + (2 * c) * F + 4 * t) = lo;
      if (2 * c + 1 < C) *reinterpret_cast<float4*>(gp + (2 * c + 1) * F + 4 * t) = hi;
    }
  }
  loss = warp_sum_d(loss);
  __syncthreads();
  if (lane == 0) shd[w] = loss;
  __syncthreads();
  if (t == 0) {
    double l = 0.0;
    for (int j = 0; j < kSwThreads / 32; ++j) l += shd[j];
    P.lpart[(long long)m * gbpw + blockIdx.x] = l;
  }
}

// shapes that take the wide path: the 28 x 28 inputs and ten classes of the paper's tests
static bool softmax_wide_path(int F, int C) { return F == 784 && C == 10; }

bool softmax_classes_supported(int C) { return C >= 2 && C <= 16; }

// Row tiles of the largest shard: more gradient blocks per worker than this would only write zeros.
int grad_tiles_per_worker(int model, int F, int C, long long n_max);

// rows per tile: a multiple of 4 (so every tile starts 16-byte aligned), at most 160 KB of samples
static int logreg_rows(int F) {
  int r = (40960 / F) & ~3;
  return r > kLrMaxRows ? kLrMaxRows : r;
}
static size_t logreg_smem(int F) {
  if ((F & 1) == 0) return sizeof(float) * (2 * (size_t)kLr2Rows * F + ((F + 3) & ~3) + kLr2Rows + 2 * kLrThreads);
  return sizeof(float) * ((size_t)logreg_rows(F) * F + ((F + 3) & ~3) + kLrMaxRows + kLrThreads);
}
static size_t softmax_smem(int F, int C) { return sizeof(float) * ((size_t)kSmRows * F + (size_t)kSmRows * C); }

int grad_tiles_per_worker(int model, int F, int C, long long n_max) {
  const long long rows = (model == LAQ_MODEL_LOGREG_BIN) ? (logreg_warp_path(F) ? kLwRows : (F & 1) ? logreg_rows(F) : kLr2Rows)
                                                         : (softmax_wide_path(F, C) ? kSwRows : 8);
  const long long t = (n_max + rows - 1) / rows;
  return (int)(t > 1024 ? 1024 : (t < 1 ? 1 : t));
}

// Blocks of the gradient kernel that fit on one SM (shared memory bound): the grid is sized to one such wave.
int grad_blocks_per_sm(int model, int F, int C) {
  if (model != LAQ_MODEL_LOGREG_BIN) return softmax_wide_path(F, C) ? 1 : 2;
  if (logreg_warp_path(F)) return (int)((227 * 1024) / (logreg_warp_smem(F) + 2048));
  const int fit = (int)((227 * 1024) / (logreg_smem(F) + 1024));
  return fit < 1 ? 1 : (fit > 8 ? 8 : fit);
}

int launch_grad_logreg(const Params& P, const LaunchShape&, int gbpw, cudaStream_t st) {
  if (logreg_warp_path(P.F)) {
    const size_t smw = logreg_warp_smem(P.F);
    const dim3 gridw(gbpw, P.M);
    if (P.F == 54) {
      cudaFuncSetAttribute(grad_logreg_ring_kernel<54>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smw);
      grad_logreg_ring_kernel<54><<<gridw, kLwThreads, smw, st>>>(P, gbpw);
    } else {
      cudaFuncSetAttribute(grad_logreg_ring_kernel<22>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smw);
      grad_logreg_ring_kernel<22><<<gridw, kLwThreads, smw, st>>>(P, gbpw);
    }
    return 1;
  }
  const size_t sm = logreg_smem(P.F);
  const dim3 grid(gbpw, P.M);
  // more than the default 48 KB of dynamic shared memory is asked for per kernel and per device; the call is cheap
  // and idempotent, so it goes with every launch rather than behind a process-wide flag
  auto launch = [&](auto kernel, auto... extra) {
    if (sm > 40 * 1024) cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    kernel<<<grid, kLrThreads, sm, st>>>(P, gbpw, extra...);
  };
  if (P.F & 1) launch(grad_logreg_kernel, logreg_rows(P.F));
  else if (P.F == 54) launch(grad_logreg_pair_kernel<54>);
  else if (P.F == 22) launch(grad_logreg_pair_kernel<22>);
  else launch(grad_logreg_pair_kernel<0>);
  return 1;
}

static bool softmax_tile_path(int F, int C) { return (F % 4) == 0 && F / 4 <= kS2Threads && C <= 12; }
static size_t softmax_tile_smem(int F, int C) {
  const int FP = ((F >> 2) | 1) << 2;
  return sizeof(float) * (2 * (size_t)kS2Rows * FP + (size_t)C * F + (size_t)kS2Parts * kS2Rows * C + (size_t)kS2Rows * 24);
}

template <int C>
static void launch_sm(const Params& P, int gbpw, cudaStream_t st) {
  constexpr int CT = (C <= 12 ? C : 2);   // the tile kernel is only instantiated for C <= 12
  if (C == 10 && softmax_wide_path(P.F, C)) {
    constexpr int CW = (C == 10 ? 10 : 2);
    const size_t sm = SwShape<CW, 784>::kFloats * sizeof(float);
    cudaFuncSetAttribute(grad_softmax_wide_kernel<CW, 784>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    grad_softmax_wide_kernel<CW, 784><<<dim3(gbpw, P.M), kSwThreads, sm, st>>>(P, gbpw);
    return;
  }
  if (softmax_tile_path(P.F, C) && softmax_tile_smem(P.F, C) <= 112 * 1024) {
    const size_t sm = softmax_tile_smem(P.F, C);
    auto launch = [&](auto kernel) {
      cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
      cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                           cudaSharedmemCarveoutMaxShared);  // room for two blocks per SM
      kernel<<<dim3(gbpw, P.M), kS2Threads, sm, st>>>(P, gbpw);
    };
    if (C == 10 && P.F == 784)
      launch(grad_softmax_tile_kernel<CT, (C == 10 ? 784 : 0)>);
    else
      launch(grad_softmax_tile_kernel<CT, 0>);
    return;
  }
  const size_t sm = softmax_smem(P.F, C);
  cudaFuncSetAttribute(grad_softmax_kernel<C>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  grad_softmax_kernel<C><<<dim3(gbpw, P.M), kSmThreads, sm, st>>>(P, gbpw);
}

int launch_grad_softmax(const Params& P, const LaunchShape&, int gbpw, cudaStream_t st) {
  switch (P.C) {
#define LAQ_SM_CASE(c) case c: launch_sm<c>(P, gbpw, st); break;
    LAQ_SM_CASE(2) LAQ_SM_CASE(3) LAQ_SM_CASE(4) LAQ_SM_CASE(5) LAQ_SM_CASE(6) LAQ_SM_CASE(7) LAQ_SM_CASE(8)
    LAQ_SM_CASE(9) LAQ_SM_CASE(10) LAQ_SM_CASE(11) LAQ_SM_CASE(12) LAQ_SM_CASE(13) LAQ_SM_CASE(14)
    LAQ_SM_CASE(15) LAQ_SM_CASE(16)
#undef LAQ_SM_CASE
    default: return 0;
  }
  return 1;
}

int launch_grad_finalize(const Params& P, int gbpw, const double* theta_sq, bool with_radius, cudaStream_t st) {
  dim3 grid((unsigned)((P.p + 255) / 256), P.M);
  if (with_radius)
    grad_finalize_kernel<true><<<grid, 256, 0, st>>>(P, gbpw, theta_sq);
  else
    grad_finalize_kernel<false><<<grid, 256, 0, st>>>(P, gbpw, theta_sq);
  return 1;
}

}  // namespace laq
