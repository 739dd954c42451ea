// Step 1 of the LAQ iteration for the one-hidden-layer ReLU network of the paper's supplement
// ("Simulation details": 784-200-10, softmax cross-entropy, l2 regulariser).
//
// Parameter layout: W1 [H x F] row-major, b1 [H], W2 [C x H] row-major, b2 [C].
// The two large products take bf16 operands (round to nearest even) and accumulate in fp32:
//   hidden pre-activation  X~ W1~^T      (X~ = bf16(X), W1~ = bf16(W1))
//   W1 gradient            dH~^T X~      (dH~ = bf16(dH))
// everything else (output layer, softmax, bias gradients, regulariser) is fp32.
//
// Kernels per iteration:
//   mlp_pack_w1_kernel     W1 (fp32, [H][F]) -> W1T (bf16, [F][H]) so that a thread reads 8 hidden units in one load
//   mlp_forward_kernel     per tile of rows: hidden layer, logits, softmax, loss, dZ, dH (stored as bf16),
//                          block partials of the b1 / W2 / b2 gradients
//   mlp_dw1_kernel         dW1_m = dH~_m^T X~_m per worker, written straight into g (scaled, regularised)
//   mlp_finalize_kernel    block partials -> g for b1, W2, b2, and the worker's loss term
// Tensor-core path (n_features a multiple of 8): the two large products run on tcgen05 (laq_umma_gemm.cuh):
//   umma_hidden_kernel     H = relu(X~ W1~^T + b1) for all workers' rows at once, fp32 to memory
//   mlp_forward_kernel<1>  as above without the hidden product; writes dH~ transposed ([H][rows], K-major for
//                          the second product; every worker's row segment padded to a multiple of 64 with zeros)
//   umma_dw1_kernel        dW1_m = dH~_m^T X~_m from the transposed copies dH~^T and X~^T (made once per shard)
#include <cuda_bf16.h>

#include <vector>

#include "laq_internal.cuh"
#include "laq_umma_gemm.cuh"

namespace laq {

namespace {

constexpr int kThreads = 256;
constexpr int kMaxC = 16;

struct MlpDev {          // device pointers inside the scratch area
  int window_tiles = 0;  // 1: the fused hidden kernel skips tiles outside the minibatch window
  __nv_bfloat16* W1T;    // [F][H]
  __nv_bfloat16* Xb;     // all shards, bf16, worker m at row offset rowoff[m]
  __nv_bfloat16* dHb;    // [Ntot][H]
  float* spart;          // [M][gb][H + C*H + C]   block partials of db1, dW2, db2
  double* lpart;         // [M][gb]
  long long* rowoff;     // [M+1] prefix sums of N_m
  int gb;                // forward blocks per worker
  // tensor-core path
  __nv_bfloat16* W1b;    // [H][F]
  float* Hbuf;           // [Ntot][H]  hidden activations
  // The transposed copies are stored in blocks of 64 rows of the data (= 64 columns of the transposed matrix):
  // element (j, col) at ((col / 64) rpk + j) 64 + col mod 64, so that the tile of a K block that the W1-gradient
  // product loads is one contiguous piece of memory instead of one 128-byte piece per row, 2 ldT bytes apart.
  __nv_bfloat16* dHT;    // dH~ transposed, rpk = rpk_d (H rounded up to the 128-row tiles of the product)
  __nv_bfloat16* XbT;    // X~ transposed, rpk = rpk_x (F rounded up to the product's column tiles)
  long long* rowoffT;    // [M+1] prefix sums of N_m rounded up to 64
  long long ldT;         // sum of the rounded shard sizes
  int rpk_d, rpk_x;
};

__host__ __device__ __forceinline__ long long blocked_index(long long j, long long col, int rpk) {
  return ((col >> 6) * rpk + j) * 64 + (col & 63);
}

__global__ void __launch_bounds__(256) mlp_pack_w1_kernel(const float* __restrict__ theta, __nv_bfloat16* __restrict__ W1T,
                                                          int F, int H) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;  // index into W1T: k * H + j
  if (i < F * H) {
    const int k = i / H, j = i - k * H;
    W1T[i] = __float2bfloat16_rn(theta[(long long)j * F + k]);
  }
}

__global__ void __launch_bounds__(256) mlp_pack_x_kernel(const float* __restrict__ X, __nv_bfloat16* __restrict__ Xb,
                                                         long long n) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride)
    Xb[i] = __float2bfloat16_rn(__ldg(X + i));
}

// Thread layout of the two tile products: CG = H/8 column groups of 8 hidden units, RG = 256/CG row groups of
// 4 rows; a tile has TR = 4 RG rows.
template <bool TC>
__global__ void __launch_bounds__(kThreads) mlp_forward_kernel(const Params P, const MlpDev D) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int F = P.F, H = P.H, C = P.C, m = blockIdx.y, t = threadIdx.x, lane = t & 31, w = t >> 5;
  const int CG = H >> 3, RG = kThreads / CG, TR = 4 * RG;
  const int cg = t % CG, rg = t / CG;
  const bool active = rg < RG;
  __nv_bfloat16* xs = reinterpret_cast<__nv_bfloat16*>(smem_raw);                 // [TR][F]   (not for TC)
  float* hs = reinterpret_cast<float*>(smem_raw + (TC ? 0 : (((size_t)TR * F * 2 + 15) & ~(size_t)15)));  // [TR][H]
  float* dz = hs + (size_t)TR * H;                                                 // [TR][kMaxC]
  __shared__ double shd[32];
  const float* __restrict__ theta = P.theta;
  const float* __restrict__ b1 = theta + (long long)H * F;
  const float* __restrict__ W2 = b1 + H;
  const float* __restrict__ b2 = W2 + (long long)C * H;
  const long long n = P.N[m], row0 = D.rowoff[m];
  const __nv_bfloat16* __restrict__ Xm = D.Xb + row0 * F;
  const int32_t* __restrict__ y = P.y[m];
  float acc_db1[8];
#pragma unroll
  for (int c = 0; c < 8; ++c) acc_db1[c] = 0.f;
  float acc_w2[kMaxC];      // thread t < H owns hidden unit t for the W2 gradient
#pragma unroll
  for (int c = 0; c < kMaxC; ++c) acc_w2[c] = 0.f;
  float acc_b2 = 0.f;       // thread t < C
  double loss = 0.0;
  const RowWindow win = row_window(P, m);   // minibatch: rows outside the window contribute nothing
  const long long ntiles = (n + TR - 1) / TR;
  for (long long tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
    const long long r0 = tile * TR;
    const int nr = (int)((n - r0 < TR) ? (n - r0) : TR);
    __syncthreads();
    if (TC) {  // the hidden activations come from the tensor-core product
      const float4* src = reinterpret_cast<const float4*>(D.Hbuf + (row0 + r0) * H);
      float4* dst = reinterpret_cast<float4*>(hs);
      const int cnt4 = nr * H / 4, tot4 = TR * H / 4;
      for (int i = t; i < tot4; i += kThreads) dst[i] = (i < cnt4) ? __ldg(src + i) : make_float4(0.f, 0.f, 0.f, 0.f);
    } else {  // stage the rows (contiguous) and zero the unused ones
      const int cnt = nr * F, tot = TR * F;
      const __nv_bfloat16* src = Xm + r0 * F;
      if (((reinterpret_cast<uintptr_t>(src) & 15u) == 0)) {
        const int n8 = cnt >> 3;
        const uint4* s4 = reinterpret_cast<const uint4*>(src);
        uint4* d4 = reinterpret_cast<uint4*>(xs);
        for (int i = t; i < n8; i += kThreads) d4[i] = __ldg(s4 + i);
        for (int i = (n8 << 3) + t; i < cnt; i += kThreads) xs[i] = src[i];
      } else {
        for (int i = t; i < cnt; i += kThreads) xs[i] = src[i];
      }
      for (int i = cnt + t; i < tot; i += kThreads) xs[i] = __float2bfloat16_rn(0.f);
    }
    __syncthreads();
    // hidden layer: 4 rows x 8 hidden units per thread
    if (!TC && active) {
      float acc[4][8];
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < 8; ++c) acc[r][c] = 0.f;
      const __nv_bfloat16* xr = xs + (size_t)(4 * rg) * F;
      const uint4* wp = reinterpret_cast<const uint4*>(D.W1T) + cg;   // 8 bf16 = 16 bytes per column group
      for (int k = 0; k < F; ++k) {
        const uint4 wv = __ldg(wp + (size_t)k * CG);
        const __nv_bfloat162* w2p = reinterpret_cast<const __nv_bfloat162*>(&wv);
        float wf[8];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const float2 f2 = __bfloat1622float2(w2p[c]);
          wf[2 * c] = f2.x;
          wf[2 * c + 1] = f2.y;
        }
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          const float xv = __bfloat162float(xr[(size_t)r * F + k]);
#pragma unroll
          for (int c = 0; c < 8; ++c) acc[r][c] = fmaf(xv, wf[c], acc[r][c]);
        }
      }
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const int j = 8 * cg + c;
          hs[(size_t)(4 * rg + r) * H + j] = fmaxf(acc[r][c] + __ldg(b1 + j), 0.f);
        }
    }
    __syncthreads();
    // output layer, softmax, loss, dZ: a warp per row
    for (int r = w; r < TR; r += kThreads / 32) {
      float z[kMaxC];
#pragma unroll
      for (int c = 0; c < kMaxC; ++c) z[c] = 0.f;
      if (r < nr) {
        const float* hr = hs + (size_t)r * H;
        for (int j = lane; j < H; j += 32) {
          const float hv = hr[j];
#pragma unroll
          for (int c = 0; c < kMaxC; ++c)
            if (c < C) z[c] = fmaf(hv, __ldg(W2 + (size_t)c * H + j), z[c]);
        }
      }
#pragma unroll
      for (int c = 0; c < kMaxC; ++c) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) z[c] += __shfl_xor_sync(0xffffffffu, z[c], o);
      }
      if (r < nr && win.contains(r0 + r)) {
        float zmax = -3.0e38f;
#pragma unroll
        for (int c = 0; c < kMaxC; ++c)
          if (c < C) {
            z[c] += __ldg(b2 + c);
            zmax = fmaxf(zmax, z[c]);
          }
        float e[kMaxC], sum = 0.f;
#pragma unroll
        for (int c = 0; c < kMaxC; ++c) {
          e[c] = (c < C) ? expf(z[c] - zmax) : 0.f;
          sum += e[c];
        }
        const int yv = y[r0 + r];
        const float inv = 1.0f / sum;
        float zy = 0.f;
#pragma unroll
        for (int c = 0; c < kMaxC; ++c) {
          if (c == yv) zy = z[c];
          if (lane == 0 && c < C) dz[r * kMaxC + c] = e[c] * inv - (c == yv ? 1.f : 0.f);
        }
        if (lane == 0) loss += (double)((zmax + logf(sum)) - zy);
      } else if (lane < kMaxC) {
        dz[r * kMaxC + lane] = 0.f;   // rows beyond the shard or outside the minibatch contribute nothing
      }
    }
    __syncthreads();
    // W2 and b2 gradients (thread = hidden unit / class), on the unrounded hidden activations
    if (t < H) {
      for (int r = 0; r < nr; ++r) {
        const float hv = hs[(size_t)r * H + t];
#pragma unroll
        for (int c = 0; c < kMaxC; ++c)
          if (c < C) acc_w2[c] = fmaf(dz[r * kMaxC + c], hv, acc_w2[c]);
      }
    }
    if (t < C)
      for (int r = 0; r < nr; ++r) acc_b2 += dz[r * kMaxC + t];
    // dH = (dZ W2) o relu'(H): same 4 x 8 layout; b1 gradient from the unrounded dH; dH stored as bf16
    if (active) {
      __nv_bfloat16 dht[4][8];
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int row = 4 * rg + r;
        float d[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) d[c] = 0.f;
        for (int cc = 0; cc < C; ++cc) {
          const float dzv = dz[row * kMaxC + cc];
          const float4 wa = __ldg(reinterpret_cast<const float4*>(W2 + (size_t)cc * H + 8 * cg));
          const float4 wb = __ldg(reinterpret_cast<const float4*>(W2 + (size_t)cc * H + 8 * cg) + 1);
          d[0] = fmaf(dzv, wa.x, d[0]); d[1] = fmaf(dzv, wa.y, d[1]); d[2] = fmaf(dzv, wa.z, d[2]); d[3] = fmaf(dzv, wa.w, d[3]);
          d[4] = fmaf(dzv, wb.x, d[4]); d[5] = fmaf(dzv, wb.y, d[5]); d[6] = fmaf(dzv, wb.z, d[6]); d[7] = fmaf(dzv, wb.w, d[7]);
        }
        __nv_bfloat16 outv[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const float hv = hs[(size_t)row * H + 8 * cg + c];
          const float dh = hv > 0.f ? d[c] : 0.f;
          acc_db1[c] += dh;
          outv[c] = __float2bfloat16_rn(dh);
          if (TC) dht[r][c] = outv[c];
        }
        if (!TC && row < nr)
          *reinterpret_cast<uint4*>(D.dHb + (row0 + r0 + row) * H + 8 * cg) = *reinterpret_cast<const uint4*>(outv);
      }
      if (TC) {  // transposed store: four consecutive rows of one hidden unit are 8 contiguous bytes
        const long long col = D.rowoffT[m] + r0 + 4 * rg;
        if (col + 3 < D.rowoffT[m + 1]) {
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            __nv_bfloat16 v4[4] = {dht[0][c], dht[1][c], dht[2][c], dht[3][c]};   // rows >= nr hold dh = 0
            *reinterpret_cast<uint2*>(D.dHT + blocked_index(8 * cg + c, col, D.rpk_d)) = *reinterpret_cast<const uint2*>(v4);
          }
        }
      }
    }
  }
  // block partials: [db1 (H) | dW2 (C*H) | db2 (C)]
  __syncthreads();
  float* red = hs;   // reuse the hidden-activation tile: [RG][H]
  if (active)
#pragma unroll
    for (int c = 0; c < 8; ++c) red[rg * H + 8 * cg + c] = acc_db1[c];
  __syncthreads();
  float* sp = D.spart + ((long long)m * D.gb + blockIdx.x) * (H + C * H + C);
  if (t < H) {
    float s = 0.f;
    for (int g = 0; g < RG; ++g) s += red[g * H + t];
    sp[t] = s;
    for (int c = 0; c < C; ++c) sp[H + c * H + t] = acc_w2[c];
  }
  if (t < C) sp[H + C * H + t] = acc_b2;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) loss += __shfl_xor_sync(0xffffffffu, loss, o);
  if (lane == 0) shd[w] = loss;
  __syncthreads();
  if (t == 0) {
    double l = 0.0;
    for (int i = 0; i < kThreads / 32; ++i) l += shd[i];
    D.lpart[(long long)m * D.gb + blockIdx.x] = l;
  }
}

// dW1_m[j][k] = sum_r dH~[r][j] X~[r][k]: a block owns a 32 x 128 output tile and walks the worker's rows.
constexpr int kTJ = 32, kTK = 128, kRB = 32;

__global__ void __launch_bounds__(kThreads) mlp_dw1_kernel(const Params P, const MlpDev D) {
  __shared__ __align__(16) __nv_bfloat16 dhs[kRB][kTJ];
  __shared__ __align__(16) __nv_bfloat16 xs[kRB][kTK];
  const int F = P.F, H = P.H, m = blockIdx.z, t = threadIdx.x;
  const int j0 = blockIdx.y * kTJ, k0 = blockIdx.x * kTK;
  const int tx = t & 31, ty = t >> 5;       // 4 k per tx, 4 j per ty
  const long long n = P.N[m], row0 = D.rowoff[m];
  const __nv_bfloat16* __restrict__ Xm = D.Xb + row0 * F;
  const __nv_bfloat16* __restrict__ dHm = D.dHb + row0 * H;
  float acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
  const __nv_bfloat16 zero = __float2bfloat16_rn(0.f);
  for (long long r0 = 0; r0 < n; r0 += kRB) {
    __syncthreads();
    for (int i = t; i < kRB * kTJ; i += kThreads) {
      const int r = i / kTJ, j = i - r * kTJ;
      dhs[r][j] = (r0 + r < n && j0 + j < H) ? dHm[(r0 + r) * H + j0 + j] : zero;
    }
    for (int i = t; i < kRB * kTK; i += kThreads) {
      const int r = i / kTK, k = i - r * kTK;
      xs[r][k] = (r0 + r < n && k0 + k < F) ? Xm[(r0 + r) * F + k0 + k] : zero;
    }
    __syncthreads();
#pragma unroll 4
    for (int r = 0; r < kRB; ++r) {
      const __nv_bfloat162* dp = reinterpret_cast<const __nv_bfloat162*>(&dhs[r][4 * ty]);
      const __nv_bfloat162* xp = reinterpret_cast<const __nv_bfloat162*>(&xs[r][4 * tx]);
      const float2 d01 = __bfloat1622float2(dp[0]), d23 = __bfloat1622float2(dp[1]);
      const float2 x01 = __bfloat1622float2(xp[0]), x23 = __bfloat1622float2(xp[1]);
      const float dv[4] = {d01.x, d01.y, d23.x, d23.y}, xv[4] = {x01.x, x01.y, x23.x, x23.y};
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(dv[a], xv[b], acc[a][b]);
    }
  }
  const float inv_N = (float)(batch_scale(P, m) / (double)P.Ntot);
  const float reg = (float)((double)n / (double)P.Ntot * (double)P.lambda);
#pragma unroll
  for (int a = 0; a < 4; ++a) {
    const int j = j0 + 4 * ty + a;
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int k = k0 + 4 * tx + b;
      if (j < H && k < F) {
        const long long i = (long long)j * F + k;
        P.g[(long long)m * P.ps + i] = fmaf(acc[a][b], inv_N, reg * P.theta[i]);
      }
    }
  }
}

// Tile (or block) partials -> g for b1, W2, b2, and the worker's loss term.  Eight neighbouring lanes share an
// output: lane l adds the partials l, l + 8, ... (all of its loads independent), the eight sums are then added in
// lane order, so the result does not depend on timing and costs about one trip to the L2 instead of one per tile.
__global__ void __launch_bounds__(256) mlp_finalize_kernel(const Params P, const MlpDev D, const double* theta_sq) {
  const int H = P.H, C = P.C, F = P.F, m = blockIdx.y;
  const int nsmall = H + C * H + C;
  const int sub = threadIdx.x & 7;
  const int i = blockIdx.x * 32 + (threadIdx.x >> 3);
  const double inv_N = 1.0 / (double)P.Ntot, share = (double)P.N[m] / (double)P.Ntot;
  double s = 0.0;
  if (i < nsmall) {
    const float* sp = D.spart + (long long)m * D.gb * nsmall + i;
    for (int b = sub; b < D.gb; b += 8) s += (double)__ldg(sp + (long long)b * nsmall);
  }
  double tot = 0.0;
#pragma unroll
  for (int l = 0; l < 8; ++l) tot += __shfl_sync(0xffffffffu, s, (threadIdx.x & 24) + l);
  if (i < nsmall && sub == 0) {
    const long long pi = (long long)H * F + i;   // b1, W2, b2 follow W1 in theta in the same order as the partials
    P.g[(long long)m * P.ps + pi] =
        (float)(tot * (inv_N * batch_scale(P, m)) + share * (double)P.lambda * (double)P.theta[pi]);
  }
  if (blockIdx.x == 0 && threadIdx.x < 32) {
    double l = 0.0;
    for (int b = threadIdx.x; b < D.gb; b += 32) l += D.lpart[(long long)m * D.gb + b];
    double lt = 0.0;
    for (int k = 0; k < 32; ++k) lt += __shfl_sync(0xffffffffu, l, k);
    if (threadIdx.x == 0) P.loss_m[m] = lt * (inv_N * batch_scale(P, m)) + share * 0.5 * (double)P.lambda * (*theta_sq);
  }
}

// ---- tensor-core path ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) mlp_pack_w1b_kernel(const float* __restrict__ theta, __nv_bfloat16* __restrict__ W1b,
                                                           int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) W1b[i] = __float2bfloat16_rn(theta[i]);
}

// XbT[k][col0 + r] = bf16(X[r][k]) for one shard (done once, when the shard is loaded)
__global__ void __launch_bounds__(256) mlp_transpose_x_kernel(const float* __restrict__ X, __nv_bfloat16* __restrict__ XbT,
                                                              long long n, int F, int rpk, long long col0) {
  __shared__ float tile[32][33];
  const long long r0 = (long long)blockIdx.x * 32;
  const int k0 = blockIdx.y * 32, tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  for (int i = ty; i < 32; i += 8)
    tile[i][tx] = (r0 + i < n && k0 + tx < F) ? __ldg(X + (r0 + i) * F + k0 + tx) : 0.f;
  __syncthreads();
  for (int i = ty; i < 32; i += 8)
    if (k0 + i < F && r0 + tx < n) XbT[blocked_index(k0 + i, col0 + r0 + tx, rpk)] = __float2bfloat16_rn(tile[tx][i]);
}

struct HiddenEpi {
  float* Hbuf;
  const float* b1;
  long long Ntot;
  int H, i0;
  __device__ __forceinline__ void operator()(int r, int c0, const float (&acc)[32]) const {
    const long long row = (long long)i0 + r;
    if (row >= Ntot) return;
    float* out = Hbuf + row * H + c0;
#pragma unroll
    for (int c = 0; c < 32; c += 4) {
      if (c0 + c < H) {   // H is a multiple of 8, chunks of 4 columns are all in or all out
        const float4 b = __ldg(reinterpret_cast<const float4*>(b1 + c0 + c));
        float4 v;
        v.x = fmaxf(acc[c] + b.x, 0.f);
        v.y = fmaxf(acc[c + 1] + b.y, 0.f);
        v.z = fmaxf(acc[c + 2] + b.z, 0.f);
        v.w = fmaxf(acc[c + 3] + b.w, 0.f);
        *reinterpret_cast<float4*>(out + c) = v;
      }
    }
  }
};

__global__ void __launch_bounds__(umma::kThreads) umma_hidden_kernel(const __grid_constant__ CUtensorMap tmX,
                                                                     const __grid_constant__ CUtensorMap tmW,
                                                                     const Params P, const MlpDev D, int nt) {
  umma::TileCoord tc{(int)blockIdx.x * umma::kTileM, 0, 0, (P.F + umma::kBlockK - 1) / umma::kBlockK};
  umma::ChunkEpilogue<HiddenEpi> epi{HiddenEpi{D.Hbuf, P.theta + (long long)P.H * P.F, P.Nloc, P.H, tc.i0}, nt};
  umma::gemm_tn_tile(&tmX, &tmW, nt, tc, &P.sc->err, epi);
}

// Fused epilogue of the hidden product: from the accumulator tile (thread = row) straight to the loss, dZ, the
// bf16 dH~ (stored transposed: consecutive lanes = consecutive rows = consecutive addresses) and the tile's
// contributions to the b1 / W2 / b2 gradients, without writing the hidden activations to memory.
//   pass 1  h = relu(acc + b1); scores z += h W2^T chunk by chunk; softmax, loss, dZ (kept in registers)
//   pass 2  the accumulator is read again from tensor memory: dh = (dZ W2) o [h > 0] -> bf16 -> dH~^T; the h and dh
//           chunks go through shared memory so that threads that own columns can sum over the tile's rows
//               A[c][j] = sum_r dZ[r][c] h[r][j]   (the W2 gradient),      db1[j] = sum_r dh[r][j]
//           in a fixed order (no atomics).
// Sixteen epilogue warps: four sets of four.  A set's four warps cover the four lane quarters of tensor memory
// (all 128 rows); the sets share the 16-column chunks of the accumulator round robin in both passes.
#ifndef LAQ_DW1_STAGES
#define LAQ_DW1_STAGES 5
#endif
constexpr int kDw1Stages = LAQ_DW1_STAGES;   // ring depth of the W1-gradient product (one block per SM)

// The fused kernel is persistent: one block per SM walks the 128-row tiles of all workers.  The loader warp and the
// tensor-core warp run ahead of the epilogue warps through a ring of kFusedStages stages and TWO accumulators in
// tensor memory (2 x 256 columns), so the 13 K blocks of the next tile are loaded and multiplied while the
// epilogue warps work on the current one; the epilogue's scratch is its own shared memory, not the ring.
constexpr int kFusedStages = 3;
constexpr int kFusedSets = 4;
constexpr int kFusedEpiWarps = 4 * kFusedSets;
constexpr int kFusedEpiThreads = 32 * kFusedEpiWarps;
constexpr int kFusedThreads = 64 + kFusedEpiThreads;
constexpr uint32_t kFusedAccCols = 256;                // tensor-memory columns per accumulator
constexpr int kFusedChunk = 16;                        // columns per chunk
constexpr int kFusedPitch = kFusedChunk + 1;           // row pitch of a chunk plane in shared memory (floats)
constexpr int kFusedPlane = 128 * kFusedPitch;         // one plane: 128 rows of a chunk

__host__ __device__ inline size_t fused_extra_floats(int H) {
  return (size_t)H * 12 + 16 + (size_t)kFusedSets * 2 * kFusedPlane + 128 * 12 + 16;
}
__host__ __device__ inline size_t fused_smem_bytes(int nt, int H) {
  return kFusedStages * umma::stage_bytes(nt) + 1024 + fused_extra_floats(H) * 4;
}

struct FusedEpi {
  const Params& P;
  const MlpDev& D;
  int nt;
  float* base;              // the epilogue's scratch (shared memory behind the stage ring)
  static __device__ __forceinline__ void sync_all() { umma::named_sync<1, kFusedEpiThreads>(); }
  static __device__ __forceinline__ void sync_set(int set) {
    switch (set) {
      case 0: umma::named_sync<2, 128>(); break;
      case 1: umma::named_sync<3, 128>(); break;
      case 2: umma::named_sync<4, 128>(); break;
      default: umma::named_sync<5, 128>(); break;
    }
  }
  __device__ __forceinline__ float* w2t() const { return base; }                                   // [H][12]
  __device__ __forceinline__ float* b2s() const { return base + (size_t)P.H * 12; }               // [16]: b2, then zeros
  __device__ __forceinline__ float* chunks() const { return b2s() + 16; }                         // [sets][h, dh][128][17]

  // once per block: W2 transposed (j-major, rows of 12: ten classes at most, then b1[j], then zero) into shared
  // memory, so that the three 16-byte reads of a row bring the bias along
  __device__ __forceinline__ void load_constants(int et) const {
    const int H = P.H, C = P.C;
    const float* __restrict__ b1 = P.theta + (long long)H * P.F;
    const float* __restrict__ W2 = b1 + H;
    float* w = w2t();
    for (int i = et; i < H * 12; i += kFusedEpiThreads) {
      const int j = i / 12, c = i - 12 * j;
      w[i] = (c < C) ? __ldg(W2 + (size_t)c * H + j) : (c == 10 ? __ldg(b1 + j) : 0.f);
    }
    if (et < 16) b2s()[et] = (et < C) ? __ldg(W2 + (size_t)C * H + et) : 0.f;
  }

  // One tile.  tmem_acc: the accumulator's first column; released(): called by every epilogue thread after its last
  // read of tensor memory (the tensor-core warp may then overwrite the accumulator).
  template <class Release>
  __device__ __forceinline__ void run(uint32_t tmem_acc, int q, int lane, int set, int m, int tile, const RowWindow& win,
                                      Release released) {
    const int H = P.H, C = P.C, F = P.F;
    const int tt = q * 32 + lane;            // 0..127: the tile row this thread owns
    const int et = set * 128 + tt;           // among the epilogue threads
    const float* w2 = w2t();
    float* ch = chunks();
    float* dzs = ch + kFusedSets * 2 * kFusedPlane;   // [128][12]
    double* lossw = reinterpret_cast<double*>(dzs + 128 * 12);             // [4]
    // the tile's partials in memory: [db1 (H) | dW2 (C H) | db2 (C)]
    float* sp = D.spart + ((long long)m * D.gb + tile) * (H + C * H + C);
    float* chunk_h = ch + set * (2 * kFusedPlane);   // this set's h chunk, the dh chunk behind it
    float* chunk_d = chunk_h + kFusedPlane;
    float* red = chunk_h;                    // [16][11][16] partial column sums, reuses both chunk planes
    float* zpart = ch;                       // [sets][128][12] partial scores of the sets, before the chunks are used
    const float* b2 = b2s();                 // shared-memory copy
    const long long n = P.N[m];
    const long long trow = (long long)tile * umma::kTileM + tt;   // row within the worker's shard
    const bool valid = trow < n && win.contains(trow);
    const int yv = valid ? __ldg(P.y[m] + trow) : -1;             // asked for now, used after the first pass
    const uint32_t taddr = tmem_acc + ((uint32_t)(q * 32) << 16);
    constexpr int kStep = kFusedChunk * kFusedSets;
    // ---- pass 1: partial scores over this set's chunks, as packed pairs of classes z2[k] = (z[2k], z[2k+1])
    unsigned long long z2[5];
#pragma unroll
    for (int c = 0; c < 5; ++c) z2[c] = 0ull;
    for (int c0 = kFusedChunk * set; c0 < nt; c0 += kStep) {
      uint32_t v[kFusedChunk];
      umma::tmem_load_16(taddr + (uint32_t)c0, v);
      const float* wch = w2 + c0 * 12;                 // this chunk's rows of W2^T (with b1 in slot 10)
      const int ncol = H - c0 < kFusedChunk ? H - c0 : kFusedChunk;   // columns of the chunk that exist (<= 0: none)
      auto score = [&](int i) {
        const ulonglong2 wa = *reinterpret_cast<const ulonglong2*>(wch + i * 12);
        const ulonglong2 wb = *reinterpret_cast<const ulonglong2*>(wch + i * 12 + 4);
        const ulonglong2 wc = *reinterpret_cast<const ulonglong2*>(wch + i * 12 + 8);
        const float h = fmaxf(__uint_as_float(v[i]) + __uint_as_float((uint32_t)wc.y), 0.f);
        const unsigned long long hh = pack2(h, h);
        z2[0] = ffma2(hh, wa.x, z2[0]); z2[1] = ffma2(hh, wa.y, z2[1]);
        z2[2] = ffma2(hh, wb.x, z2[2]); z2[3] = ffma2(hh, wb.y, z2[3]);
        z2[4] = ffma2(hh, wc.x, z2[4]);
      };
      if (ncol == kFusedChunk) {                       // every chunk but the last: no per-column test
#pragma unroll
        for (int i = 0; i < kFusedChunk; ++i) score(i);
      } else {
#pragma unroll
        for (int i = 0; i < kFusedChunk; ++i)
          if (i < ncol) score(i);
      }
    }
    {
      ulonglong2* zp = reinterpret_cast<ulonglong2*>(zpart + (set * 128 + tt) * 12);
      zp[0] = make_ulonglong2(z2[0], z2[1]);
      zp[1] = make_ulonglong2(z2[2], z2[3]);
      zp[2] = make_ulonglong2(z2[4], 0ull);
    }
    sync_all();
    float dz[12];
    double loss = 0.0;
    {  // every set does the softmax of the row (the same arithmetic), set 0 keeps the loss and publishes dZ
      float z[12];
      {  // the sets' partials in order, three 16-byte reads per set
        const float4* zp4 = reinterpret_cast<const float4*>(zpart + tt * 12);
        const float4 a0 = zp4[0], a1 = zp4[1], a2 = zp4[2];
        z[0] = a0.x; z[1] = a0.y; z[2] = a0.z; z[3] = a0.w;
        z[4] = a1.x; z[5] = a1.y; z[6] = a1.z; z[7] = a1.w;
        z[8] = a2.x; z[9] = a2.y; z[10] = a2.z; z[11] = a2.w;
#pragma unroll
        for (int s2 = 1; s2 < kFusedSets; ++s2) {
          const float4* p4 = zp4 + s2 * (128 * 12 / 4);
          const float4 b0 = p4[0], b1q = p4[1], b2q = p4[2];
          z[0] += b0.x; z[1] += b0.y; z[2] += b0.z; z[3] += b0.w;
          z[4] += b1q.x; z[5] += b1q.y; z[6] += b1q.z; z[7] += b1q.w;
          z[8] += b2q.x; z[9] += b2q.y; z[10] += b2q.z; z[11] += b2q.w;
        }
      }
      float zmax = -3.0e38f;
#pragma unroll
      for (int c = 0; c < 12; ++c)
        if (c < C) {
          z[c] += b2[c];
          zmax = fmaxf(zmax, z[c]);
        }
      float e[12], sum = 0.f;
#pragma unroll
      for (int c = 0; c < 12; ++c) {
        e[c] = (c < C) ? expf(z[c] - zmax) : 0.f;
        sum += e[c];
      }
      const float inv = 1.0f / sum;
      float zy = 0.f;
#pragma unroll
      for (int c = 0; c < 12; ++c) {
        if (c == yv) zy = z[c];
        dz[c] = (valid && c < C) ? (e[c] * inv - (c == yv ? 1.f : 0.f)) : 0.f;
      }
      if (set == 0) {
        float4* d4 = reinterpret_cast<float4*>(dzs + tt * 12);
        d4[0] = make_float4(dz[0], dz[1], dz[2], dz[3]);
        d4[1] = make_float4(dz[4], dz[5], dz[6], dz[7]);
        d4[2] = make_float4(dz[8], dz[9], dz[10], dz[11]);
      }
      if (valid && set == 0) loss = (double)((zmax + logf(sum)) - zy);
    }
    sync_all();   // dZ is published; nobody reads the partial scores any more (the chunk buffers take their place)
    // ---- pass 2
    unsigned long long dz2[5];
#pragma unroll
    for (int c = 0; c < 5; ++c) dz2[c] = pack2(dz[2 * c], dz[2 * c + 1]);
    const long long col = D.rowoffT[m] + trow;
    const bool in_segment = col < D.rowoffT[m + 1];        // rows of the padded segment (zeros beyond the shard)
    // column phase: this thread sums the columns 2 cg, 2 cg + 1 of a chunk over the rows 32 q + rho + 2 k, k = 0..7;
    // with rows rho in {0, 1, 16, 17} and a pitch of 17 floats the 32 lanes of a warp read 32 different banks
    const int cg = lane & 7, rsub = lane >> 3, rho = (rsub & 1) + 16 * (rsub >> 1);
    bool released_yet = false;
    for (int c0 = kFusedChunk * set; c0 < nt; c0 += kStep) {
      uint32_t v[kFusedChunk];
      umma::tmem_load_16(taddr + (uint32_t)c0, v);
      if (c0 + kStep >= nt) {                              // that was this thread's last read of the accumulator
        released();
        released_yet = true;
      }
      const float* wch = w2 + c0 * 12;
      const int ncol = H - c0 < kFusedChunk ? H - c0 : kFusedChunk;
      __nv_bfloat16* dcol = D.dHT + blocked_index(c0, col, D.rpk_d);   // column c0 + i of this row: dcol[64 i]
      float* ph = chunk_h + tt * kFusedPitch;
      float* pd = chunk_d + tt * kFusedPitch;
      auto back = [&](int i) {
        const ulonglong2 wa = *reinterpret_cast<const ulonglong2*>(wch + i * 12);
        const ulonglong2 wb = *reinterpret_cast<const ulonglong2*>(wch + i * 12 + 4);
        const ulonglong2 wc = *reinterpret_cast<const ulonglong2*>(wch + i * 12 + 8);
        const float h = fmaxf(__uint_as_float(v[i]) + __uint_as_float((uint32_t)wc.y), 0.f);
        // even and odd classes in the two halves of a packed sum, added at the end
        unsigned long long d2 = ffma2(dz2[0], wa.x, 0ull);
        d2 = ffma2(dz2[1], wa.y, d2); d2 = ffma2(dz2[2], wb.x, d2); d2 = ffma2(dz2[3], wb.y, d2);
        d2 = ffma2(dz2[4], wc.x, d2);
        float d_even, d_odd;
        unpack2(d2, d_even, d_odd);
        const float dh = h > 0.f ? d_even + d_odd : 0.f;
        if (in_segment) dcol[64 * i] = __float2bfloat16_rn(dh);
        ph[i] = h;
        pd[i] = dh;
      };
      if (ncol == kFusedChunk) {
#pragma unroll
        for (int i = 0; i < kFusedChunk; ++i) back(i);
      } else {
#pragma unroll
        for (int i = 0; i < kFusedChunk; ++i) {
          if (i < ncol) {
            back(i);
          } else {
            ph[i] = 0.f;
            pd[i] = 0.f;
          }
        }
      }
      sync_set(set);
      {
        unsigned long long a2[2][5];        // [column][pair of classes]
        float db[2] = {0.f, 0.f};
#pragma unroll
        for (int i = 0; i < 2; ++i)
#pragma unroll
          for (int c = 0; c < 5; ++c) a2[i][c] = 0ull;
#pragma unroll 4
        for (int k = 0; k < 8; ++k) {
          const int r = 32 * q + rho + 2 * k;
          const ulonglong2 da = *reinterpret_cast<const ulonglong2*>(dzs + r * 12);
          const ulonglong2 dbq = *reinterpret_cast<const ulonglong2*>(dzs + r * 12 + 4);
          const unsigned long long dc = *reinterpret_cast<const unsigned long long*>(dzs + r * 12 + 8);
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            const float h = chunk_h[r * kFusedPitch + 2 * cg + i];
            db[i] += chunk_d[r * kFusedPitch + 2 * cg + i];
            const unsigned long long hh = pack2(h, h);
            a2[i][0] = ffma2(da.x, hh, a2[i][0]); a2[i][1] = ffma2(da.y, hh, a2[i][1]);
            a2[i][2] = ffma2(dbq.x, hh, a2[i][2]); a2[i][3] = ffma2(dbq.y, hh, a2[i][3]);
            a2[i][4] = ffma2(dc, hh, a2[i][4]);
          }
        }
        sync_set(set);              // the set has read the chunks: reuse them for the partial sums
        float* rp = red + ((q * 4 + rsub) * 11) * kFusedChunk + 2 * cg;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
#pragma unroll
          for (int c = 0; c < 5; ++c) {
            float lo, hi;
            unpack2(a2[i][c], lo, hi);
            rp[(2 * c) * kFusedChunk + i] = lo;
            rp[(2 * c + 1) * kFusedChunk + i] = hi;
          }
          rp[10 * kFusedChunk + i] = db[i];
        }
      }
      sync_set(set);
      for (int i = tt; i < 11 * kFusedChunk; i += 128) {   // fixed order over the sixteen row groups
        const int k = i / kFusedChunk, cc = i % kFusedChunk, j = c0 + cc;
        if (j < H) {
          float sum = 0.f;
#pragma unroll
          for (int gq = 0; gq < 16; ++gq) sum += red[(gq * 11 + k) * kFusedChunk + cc];
          if (k < C) sp[H + k * H + j] = sum;              // dW2[k][j]
          else if (k == 10) sp[j] = sum;                   // db1[j]
        }
      }
      sync_set(set);
    }
    if (!released_yet) released();                         // a set without chunks never read the accumulator
    // ---- db2 and the loss (every set has written the column sums of its own chunks above)
    if (set == 1 && tt < C) {
      float s = 0.f;
      for (int r = 0; r < 128; ++r) s += dzs[r * 12 + tt];
      sp[H + C * H + tt] = s;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) loss += __shfl_xor_sync(0xffffffffu, loss, o);
    if (lane == 0 && set == 0) lossw[q] = loss;
    sync_all();   // the scratch is free for the next tile (its loss terms are only written again after two more of these)
    if (et == 0) D.lpart[(long long)m * D.gb + tile] = ((lossw[0] + lossw[1]) + lossw[2]) + lossw[3];
  }
};

// the tile has rows of the shard that lie in the window (all rows without a minibatch)
__device__ __forceinline__ bool fused_tile_has_rows(const Params& P, const RowWindow& win, int m, int tile) {
  const long long t0 = (long long)tile * umma::kTileM, t1 = t0 + umma::kTileM;
  return t0 < P.N[m] && ((t0 < win.start + win.len_a && t1 > win.start) || t0 < win.len_b);
}

// grid: one block per SM (at most); block b takes the tiles b, b + gridDim.x, ... of the list (worker m, tile t),
// tile t of worker m covering the worker's rows 128 t .. 128 t + 127.
__global__ void __launch_bounds__(kFusedThreads, 1) umma_hidden_fused_kernel(const __grid_constant__ CUtensorMap tmX,
                                                                           const __grid_constant__ CUtensorMap tmW,
                                                                           const Params P, const MlpDev D, int nt) {
  extern __shared__ unsigned char umma_smem_raw[];
  __shared__ uint64_t bars[2 * kFusedStages + 5];
  __shared__ uint32_t tmem_base_sh;
  __shared__ int abort_sh;      // set by the first thread whose wait runs out: everybody stops waiting
  __shared__ int never_sh;      // stays 0: for the last waits of a block, which must not be cut short
  __shared__ int epi_ok[kFusedEpiWarps];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t smem0 = (umma::smem_u32(umma_smem_raw) + 1023u) & ~1023u;   // stages are 1024-byte aligned
  const uint32_t a_bytes = umma::kTileM * umma::kBlockK * 2, st_bytes = (uint32_t)umma::stage_bytes(nt);
  const uint32_t full0 = umma::smem_u32(&bars[0]), empty0 = umma::smem_u32(&bars[kFusedStages]);
  const uint32_t accf0 = umma::smem_u32(&bars[2 * kFusedStages]), acce0 = accf0 + 16, drain = accf0 + 32;
  float* scratch = reinterpret_cast<float*>(umma_smem_raw + (smem0 - umma::smem_u32(umma_smem_raw)) +
                                            (size_t)kFusedStages * st_bytes);
  uint32_t* err_flag = &P.sc->err;
  volatile int* abort_flag = &abort_sh;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kFusedStages; ++s) {
      umma::mbar_init(full0 + 8 * s, 1);
      umma::mbar_init(empty0 + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      umma::mbar_init(accf0 + 8 * a, 1);
      umma::mbar_init(acce0 + 8 * a, kFusedEpiThreads);   // every epilogue thread arrives once per tile
    }
    umma::mbar_init(drain, 1);
    abort_sh = 0;
    never_sh = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {  // all of the SM's tensor memory: two accumulators (whole warp)
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(umma::smem_u32(&tmem_base_sh)),
                 "r"(2 * kFusedAccCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = tmem_base_sh;
  const int gb = D.gb, total = gb * P.M;
  const int nkb = (P.F + umma::kBlockK - 1) / umma::kBlockK;
  // test hook: the loader of block 0 issues nothing and the block polls with a short limit (laq_tune "starve_copies")
  const bool starved = P.starve != 0u && blockIdx.x == 0;
  const uint32_t limit = starved ? kStarvedWaitLimit : umma::kWaitLimit;

  if (warp == 0) {
    if (lane == 0 && !starved) {
      uint32_t it = 0;
      bool ok = true;
      for (int g = blockIdx.x; g < total && ok; g += gridDim.x) {
        const int m = g / gb, tile = g - m * gb;
        const RowWindow win = row_window(P, m);
        if (!fused_tile_has_rows(P, win, m, tile)) continue;
        const int i0 = (int)(D.rowoff[m] + (long long)tile * umma::kTileM);
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const uint32_t s = it % kFusedStages, par = ((it / kFusedStages) & 1u) ^ 1u;
          if (!umma::mbar_wait_abortable(empty0 + 8 * s, par, limit, abort_flag, err_flag, 2u)) {
            ok = false;
            break;
          }
          umma::mbar_expect_tx(full0 + 8 * s, st_bytes);
          const uint32_t sa = smem0 + s * st_bytes;
          umma::tma_load_2d(sa, &tmX, full0 + 8 * s, kb * umma::kBlockK, i0);
          umma::tma_load_2d(sa + a_bytes, &tmW, full0 + 8 * s, kb * umma::kBlockK, 0);
        }
      }
      if (!ok) {
        // a wait ran out somewhere: give the copies still in flight (at most one per stage) the same bounded time to
        // land before the block leaves
        for (uint32_t back = 1; back <= (uint32_t)kFusedStages && back <= it; ++back) {
          const uint32_t j = it - back;
          umma::mbar_wait_abortable(full0 + 8 * (j % kFusedStages), (j / kFusedStages) & 1u, umma::kWaitLimit, &never_sh,
                                    err_flag, 2u);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = umma::instr_desc_bf16(nt);
      uint32_t it = 0, done = 0;
      bool ok = true;
      for (int g = blockIdx.x; g < total && ok; g += gridDim.x) {
        const int m = g / gb, tile = g - m * gb;
        const RowWindow win = row_window(P, m);
        if (!fused_tile_has_rows(P, win, m, tile)) continue;
        const uint32_t a = done & 1u, use = done >> 1;
        // the epilogue has drained this accumulator (passes at once on its first use)
        ok = umma::mbar_wait_abortable(acce0 + 8 * a, (use & 1u) ^ 1u, limit, abort_flag, err_flag, 16u);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t d_tmem = tmem_base + a * kFusedAccCols;
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const uint32_t s = it % kFusedStages;
          ok = umma::mbar_wait_abortable(full0 + 8 * s, (it / kFusedStages) & 1u, limit, abort_flag, err_flag, 4u);
          if (!ok) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t sa = smem0 + s * st_bytes;
          const uint64_t da = umma::smem_desc_sw128(sa), db = umma::smem_desc_sw128(sa + a_bytes);
#pragma unroll
          for (int kk = 0; kk < umma::kBlockK / 16; ++kk)   // 16 elements = 32 bytes = 2 descriptor address units
            umma::mma_bf16_ss(d_tmem, da + 2 * kk, db + 2 * kk, idesc, (kb | kk) != 0 ? 1u : 0u);
          umma::mma_commit(empty0 + 8 * s);                 // the stage is free once these MMAs have read it
        }
        if (!ok) break;
        umma::mma_commit(accf0 + 8 * a);                    // accumulator complete
        ++done;
      }
      // every product issued above has finished before the tensor memory is given back
      umma::mma_commit(drain);
      umma::mbar_wait_abortable(drain, 0u, umma::kWaitLimit, &never_sh, err_flag, 32u);
    }
  } else {
    const int ew = warp - 2, q = warp & 3, set = ew >> 2, et = ew * 32 + lane;
    FusedEpi epi{P, D, nt, scratch};
    epi.load_constants(et);
    FusedEpi::sync_all();
    uint32_t done = 0;
    for (int g = blockIdx.x; g < total; g += gridDim.x) {
      const int m = g / gb, tile = g - m * gb;
      const RowWindow win = row_window(P, m);
      if (!fused_tile_has_rows(P, win, m, tile)) {
        // nothing to add from this tile: its slot holds zeros (dH~ of its rows is not written, and the W1 product
        // does not read it)
        const int nsmall = P.H + P.C * P.H + P.C;
        float* sp = D.spart + ((long long)m * gb + tile) * nsmall;
        for (int i = et; i < nsmall; i += kFusedEpiThreads) sp[i] = 0.f;
        if (et == 0) D.lpart[(long long)m * gb + tile] = 0.0;
        continue;
      }
      const uint32_t a = done & 1u, use = done >> 1;
      const bool ok = __all_sync(0xffffffffu, umma::mbar_wait_abortable(accf0 + 8 * a, use & 1u, limit, abort_flag, err_flag, 8u));
      // all epilogue warps take the same branch (the outcomes are combined): the epilogue uses named barriers
      if (lane == 0) epi_ok[ew] = ok ? 1 : 0;
      FusedEpi::sync_all();
      int all_ok = 1;
#pragma unroll
      for (int e = 0; e < kFusedEpiWarps; ++e) all_ok &= epi_ok[e];
      if (!all_ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t acc_bar = acce0 + 8 * a;
      epi.run(tmem_base + a * kFusedAccCols, q, lane, set, m, tile, win, [&]() {
        // every epilogue thread arrives once per tile, after its last read of the accumulator
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        umma::mbar_arrive(acc_bar);
      });
      ++done;
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(2 * kFusedAccCols) : "memory");
  }
}

struct Dw1Epi {
  float* g;            // worker's gradient row
  const float* theta;
  float inv_N, reg;
  int H, F, j0, k0, nt;
  __device__ __forceinline__ void operator()(int r, int c0, const float (&acc)[32]) const {
    const int j = j0 + r;
    if (j >= H) return;
#pragma unroll
    for (int c = 0; c < 32; ++c) {
      const int k = k0 + c0 + c;
      if (c0 + c < nt && k < F) {
        const long long i = (long long)j * F + k;
        g[i] = fmaf(acc[c], inv_N, reg * theta[i]);
      }
    }
  }
};

__global__ void __launch_bounds__(umma::kThreads) umma_dw1_kernel(const __grid_constant__ CUtensorMap tmD,
                                                                  const __grid_constant__ CUtensorMap tmXT,
                                                                  const Params P, const MlpDev D, int nt) {
  const int m = blockIdx.z;
  const long long c0 = D.rowoffT[m], c1 = D.rowoffT[m + 1];
  umma::TileCoord tc{(int)blockIdx.y * umma::kTileM, (int)blockIdx.x * nt, (int)c0, (int)((c1 - c0) / umma::kBlockK)};
  tc.a_rpk = D.rpk_d;
  tc.b_rpk = D.rpk_x;
  const long long n = P.N[m];
  if (D.window_tiles) {
    // minibatch: only the 128-row tiles that meet the window were written by the hidden kernel in this iteration;
    // K runs over their 64-column blocks, in two pieces when the window wraps
    const RowWindow win = row_window(P, m);
    const int nblk = tc.nkb, per = umma::kTileM / umma::kBlockK;
    const int a0 = (int)(win.start / umma::kTileM) * per;
    int a1 = (int)((win.start + win.len_a - 1) / umma::kTileM + 1) * per;
    a1 = a1 < nblk ? a1 : nblk;
    int b1 = win.len_b > 0 ? (int)((win.len_b - 1) / umma::kTileM + 1) * per : 0;
    b1 = b1 < nblk ? b1 : nblk;
    if (b1 >= a0) {             // one piece from the start of the segment (or no wrap at all and a0 = 0)
      tc.k0 = (int)c0 + (b1 > 0 ? 0 : a0) * umma::kBlockK;
      tc.nkb = b1 > 0 ? a1 : a1 - a0;
    } else {
      tc.k0 = (int)c0 + a0 * umma::kBlockK;
      tc.nkb_first = a1 - a0;
      tc.k1 = (int)c0;
      tc.nkb = (a1 - a0) + b1;
    }
  }
  umma::ChunkEpilogue<Dw1Epi> epi{Dw1Epi{P.g + (long long)m * P.ps, P.theta, (float)(batch_scale(P, m) / (double)P.Ntot),
                                         (float)((double)n / (double)P.Ntot * (double)P.lambda), P.H, P.F, tc.i0,
                                         tc.j0, nt},
                                  nt};
  umma::gemm_tn_tile<kDw1Stages>(&tmD, &tmXT, nt, tc, &P.sc->err, epi);
}

struct HostPlan {
  MlpDev d;
  size_t fwd_smem;
  char* scratch_tc = nullptr;
  std::vector<long long> N_host, offT_host;
  bool tc = false;          // tensor-core path in use
  int nt1 = 0, nt2 = 0;     // N tiles of the two products
  int fused_tiles = 0;      // > 0: the hidden product runs with the fused epilogue, this many tiles per worker
  CUtensorMap tmX, tmW, tmD, tmXT;
  // the small-gradient kernel runs beside the W1 product (both only read what the fused kernel wrote)
  cudaStream_t side = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
};

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

int forward_blocks_per_worker(int M) {
  int g = (2 * kNumSMs + M - 1) / M;
  return g < 1 ? 1 : (g > 64 ? 64 : g);
}

// column tile of the W1-gradient product and the rows per K block of the two blocked transposed copies
int dw1_nt(int F) { return (F % 112 == 0) ? 112 : ((F >= 128) ? 128 : (F + 15) / 16 * 16); }
int rpk_d_for(int H) { return (H + umma::kTileM - 1) / umma::kTileM * umma::kTileM; }
int rpk_x_for(int F) { return (F + dw1_nt(F) - 1) / dw1_nt(F) * dw1_nt(F); }

// the tcgen05 path needs 16-byte row pitches for its tensor maps
bool tc_shape_ok(int F, int H) { return (F % 8) == 0 && (H % 8) == 0 && H >= 16 && H <= 256; }

size_t forward_smem_tc(int H) {
  const int CG = H / 8, RG = kThreads / CG, TR = 4 * RG;
  return (size_t)TR * H * 4 + (size_t)TR * kMaxC * 4;
}

// tiles per worker of the fused hidden kernel, or 0 if the fused epilogue cannot be used for this shape
int fused_tiles_for(int F, int H, int C, const long long* N, int M) {
  if (!tc_shape_ok(F, H) || C > 10) return 0;        // the epilogue sums five pairs of classes
  const int nt1 = (H + 15) / 16 * 16;
  if (fused_smem_bytes(nt1, H) > 226 * 1024) return 0;   // stage ring + the epilogue's scratch must fit one SM
  long long tiles = 0;
  for (int m = 0; m < M; ++m) {
    const long long t = (N[m] + umma::kTileM - 1) / umma::kTileM;
    if (t > tiles) tiles = t;
  }
  return tiles <= 256 ? (int)tiles : 0;
}

size_t forward_smem(int F, int H) {
  const int CG = H / 8, RG = kThreads / CG, TR = 4 * RG;
  return (((size_t)TR * F * 2 + 15) & ~(size_t)15) + (size_t)TR * H * 4 + (size_t)TR * kMaxC * 4;
}

}  // namespace

const char* mlp_check_shape(int F, int H, int C) {
  if (H < 8 || H > 256 || (H % 8) != 0) return "MLP2 supports n_hidden in 8..256, a multiple of 8";
  if (C < 2 || C > kMaxC) return "MLP2 supports 2..16 classes";
  if (F < 1 || forward_smem(F, H) > 200 * 1024) return "MLP2: n_features too large for the row tile";
  return nullptr;
}

size_t mlp_scratch_bytes(const laq_config& c) {
  long long Ntot = 0;
  for (int m = 0; m < c.M; ++m) Ntot += c.N[m];
  std::vector<long long> Nv(c.N, c.N + c.M);
  const int ft = fused_tiles_for(c.n_features, c.n_hidden, c.n_classes, Nv.data(), c.M);
  const int gb = ft > forward_blocks_per_worker(c.M) ? ft : forward_blocks_per_worker(c.M);
  const size_t nsmall = (size_t)c.n_hidden + (size_t)c.n_classes * c.n_hidden + c.n_classes;
  size_t b = 0;
  b += align256((size_t)c.n_features * c.n_hidden * 2);          // W1T
  b += align256((size_t)Ntot * c.n_features * 2);                // Xb
  b += align256((size_t)Ntot * c.n_hidden * 2);                  // dHb
  b += align256((size_t)c.M * gb * nsmall * 4);                  // spart
  b += align256((size_t)c.M * gb * 8);                           // lpart
  b += align256((size_t)(c.M + 1) * 8);                          // rowoff
  if (tc_shape_ok(c.n_features, c.n_hidden)) {
    long long ldT = 0;
    for (int m = 0; m < c.M; ++m) ldT += (c.N[m] + 63) / 64 * 64;
    b += align256((size_t)c.n_hidden * c.n_features * 2);        // W1b
    b += align256((size_t)Ntot * c.n_hidden * 4);                // Hbuf
    b += align256((size_t)rpk_d_for(c.n_hidden) * ldT * 2);      // dHT
    b += align256((size_t)rpk_x_for(c.n_features) * ldT * 2);    // XbT
    b += align256((size_t)(c.M + 1) * 8);                        // rowoffT
  }
  return b;
}

laq_status mlp_setup(MlpPlan& mp, const Params& P, const long long* N_host, void* scratch, cudaStream_t st) {
  HostPlan* hp = new HostPlan();
  const int ft = fused_tiles_for(P.F, P.H, P.C, N_host, P.M);
  const int gb_alloc = ft > forward_blocks_per_worker(P.M) ? ft : forward_blocks_per_worker(P.M);
  char* p = (char*)scratch;
  const size_t nsmall = (size_t)P.H + (size_t)P.C * P.H + P.C;
  hp->d.gb = forward_blocks_per_worker(P.M);
  hp->d.W1T = (__nv_bfloat16*)p; p += align256((size_t)P.F * P.H * 2);
  hp->d.Xb = (__nv_bfloat16*)p; p += align256((size_t)P.Nloc * P.F * 2);
  hp->d.dHb = (__nv_bfloat16*)p; p += align256((size_t)P.Nloc * P.H * 2);
  hp->d.spart = (float*)p; p += align256((size_t)P.M * gb_alloc * nsmall * 4);
  hp->d.lpart = (double*)p; p += align256((size_t)P.M * gb_alloc * 8);
  hp->d.rowoff = (long long*)p; p += align256((size_t)(P.M + 1) * 8);
  hp->fwd_smem = forward_smem(P.F, P.H);
  hp->scratch_tc = p;
  // prefix sums of the shard sizes (N is not yet on the device when this runs, so it comes from the host copy)
  mp.scratch = hp;
  mp.ready = 0;
  if (cudaFuncSetAttribute(mlp_forward_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)hp->fwd_smem) !=
      cudaSuccess)
    return LAQ_ECUDA;
  (void)st;
  return LAQ_OK;
}

laq_status mlp_set_row_offsets(MlpPlan& mp, const long long* N_host, int M, cudaStream_t st) {
  HostPlan* hp = (HostPlan*)mp.scratch;
  long long off[1025];
  off[0] = 0;
  for (int m = 0; m < M; ++m) off[m + 1] = off[m] + N_host[m];
  if (cudaMemcpyAsync(hp->d.rowoff, off, sizeof(long long) * (M + 1), cudaMemcpyHostToDevice, st) != cudaSuccess)
    return LAQ_ECUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return LAQ_ECUDA;
  hp->N_host.assign(N_host, N_host + M);
  return LAQ_OK;
}

// Tensor-core path: carve its buffers, zero the transposed copies (their padding columns must stay zero), build
// the four tensor maps.  Falls back to the plain kernels if the shape does not fit or a map cannot be made.
laq_status mlp_setup_tensor_path(MlpPlan& mp, const Params& P, cudaStream_t st) {
  HostPlan* hp = (HostPlan*)mp.scratch;
  hp->tc = false;
  if (!tc_shape_ok(P.F, P.H)) return LAQ_OK;
  const int M = P.M;
  long long offT[1025];
  offT[0] = 0;
  for (int m = 0; m < M; ++m) offT[m + 1] = offT[m] + (hp->N_host[m] + 63) / 64 * 64;
  const long long ldT = offT[M];
  if (ldT >= (1ll << 31) || P.Nloc >= (1ll << 31)) return LAQ_OK;
  char* p = hp->scratch_tc;
  hp->d.W1b = (__nv_bfloat16*)p; p += align256((size_t)P.H * P.F * 2);
  hp->d.Hbuf = (float*)p; p += align256((size_t)P.Nloc * P.H * 4);
  hp->d.rpk_d = rpk_d_for(P.H);
  hp->d.rpk_x = rpk_x_for(P.F);
  hp->d.dHT = (__nv_bfloat16*)p; p += align256((size_t)hp->d.rpk_d * ldT * 2);
  hp->d.XbT = (__nv_bfloat16*)p; p += align256((size_t)hp->d.rpk_x * ldT * 2);
  hp->d.rowoffT = (long long*)p;
  hp->d.ldT = ldT;
  hp->nt1 = (P.H + 15) / 16 * 16;
  hp->nt2 = dw1_nt(P.F);
  if (cudaMemsetAsync(hp->d.dHT, 0, (size_t)hp->d.rpk_d * ldT * 2, st) != cudaSuccess) return LAQ_ECUDA;
  if (cudaMemsetAsync(hp->d.XbT, 0, (size_t)hp->d.rpk_x * ldT * 2, st) != cudaSuccess) return LAQ_ECUDA;
  if (cudaMemcpyAsync(hp->d.rowoffT, offT, sizeof(long long) * (M + 1), cudaMemcpyHostToDevice, st) != cudaSuccess)
    return LAQ_ECUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return LAQ_ECUDA;
  bool ok = umma::make_map_bf16_2d(&hp->tmX, hp->d.Xb, (uint64_t)P.Nloc, (uint64_t)P.F, (uint64_t)P.F * 2, umma::kTileM);
  ok = ok && umma::make_map_bf16_2d(&hp->tmW, hp->d.W1b, (uint64_t)P.H, (uint64_t)P.F, (uint64_t)P.F * 2, hp->nt1);
  // blocked copies: 64 columns, (ldT / 64) rpk rows
  ok = ok && umma::make_map_bf16_2d(&hp->tmD, hp->d.dHT, (uint64_t)(ldT / 64) * hp->d.rpk_d, 64, 128, umma::kTileM);
  ok = ok && umma::make_map_bf16_2d(&hp->tmXT, hp->d.XbT, (uint64_t)(ldT / 64) * hp->d.rpk_x, 64, 128, hp->nt2);
  if (!ok) return LAQ_OK;   // plain kernels
  if (cudaFuncSetAttribute(umma_hidden_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)umma::smem_bytes(hp->nt1)) != cudaSuccess ||
      cudaFuncSetAttribute(umma_dw1_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)umma::smem_bytes(hp->nt2, kDw1Stages)) != cudaSuccess ||
      cudaFuncSetAttribute(mlp_forward_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)forward_smem_tc(P.H)) != cudaSuccess) {
    cudaGetLastError();
    return LAQ_OK;
  }
  hp->offT_host.assign(offT, offT + M + 1);
  hp->tc = true;
  if (cudaStreamCreateWithFlags(&hp->side, cudaStreamNonBlocking) != cudaSuccess ||
      cudaEventCreateWithFlags(&hp->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&hp->ev_join, cudaEventDisableTiming) != cudaSuccess) {
    cudaGetLastError();
    hp->side = nullptr;            // everything on the caller's stream then
  }
  const int ft = fused_tiles_for(P.F, P.H, P.C, hp->N_host.data(), M);
  if (ft > 0 && cudaFuncSetAttribute(umma_hidden_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)fused_smem_bytes(hp->nt1, P.H)) == cudaSuccess) {
    hp->fused_tiles = ft;
    hp->d.gb = ft;        // one partial slot per tile
    hp->d.window_tiles = P.batch > 0 ? 1 : 0;
  } else {
    cudaGetLastError();
  }
  return LAQ_OK;
}

int mlp_convert_shard(MlpPlan& mp, const Params& P, int m, const float* X, long long n, long long row_offset,
                      cudaStream_t st) {
  HostPlan* hp = (HostPlan*)mp.scratch;
  const long long cnt = n * P.F;
  mlp_pack_x_kernel<<<kNumSMs * 4, 256, 0, st>>>(X, hp->d.Xb + row_offset * P.F, cnt);
  if (!hp->tc) return 1;
  mlp_transpose_x_kernel<<<dim3((unsigned)((n + 31) / 32), (unsigned)((P.F + 31) / 32)), 256, 0, st>>>(
      X, hp->d.XbT, n, P.F, hp->d.rpk_x, hp->offT_host[m]);
  return 2;
}

int mlp_launch_gradients(MlpPlan& mp, const Params& P, const double* theta_sq, cudaStream_t st) {
  HostPlan* hp = (HostPlan*)mp.scratch;
  const int F = P.F, H = P.H, C = P.C;
  const int nsmall = H + C * H + C;
  if (hp->tc) {
    // the bf16 copy of W1 is kept up to date by the theta step (Params::w1b); without that hook it is made here
    int extra = 0;
    if (P.w1b == nullptr) {
      mlp_pack_w1b_kernel<<<(F * H + 255) / 256, 256, 0, st>>>(P.theta, hp->d.W1b, F * H);
      extra = 1;
    }
    if (hp->fused_tiles > 0) {
      const int tiles = hp->fused_tiles * P.M;
      umma_hidden_fused_kernel<<<tiles < kNumSMs ? tiles : kNumSMs, kFusedThreads, fused_smem_bytes(hp->nt1, H), st>>>(
          hp->tmX, hp->tmW, P, hp->d, hp->nt1);
      // fork: the small-gradient kernel on a side stream, the W1 product on the caller's; join before the sweeps
      // (the same pattern inside a stream capture makes the two kernels siblings in the graph)
      const bool forked = hp->side != nullptr && cudaEventRecord(hp->ev_fork, st) == cudaSuccess &&
                          cudaStreamWaitEvent(hp->side, hp->ev_fork, 0) == cudaSuccess;
      mlp_finalize_kernel<<<dim3((nsmall + 31) / 32, P.M), 256, 0, forked ? hp->side : st>>>(P, hp->d, theta_sq);
      if (forked) cudaEventRecord(hp->ev_join, hp->side);
      umma_dw1_kernel<<<dim3((F + hp->nt2 - 1) / hp->nt2, (H + umma::kTileM - 1) / umma::kTileM, P.M), umma::kThreads,
                        umma::smem_bytes(hp->nt2, kDw1Stages), st>>>(hp->tmD, hp->tmXT, P, hp->d, hp->nt2);
      if (forked) cudaStreamWaitEvent(st, hp->ev_join, 0);
      return 3 + extra;
    }
    umma_hidden_kernel<<<(unsigned)((P.Nloc + umma::kTileM - 1) / umma::kTileM), umma::kThreads,
                         umma::smem_bytes(hp->nt1), st>>>(hp->tmX, hp->tmW, P, hp->d, hp->nt1);
    mlp_forward_kernel<true><<<dim3(hp->d.gb, P.M), kThreads, forward_smem_tc(H), st>>>(P, hp->d);
    umma_dw1_kernel<<<dim3((F + hp->nt2 - 1) / hp->nt2, (H + umma::kTileM - 1) / umma::kTileM, P.M), umma::kThreads,
                      umma::smem_bytes(hp->nt2, kDw1Stages), st>>>(hp->tmD, hp->tmXT, P, hp->d, hp->nt2);
    mlp_finalize_kernel<<<dim3((nsmall + 31) / 32, P.M), 256, 0, st>>>(P, hp->d, theta_sq);
    return 4 + extra;
  }
  mlp_pack_w1_kernel<<<(F * H + 255) / 256, 256, 0, st>>>(P.theta, hp->d.W1T, F, H);
  mlp_forward_kernel<false><<<dim3(hp->d.gb, P.M), kThreads, hp->fwd_smem, st>>>(P, hp->d);
  mlp_dw1_kernel<<<dim3((F + kTK - 1) / kTK, (H + kTJ - 1) / kTJ, P.M), kThreads, 0, st>>>(P, hp->d);
  mlp_finalize_kernel<<<dim3((nsmall + 31) / 32, P.M), 256, 0, st>>>(P, hp->d, theta_sq);
  return 4;
}

void* mlp_w1_copy(const MlpPlan& mp) {
  const HostPlan* hp = (const HostPlan*)mp.scratch;
  return (hp && hp->tc) ? (void*)hp->d.W1b : nullptr;
}

int mlp_refresh_w1_copy(MlpPlan& mp, const Params& P, cudaStream_t st) {
  HostPlan* hp = (HostPlan*)mp.scratch;
  if (!hp || !hp->tc) return 0;
  mlp_pack_w1b_kernel<<<(P.F * P.H + 255) / 256, 256, 0, st>>>(P.theta, hp->d.W1b, P.F * P.H);
  return 1;
}

void mlp_teardown(MlpPlan& mp) {
  HostPlan* hp = (HostPlan*)mp.scratch;
  if (hp) {
    if (hp->side) cudaStreamDestroy(hp->side);
    if (hp->ev_fork) cudaEventDestroy(hp->ev_fork);
    if (hp->ev_join) cudaEventDestroy(hp->ev_join);
  }
  delete (HostPlan*)mp.scratch;
  mp.scratch = nullptr;
}

}  // namespace laq
