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
  __nv_bfloat16* dHT;    // [H][ldT]   dH~ transposed
  __nv_bfloat16* XbT;    // [F][ldT]   X~ transposed
  long long* rowoffT;    // [M+1] prefix sums of N_m rounded up to 64
  long long ldT;         // sum of the rounded shard sizes
};

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
            *reinterpret_cast<uint2*>(D.dHT + (long long)(8 * cg + c) * D.ldT + col) = *reinterpret_cast<const uint2*>(v4);
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

__global__ void __launch_bounds__(256) mlp_finalize_kernel(const Params P, const MlpDev D, const double* theta_sq) {
  const int H = P.H, C = P.C, F = P.F, m = blockIdx.y;
  const int nsmall = H + C * H + C;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  const double inv_N = 1.0 / (double)P.Ntot, share = (double)P.N[m] / (double)P.Ntot;
  if (i < nsmall) {
    double s = 0.0;
    for (int b = 0; b < D.gb; ++b) s += (double)D.spart[((long long)m * D.gb + b) * nsmall + i];
    const long long pi = (long long)H * F + i;   // b1, W2, b2 follow W1 in theta in the same order as the partials
    P.g[(long long)m * P.ps + pi] =
        (float)(s * (inv_N * batch_scale(P, m)) + share * (double)P.lambda * (double)P.theta[pi]);
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    double l = 0.0;
    for (int b = 0; b < D.gb; ++b) l += D.lpart[(long long)m * D.gb + b];
    P.loss_m[m] = l * (inv_N * batch_scale(P, m)) + share * 0.5 * (double)P.lambda * (*theta_sq);
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
                                                              long long n, int F, long long ldT, long long col0) {
  __shared__ float tile[32][33];
  const long long r0 = (long long)blockIdx.x * 32;
  const int k0 = blockIdx.y * 32, tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  for (int i = ty; i < 32; i += 8)
    tile[i][tx] = (r0 + i < n && k0 + tx < F) ? __ldg(X + (r0 + i) * F + k0 + tx) : 0.f;
  __syncthreads();
  for (int i = ty; i < 32; i += 8)
    if (k0 + i < F && r0 + tx < n) XbT[(long long)(k0 + i) * ldT + col0 + r0 + tx] = __float2bfloat16_rn(tile[tx][i]);
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
  umma::ChunkEpilogue<HiddenEpi> epi{HiddenEpi{D.Hbuf, P.theta + (long long)P.H * P.F, P.Ntot, P.H, tc.i0}, nt};
  umma::gemm_tn_tile(&tmX, &tmW, nt, tc, &P.sc->err, epi);
}

// Fused epilogue of the hidden product: from the accumulator tile (thread = row) straight to the loss, dZ, the
// bf16 dH~ (stored transposed: consecutive lanes = consecutive rows = consecutive addresses) and the tile's
// contributions to the b1 / W2 / b2 gradients, without writing the hidden activations to memory.
//   pass 1  h = relu(acc + b1); scores z += h W2^T chunk by chunk; softmax, loss, dZ (kept in registers)
//   pass 2  the accumulator is read again from tensor memory: dh = (dZ W2) o [h > 0] -> bf16 -> dH~^T; the h chunk
//           goes through shared memory so that a thread per column can sum over the tile's rows
//               A[c][j] = sum_r dZ[r][c] h[r][j]         (the W2 gradient)
//               S[c][j] = sum_r dZ[r][c] [h[r][j] > 0]   (then db1[j] = sum_c W2[c][j] S[c][j])
//           in a fixed order (no atomics).
// Eight epilogue warps: two sets of four, each set taking every other 32-column chunk in both passes.
constexpr int kFusedStages = 2;   // two stages of ring per block, two blocks per SM
#ifndef LAQ_DW1_STAGES
#define LAQ_DW1_STAGES 4
#endif
constexpr int kDw1Stages = LAQ_DW1_STAGES;   // ring depth of the W1-gradient product (one block per SM)

constexpr int kFusedEpiWarps = 8;                      // two sets of four epilogue warps
constexpr int kFusedThreads = 64 + 32 * kFusedEpiWarps;

__host__ __device__ inline size_t fused_extra_floats(int H) {
  return (size_t)H * 12 + (size_t)((H + 3) & ~3) + 2 * 128 * 33 + 128 * 12 + 2 * (size_t)12 * H + 16;
}

// Both sets of epilogue warps own all 128 rows (thread = row) and share the 32-column chunks of the accumulator
// between them: set 0 takes chunks 0, 2, 4, ..., set 1 chunks 1, 3, 5, ...  The scores are the sum of the two sets'
// partial scores (set 0's first); every later step is per column, so the sets only meet at three block-wide points.
struct FusedEpi {
  const Params& P;
  const MlpDev& D;
  int nt, m, tile;          // worker and tile index within the worker
  RowWindow win;            // rows of the worker that enter this iteration's gradient
  static __device__ __forceinline__ void sync_all() { umma::named_sync<1, 32 * kFusedEpiWarps>(); }
  static __device__ __forceinline__ void sync_set(int set) {
    if (set == 0) umma::named_sync<2, 128>(); else umma::named_sync<3, 128>();
  }
  __device__ __forceinline__ void run(uint32_t tmem_base, int q, int lane, int set) {
    const int H = P.H, C = P.C, F = P.F;
    const int tt = q * 32 + lane;            // 0..127: the tile row this thread owns
    const int et = set * 128 + tt;           // 0..255 among the epilogue threads
    float* base = reinterpret_cast<float*>(umma::ring_smem());   // the ring is free once the accumulator is complete
    float* w2t = base;                       // [H][12]   W2 transposed (j-major), padded rows of 12
    float* b1s = w2t + (size_t)H * 12;       // [H]
    float* chunks = b1s + ((H + 3) & ~3);    // [2][128][33] one 32-column chunk of h per set
    float* dzs = chunks + 2 * 128 * 33;      // [128][12]
    float* accA = dzs + 128 * 12;            // [12][H]
    float* accS = accA + (size_t)12 * H;     // [12][H]
    double* lossw = reinterpret_cast<double*>(accS + (size_t)12 * H);      // [4] (8-byte aligned: all sizes even)
    float* chunk = chunks + set * 128 * 33;  // this set's chunk buffer
    float* red = chunk;                      // [4][2 C][32] partial column sums, reuses the chunk buffer
    float* zpart = chunks;                   // [2][128][12] partial scores of the two sets, before the chunks are used
    const float* __restrict__ theta = P.theta;
    const float* __restrict__ b1 = theta + (long long)H * F;
    const float* __restrict__ W2 = b1 + H;
    const float* __restrict__ b2 = W2 + (long long)C * H;
    for (int i = et; i < H * 12; i += 256) {
      const int j = i / 12, c = i - 12 * j;
      w2t[i] = (c < C) ? __ldg(W2 + (size_t)c * H + j) : 0.f;
    }
    for (int i = et; i < H; i += 256) b1s[i] = __ldg(b1 + i);
    const long long n = P.N[m];
    const long long trow = (long long)tile * umma::kTileM + tt;   // row within the worker's shard
    const bool valid = trow < n && win.contains(trow);
    const int yv = valid ? __ldg(P.y[m] + trow) : -1;             // asked for now, used after the first pass
    sync_all();
    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
    // ---- pass 1: partial scores over this set's chunks, as packed pairs of classes z2[k] = (z[2k], z[2k+1])
    unsigned long long z2[6];
#pragma unroll
    for (int c = 0; c < 6; ++c) z2[c] = 0ull;
    for (int c0 = 32 * set; c0 < nt; c0 += 64) {
      uint32_t v[32];
      umma::tmem_load_32(taddr + (uint32_t)c0, v);
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const int j = c0 + i;
        if (j < H) {
          const float h = fmaxf(__uint_as_float(v[i]) + b1s[j], 0.f);
          const unsigned long long hh = pack2(h, h);
          const ulonglong2 wa = *reinterpret_cast<const ulonglong2*>(w2t + j * 12);
          const ulonglong2 wb = *reinterpret_cast<const ulonglong2*>(w2t + j * 12 + 4);
          const ulonglong2 wc = *reinterpret_cast<const ulonglong2*>(w2t + j * 12 + 8);
          z2[0] = ffma2(hh, wa.x, z2[0]); z2[1] = ffma2(hh, wa.y, z2[1]);
          z2[2] = ffma2(hh, wb.x, z2[2]); z2[3] = ffma2(hh, wb.y, z2[3]);
          z2[4] = ffma2(hh, wc.x, z2[4]); z2[5] = ffma2(hh, wc.y, z2[5]);
        }
      }
    }
    {
      ulonglong2* zp = reinterpret_cast<ulonglong2*>(zpart + (set * 128 + tt) * 12);
      zp[0] = make_ulonglong2(z2[0], z2[1]);
      zp[1] = make_ulonglong2(z2[2], z2[3]);
      zp[2] = make_ulonglong2(z2[4], z2[5]);
    }
    sync_all();
    float dz[12];
    double loss = 0.0;
    {  // both sets do the softmax of the row (the same arithmetic), set 0 keeps the loss and publishes dZ
      float z[12];
#pragma unroll
      for (int c = 0; c < 12; ++c) z[c] = zpart[tt * 12 + c] + zpart[(128 + tt) * 12 + c];
      float zmax = -3.0e38f;
#pragma unroll
      for (int c = 0; c < 12; ++c)
        if (c < C) {
          z[c] += __ldg(b2 + c);
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
        if (set == 0) dzs[tt * 12 + c] = dz[c];
      }
      if (valid && set == 0) loss = (double)((zmax + logf(sum)) - zy);
    }
    sync_all();   // dZ is published; nobody reads the partial scores any more (the chunk buffers take their place)
    // ---- pass 2
    unsigned long long dz2[6];
#pragma unroll
    for (int c = 0; c < 6; ++c) dz2[c] = pack2(dz[2 * c], dz[2 * c + 1]);
    const long long col = D.rowoffT[m] + trow;
    const bool in_segment = col < D.rowoffT[m + 1];        // rows of the padded segment (zeros beyond the shard)
    const int rq = tt >> 5, cl = tt & 31;                  // reduce phase: column cl, rows 32 rq .. 32 rq + 31
    for (int c0 = 32 * set; c0 < nt; c0 += 64) {
      uint32_t v[32];
      umma::tmem_load_32(taddr + (uint32_t)c0, v);
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const int j = c0 + i;
        float h = 0.f;
        if (j < H) {
          h = fmaxf(__uint_as_float(v[i]) + b1s[j], 0.f);
          const ulonglong2 wa = *reinterpret_cast<const ulonglong2*>(w2t + j * 12);
          const ulonglong2 wb = *reinterpret_cast<const ulonglong2*>(w2t + j * 12 + 4);
          const ulonglong2 wc = *reinterpret_cast<const ulonglong2*>(w2t + j * 12 + 8);
          // even and odd classes in the two halves of a packed sum, added at the end
          unsigned long long d2 = ffma2(dz2[0], wa.x, 0ull);
          d2 = ffma2(dz2[1], wa.y, d2); d2 = ffma2(dz2[2], wb.x, d2); d2 = ffma2(dz2[3], wb.y, d2);
          d2 = ffma2(dz2[4], wc.x, d2); d2 = ffma2(dz2[5], wc.y, d2);
          float d_even, d_odd;
          unpack2(d2, d_even, d_odd);
          const float d = d_even + d_odd;
          const float dh = h > 0.f ? d : 0.f;
          if (in_segment) D.dHT[(long long)j * D.ldT + col] = __float2bfloat16_rn(dh);
        }
        chunk[tt * 33 + i] = h;
      }
      sync_set(set);
      {  // column sums over this thread's 32 rows
        unsigned long long a2[6], s2[6];    // packed pairs of classes
#pragma unroll
        for (int c = 0; c < 6; ++c) a2[c] = s2[c] = 0ull;
#pragma unroll 4
        for (int r = 32 * rq; r < 32 * rq + 32; ++r) {
          const float h = chunk[r * 33 + cl];
          const float pos = h > 0.f ? 1.f : 0.f;
          const unsigned long long hh = pack2(h, h), pp = pack2(pos, pos);
          const ulonglong2 da = *reinterpret_cast<const ulonglong2*>(dzs + r * 12);
          const ulonglong2 db = *reinterpret_cast<const ulonglong2*>(dzs + r * 12 + 4);
          const ulonglong2 dc = *reinterpret_cast<const ulonglong2*>(dzs + r * 12 + 8);
          a2[0] = ffma2(da.x, hh, a2[0]); a2[1] = ffma2(da.y, hh, a2[1]); a2[2] = ffma2(db.x, hh, a2[2]);
          a2[3] = ffma2(db.y, hh, a2[3]); a2[4] = ffma2(dc.x, hh, a2[4]); a2[5] = ffma2(dc.y, hh, a2[5]);
          s2[0] = ffma2(da.x, pp, s2[0]); s2[1] = ffma2(da.y, pp, s2[1]); s2[2] = ffma2(db.x, pp, s2[2]);
          s2[3] = ffma2(db.y, pp, s2[3]); s2[4] = ffma2(dc.x, pp, s2[4]); s2[5] = ffma2(dc.y, pp, s2[5]);
        }
        float a[12], sgn[12];
#pragma unroll
        for (int c = 0; c < 6; ++c) {
          unpack2(a2[c], a[2 * c], a[2 * c + 1]);
          unpack2(s2[c], sgn[2 * c], sgn[2 * c + 1]);
        }
        sync_set(set);              // the set has read the chunk: reuse it for the partial sums
#pragma unroll
        for (int c = 0; c < 12; ++c) {
          red[(rq * 24 + c) * 32 + cl] = a[c];
          red[(rq * 24 + 12 + c) * 32 + cl] = sgn[c];
        }
      }
      sync_set(set);
      for (int i = tt; i < 24 * 32; i += 128) {   // fixed order over the four row quarters
        const int k = i >> 5, cc = i & 31, j = c0 + cc;
        if (j < H) {
          const float sum4 = ((red[(0 * 24 + k) * 32 + cc] + red[(1 * 24 + k) * 32 + cc]) + red[(2 * 24 + k) * 32 + cc]) +
                             red[(3 * 24 + k) * 32 + cc];
          if (k < 12) accA[k * H + j] = sum4; else accS[(k - 12) * H + j] = sum4;
        }
      }
      sync_set(set);
    }
    // ---- the tile's partials: [db1 (H) | dW2 (C H) | db2 (C)] and the loss
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) loss += __shfl_xor_sync(0xffffffffu, loss, o);
    if (lane == 0 && set == 0) lossw[q] = loss;
    sync_all();
    const int gb = D.gb;
    float* sp = D.spart + ((long long)m * gb + tile) * (H + C * H + C);
    for (int j = et; j < H; j += 256) {
      float s = 0.f;
      for (int c = 0; c < C; ++c) s = fmaf(w2t[j * 12 + c], accS[c * H + j], s);
      sp[j] = s;
      for (int c = 0; c < C; ++c) sp[H + c * H + j] = accA[c * H + j];
    }
    if (set == 1 && tt < C) {
      float s = 0.f;
      for (int r = 0; r < 128; ++r) s += dzs[r * 12 + tt];
      sp[H + C * H + tt] = s;
    }
    if (et == 0) D.lpart[(long long)m * gb + tile] = ((lossw[0] + lossw[1]) + lossw[2]) + lossw[3];
  }
};

// grid: (tiles per worker, M); tile t of worker m covers the worker's rows 128 t .. 128 t + 127
__global__ void __launch_bounds__(kFusedThreads, 2) umma_hidden_fused_kernel(const __grid_constant__ CUtensorMap tmX,
                                                                           const __grid_constant__ CUtensorMap tmW,
                                                                           const Params P, const MlpDev D, int nt) {
  const int m = blockIdx.y, tile = blockIdx.x;
  const long long n = P.N[m];
  const RowWindow win = row_window(P, m);
  const long long t0 = (long long)tile * umma::kTileM, t1 = t0 + umma::kTileM;
  // the tile has rows of the shard that lie in the window (all rows without a minibatch)
  const bool has_rows = t0 < n && ((t0 < win.start + win.len_a && t1 > win.start) || t0 < win.len_b);
  umma::TileCoord tc{(int)(D.rowoff[m] + t0), 0, 0, has_rows ? (P.F + umma::kBlockK - 1) / umma::kBlockK : 0};
  if (!has_rows) {   // nothing to add from this tile: its slot holds zeros (dH~ of its rows is not written, and
                     // the dW1 product does not read it)
    const int nsmall = P.H + P.C * P.H + P.C;
    float* sp = D.spart + ((long long)m * D.gb + tile) * nsmall;
    for (int i = threadIdx.x; i < nsmall; i += blockDim.x) sp[i] = 0.f;
    if (threadIdx.x == 0) D.lpart[(long long)m * D.gb + tile] = 0.0;
    return;
  }
  FusedEpi epi{P, D, nt, m, tile, win};
  umma::gemm_tn_tile<kFusedStages, kFusedEpiWarps>(&tmX, &tmW, nt, tc, &P.sc->err, epi);
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
};

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

int forward_blocks_per_worker(int M) {
  int g = (2 * kNumSMs + M - 1) / M;
  return g < 1 ? 1 : (g > 64 ? 64 : g);
}

// the tcgen05 path needs 16-byte row pitches for its tensor maps
bool tc_shape_ok(int F, int H) { return (F % 8) == 0 && (H % 8) == 0 && H >= 16 && H <= 256; }

size_t forward_smem_tc(int H) {
  const int CG = H / 8, RG = kThreads / CG, TR = 4 * RG;
  return (size_t)TR * H * 4 + (size_t)TR * kMaxC * 4;
}

// tiles per worker of the fused hidden kernel, or 0 if the fused epilogue cannot be used for this shape
int fused_tiles_for(int F, int H, int C, const long long* N, int M) {
  if (!tc_shape_ok(F, H) || C > 12) return 0;
  const int nt1 = (H + 15) / 16 * 16;
  if (fused_extra_floats(H) * 4 > kFusedStages * umma::stage_bytes(nt1)) return 0;   // the epilogue's scratch lives in the ring
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
    b += align256((size_t)c.n_hidden * ldT * 2);                 // dHT
    b += align256((size_t)c.n_features * ldT * 2);               // XbT
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
  hp->d.Xb = (__nv_bfloat16*)p; p += align256((size_t)P.Ntot * P.F * 2);
  hp->d.dHb = (__nv_bfloat16*)p; p += align256((size_t)P.Ntot * P.H * 2);
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
  if (ldT >= (1ll << 31) || P.Ntot >= (1ll << 31)) return LAQ_OK;
  char* p = hp->scratch_tc;
  hp->d.W1b = (__nv_bfloat16*)p; p += align256((size_t)P.H * P.F * 2);
  hp->d.Hbuf = (float*)p; p += align256((size_t)P.Ntot * P.H * 4);
  hp->d.dHT = (__nv_bfloat16*)p; p += align256((size_t)P.H * ldT * 2);
  hp->d.XbT = (__nv_bfloat16*)p; p += align256((size_t)P.F * ldT * 2);
  hp->d.rowoffT = (long long*)p;
  hp->d.ldT = ldT;
  hp->nt1 = (P.H + 15) / 16 * 16;
  hp->nt2 = (P.F % 112 == 0) ? 112 : ((P.F >= 128) ? 128 : (P.F + 15) / 16 * 16);
  if (cudaMemsetAsync(hp->d.dHT, 0, (size_t)P.H * ldT * 2, st) != cudaSuccess) return LAQ_ECUDA;
  if (cudaMemsetAsync(hp->d.XbT, 0, (size_t)P.F * ldT * 2, st) != cudaSuccess) return LAQ_ECUDA;
  if (cudaMemcpyAsync(hp->d.rowoffT, offT, sizeof(long long) * (M + 1), cudaMemcpyHostToDevice, st) != cudaSuccess)
    return LAQ_ECUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return LAQ_ECUDA;
  bool ok = umma::make_map_bf16_2d(&hp->tmX, hp->d.Xb, (uint64_t)P.Ntot, (uint64_t)P.F, (uint64_t)P.F * 2, umma::kTileM);
  ok = ok && umma::make_map_bf16_2d(&hp->tmW, hp->d.W1b, (uint64_t)P.H, (uint64_t)P.F, (uint64_t)P.F * 2, hp->nt1);
  ok = ok && umma::make_map_bf16_2d(&hp->tmD, hp->d.dHT, (uint64_t)P.H, (uint64_t)ldT, (uint64_t)ldT * 2, umma::kTileM);
  ok = ok && umma::make_map_bf16_2d(&hp->tmXT, hp->d.XbT, (uint64_t)P.F, (uint64_t)ldT, (uint64_t)ldT * 2, hp->nt2);
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
  const int ft = fused_tiles_for(P.F, P.H, P.C, hp->N_host.data(), M);
  if (ft > 0 && cudaFuncSetAttribute(umma_hidden_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)umma::smem_bytes(hp->nt1, kFusedStages)) == cudaSuccess) {
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
      X, hp->d.XbT, n, P.F, hp->d.ldT, hp->offT_host[m]);
  return 2;
}

int mlp_launch_gradients(MlpPlan& mp, const Params& P, const double* theta_sq, cudaStream_t st) {
  HostPlan* hp = (HostPlan*)mp.scratch;
  const int F = P.F, H = P.H, C = P.C;
  const int nsmall = H + C * H + C;
  if (hp->tc) {
    mlp_pack_w1b_kernel<<<(F * H + 255) / 256, 256, 0, st>>>(P.theta, hp->d.W1b, F * H);
    if (hp->fused_tiles > 0) {
      umma_hidden_fused_kernel<<<dim3(hp->fused_tiles, P.M), kFusedThreads,
                                 umma::smem_bytes(hp->nt1, kFusedStages), st>>>(hp->tmX, hp->tmW, P, hp->d,
                                                                                              hp->nt1);
      umma_dw1_kernel<<<dim3((F + hp->nt2 - 1) / hp->nt2, (H + umma::kTileM - 1) / umma::kTileM, P.M), umma::kThreads,
                        umma::smem_bytes(hp->nt2, kDw1Stages), st>>>(hp->tmD, hp->tmXT, P, hp->d, hp->nt2);
      mlp_finalize_kernel<<<dim3((nsmall + 255) / 256, P.M), 256, 0, st>>>(P, hp->d, theta_sq);
      return 4;
    }
    umma_hidden_kernel<<<(unsigned)((P.Ntot + umma::kTileM - 1) / umma::kTileM), umma::kThreads,
                         umma::smem_bytes(hp->nt1), st>>>(hp->tmX, hp->tmW, P, hp->d, hp->nt1);
    mlp_forward_kernel<true><<<dim3(hp->d.gb, P.M), kThreads, forward_smem_tc(H), st>>>(P, hp->d);
    umma_dw1_kernel<<<dim3((F + hp->nt2 - 1) / hp->nt2, (H + umma::kTileM - 1) / umma::kTileM, P.M), umma::kThreads,
                      umma::smem_bytes(hp->nt2, kDw1Stages), st>>>(hp->tmD, hp->tmXT, P, hp->d, hp->nt2);
    mlp_finalize_kernel<<<dim3((nsmall + 255) / 256, P.M), 256, 0, st>>>(P, hp->d, theta_sq);
    return 5;
  }
  mlp_pack_w1_kernel<<<(F * H + 255) / 256, 256, 0, st>>>(P.theta, hp->d.W1T, F, H);
  mlp_forward_kernel<false><<<dim3(hp->d.gb, P.M), kThreads, hp->fwd_smem, st>>>(P, hp->d);
  mlp_dw1_kernel<<<dim3((F + kTK - 1) / kTK, (H + kTJ - 1) / kTJ, P.M), kThreads, 0, st>>>(P, hp->d);
  mlp_finalize_kernel<<<dim3((nsmall + 255) / 256, P.M), 256, 0, st>>>(P, hp->d, theta_sq);
  return 4;
}

void mlp_teardown(MlpPlan& mp) {
  delete (HostPlan*)mp.scratch;
  mp.scratch = nullptr;
}

}  // namespace laq
