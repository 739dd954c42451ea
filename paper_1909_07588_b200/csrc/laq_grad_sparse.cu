// Step 1 of the LAQ iteration for softmax regression on SPARSE samples (LAQ_FLAG_SPARSE_X): the inputs of the
// paper's 784-feature tests have about one non-zero in five, so a compressed copy of a shard lets both products of
// the gradient skip the zeros:
//   scores     z[r][c]  = sum over the non-zeros (f, v) of row r of          v theta[c][f]
//   gradient   G[c][f] += sum over the non-zeros (r, v) of column f of       v residual[r][c]
// The copy is made once, when the shard is loaded, in tiles of 128 rows.  A tile is stored twice, both times with
// the k-th entry of all its rows (columns) side by side, so that a thread per row (per column) reads coalesced:
//   by rows      entry k of row r    at  off_r + k 128 + r   (feature index, value), k < Lr = longest row of the tile
//   by columns   entry k of column f at  off_c + k F + f     (row in tile, value),   k < Lc = longest column of the tile
// Short rows and columns are padded with (0, 0.0f), which adds exact zeros.  Entries keep the order of the dense
// matrix (ascending feature, ascending row), and each sum runs in that order in one thread: results do not depend
// on timing.  Block partials go to the same buffers as the dense kernels', so the same finalize kernel follows.
#include <string>
#include <vector>

#include "laq_internal.cuh"

namespace laq {

namespace {

constexpr int kSpRows = 128;       // rows per tile = threads per block
constexpr int kSpMaxColsPerThread = 7;   // F <= 7 x 128

// Longest row and longest column of every tile.  grid: tiles; block: 128 threads.
__global__ void __launch_bounds__(kSpRows) sparse_count_kernel(const float* __restrict__ X, long long n, int F,
                                                               int* __restrict__ L /* [tiles][2] */) {
  __shared__ int s_max[2];
  const int t = threadIdx.x;
  const long long r0 = (long long)blockIdx.x * kSpRows;
  if (t < 2) s_max[t] = 0;
  __syncthreads();
  int cnt = 0;
  if (r0 + t < n) {
    const float* xr = X + (r0 + t) * F;
    for (int f = 0; f < F; ++f) cnt += xr[f] != 0.f;
  }
  atomicMax(&s_max[0], cnt);
  const int nr = (int)((n - r0 < kSpRows) ? (n - r0) : kSpRows);
  for (int f = t; f < F; f += kSpRows) {
    int c = 0;
    for (int r = 0; r < nr; ++r) c += X[(r0 + r) * F + f] != 0.f;
    atomicMax(&s_max[1], c);
  }
  __syncthreads();
  if (t < 2) L[2 * blockIdx.x + t] = s_max[t];
}

// Fills the two copies of every tile.  grid: tiles; block: 128 threads.
__global__ void __launch_bounds__(kSpRows) sparse_fill_kernel(const float* __restrict__ X, long long n, int F,
                                                              const long long* __restrict__ off_r,
                                                              const long long* __restrict__ off_c, float* __restrict__ val,
                                                              uint16_t* __restrict__ idx) {
  const int t = threadIdx.x, tile = blockIdx.x;
  const long long r0 = (long long)tile * kSpRows;
  const int nr = (int)((n - r0 < kSpRows) ? (n - r0) : kSpRows);
  {
    const long long o = off_r[tile];
    const int Lr = (int)((off_r[tile + 1] - o) / kSpRows);
    int k = 0;
    if (t < nr) {
      const float* xr = X + (r0 + t) * F;
      for (int f = 0; f < F; ++f) {
        const float v = xr[f];
        if (v != 0.f) {
          val[o + (long long)k * kSpRows + t] = v;
          idx[o + (long long)k * kSpRows + t] = (uint16_t)f;
          ++k;
        }
      }
    }
    for (; k < Lr; ++k) {
      val[o + (long long)k * kSpRows + t] = 0.f;
      idx[o + (long long)k * kSpRows + t] = 0;
    }
  }
  {
    const long long o = off_c[tile];
    const int Lc = (int)((off_c[tile + 1] - o) / F);
    for (int f = t; f < F; f += kSpRows) {
      int k = 0;
      for (int r = 0; r < nr; ++r) {
        const float v = X[(r0 + r) * F + f];
        if (v != 0.f) {
          val[o + (long long)k * F + f] = v;
          idx[o + (long long)k * F + f] = (uint16_t)r;
          ++k;
        }
      }
      for (; k < Lc; ++k) {
        val[o + (long long)k * F + f] = 0.f;
        idx[o + (long long)k * F + f] = 0;
      }
    }
  }
}

// grid: (blocks per worker, M); block: 128 threads.  Dynamic shared memory: theta as [F][C] and the tile's residuals
// as [128][C], both with a row pitch of C floats (C even: 8-byte reads).
template <int C>
__global__ void __launch_bounds__(kSpRows) grad_softmax_sparse_kernel(const Params P, int gbpw) {
  static_assert((C & 1) == 0 && C <= 10, "an even number of classes, at most ten");
  extern __shared__ __align__(16) float smem[];
  __shared__ double shd[kSpRows / 32];
  const int F = P.F, m = blockIdx.y, t = threadIdx.x;
  float* th_s = smem;                 // [F][C]
  float* res_s = smem + (size_t)F * C;   // [128][C]
  const SparseShard sp = P.sp[m];
  const int32_t* __restrict__ y = P.y[m];
  const long long n = P.N[m];
  for (int i = t; i < F * C; i += kSpRows) {
    const int f = i / C, c = i - f * C;
    th_s[i] = c < P.C ? P.theta[(long long)c * F + f] : 0.f;
  }
  float acc[kSpMaxColsPerThread][C];
#pragma unroll
  for (int j = 0; j < kSpMaxColsPerThread; ++j)
#pragma unroll
    for (int c = 0; c < C; ++c) acc[j][c] = 0.f;
  double loss = 0.0;
  const RowWindow win = row_window(P, m);
  __syncthreads();
  for (int tile = blockIdx.x; tile < sp.tiles; tile += gridDim.x) {
    const long long r0 = (long long)tile * kSpRows, t1 = r0 + kSpRows;
    // tiles without a row of the minibatch window add nothing
    if (!((r0 < win.start + win.len_a && t1 > win.start) || r0 < win.len_b)) continue;
    // ---- scores, softmax, residual: thread = row
    {
      const long long o = sp.off_r[tile];
      const int Lr = (int)((sp.off_r[tile + 1] - o) / kSpRows);
      const float* __restrict__ pv = sp.val + o + t;
      const uint16_t* __restrict__ pi = sp.idx + o + t;
      float z[C];
#pragma unroll
      for (int c = 0; c < C; ++c) z[c] = 0.f;
#pragma unroll 4
      for (int k = 0; k < Lr; ++k) {
        const float v = __ldg(pv + (size_t)k * kSpRows);
        const float2* th = reinterpret_cast<const float2*>(th_s + (size_t)__ldg(pi + (size_t)k * kSpRows) * C);
#pragma unroll
        for (int c = 0; c < C; c += 2) {
          const float2 w = th[c >> 1];
          z[c] = fmaf(v, w.x, z[c]);
          z[c + 1] = fmaf(v, w.y, z[c + 1]);
        }
      }
      const long long row = r0 + t;
      const bool valid = row < n && win.contains(row);
      float zmax = -3.0e38f;
#pragma unroll
      for (int c = 0; c < C; ++c)
        if (c < P.C) zmax = fmaxf(zmax, z[c]);
      float e[C], sum = 0.f;
#pragma unroll
      for (int c = 0; c < C; ++c) {
        e[c] = c < P.C ? expf(z[c] - zmax) : 0.f;
        sum += e[c];
      }
      const int yv = valid ? __ldg(y + row) : -1;
      const float inv = 1.0f / sum;
      float zy = 0.f;
#pragma unroll
      for (int c = 0; c < C; ++c) {
        if (c == yv) zy = z[c];
        res_s[t * C + c] = (valid && c < P.C) ? (e[c] * inv - (c == yv ? 1.f : 0.f)) : 0.f;
      }
      if (valid) loss += (double)((zmax + logf(sum)) - zy);
    }
    __syncthreads();
    // ---- gradient: thread = columns t, t + 128, ...
    {
      const long long o = sp.off_c[tile];
      const int Lc = (int)((sp.off_c[tile + 1] - o) / F);
#pragma unroll
      for (int j = 0; j < kSpMaxColsPerThread; ++j) {
        const int f = t + j * kSpRows;
        if (f < F) {
          const float* __restrict__ pv = sp.val + o + f;
          const uint16_t* __restrict__ pi = sp.idx + o + f;
#pragma unroll 4
          for (int k = 0; k < Lc; ++k) {
            const float v = __ldg(pv + (size_t)k * F);
            const float2* rr = reinterpret_cast<const float2*>(res_s + (size_t)__ldg(pi + (size_t)k * F) * C);
#pragma unroll
            for (int c = 0; c < C; c += 2) {
              const float2 w = rr[c >> 1];
              acc[j][c] = fmaf(v, w.x, acc[j][c]);
              acc[j][c + 1] = fmaf(v, w.y, acc[j][c + 1]);
            }
          }
        }
      }
    }
    __syncthreads();   // the residuals are free for the next tile
  }
  // ---- block partial (theta's layout: [C][F])
  float* gp = P.gpart + ((long long)m * gbpw + blockIdx.x) * P.ps;
#pragma unroll
  for (int j = 0; j < kSpMaxColsPerThread; ++j) {
    const int f = t + j * kSpRows;
    if (f < F)
#pragma unroll
      for (int c = 0; c < C; ++c)
        if (c < P.C) gp[(long long)c * F + f] = acc[j][c];
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) loss += __shfl_xor_sync(0xffffffffu, loss, o);
  if ((t & 31) == 0) shd[t >> 5] = loss;
  __syncthreads();
  if (t == 0) {
    double l = 0.0;
    for (int i = 0; i < kSpRows / 32; ++i) l += shd[i];
    P.lpart[(long long)m * gbpw + blockIdx.x] = l;
  }
}

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

long long sparse_tiles(long long n) { return (n + kSpRows - 1) / kSpRows; }
// entries (value + index) a shard's compressed copies may take: as many as the dense matrix has elements
long long sparse_capacity(long long n, int F) { return sparse_tiles(n) * kSpRows * (long long)F; }

}  // namespace

bool sparse_shape_ok(int F, int C) { return F >= 1 && F <= kSpMaxColsPerThread * kSpRows && C >= 2 && C <= 10; }

size_t sparse_region_bytes(long long n, int F) {
  const long long T = sparse_tiles(n), cap = sparse_capacity(n, F);
  return align256((size_t)(2 * (T + 1)) * 8) + align256((size_t)(2 * T) * 4) + align256((size_t)cap * 4) +
         align256((size_t)cap * 2);
}

int sparse_blocks_per_worker(const long long* N, int M) {
  long long tmax = 1;
  for (int m = 0; m < M; ++m) tmax = sparse_tiles(N[m]) > tmax ? sparse_tiles(N[m]) : tmax;
  long long g = (4ll * kNumSMs) / M;       // four blocks of 128 threads per SM (registers)
  if (g > tmax) g = tmax;
  return (int)(g < 1 ? 1 : g);
}

// Builds the compressed copies of worker m's shard from the dense matrix X (device) inside `region` and writes the
// worker's descriptor to desc_dev[m].  Synchronises the stream (the tile lengths come back to the host to lay the
// tiles out).  Returns LAQ_EWORKSPACE when the shard has too many non-zeros for the region.
laq_status sparse_build(int m, const float* X, long long n, int F, void* region, SparseShard* desc_dev, cudaStream_t st,
                        std::string* err) {
  const long long T = sparse_tiles(n), cap = sparse_capacity(n, F);
  char* p = (char*)region;
  long long* off = (long long*)p; p += align256((size_t)(2 * (T + 1)) * 8);
  int* L = (int*)p; p += align256((size_t)(2 * T) * 4);
  float* val = (float*)p; p += align256((size_t)cap * 4);
  uint16_t* idx = (uint16_t*)p;
  sparse_count_kernel<<<(unsigned)T, kSpRows, 0, st>>>(X, n, F, L);
  std::vector<int> Lh(2 * T);
  if (cudaMemcpyAsync(Lh.data(), L, sizeof(int) * 2 * T, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) {
    *err = "sparse copy: reading the tile lengths failed";
    return LAQ_ECUDA;
  }
  // layout only: where each tile's two copies start
  std::vector<long long> offh(2 * (T + 1));
  long long e = 0;
  for (long long t = 0; t < T; ++t) {
    offh[t] = e;
    e += (long long)Lh[2 * t] * kSpRows;
  }
  offh[T] = e;
  for (long long t = 0; t < T; ++t) {
    offh[T + 1 + t] = e;
    e += (long long)Lh[2 * t + 1] * F;
  }
  offh[2 * T + 1] = e;
  if (e > cap) {
    *err = "LAQ_FLAG_SPARSE_X: the shard is too dense for its compressed copies (they may take as many entries as the dense matrix has elements)";
    return LAQ_EWORKSPACE;
  }
  SparseShard d;
  d.val = val;
  d.idx = idx;
  d.off_r = off;
  d.off_c = off + T + 1;
  d.tiles = (int)T;
  if (cudaMemcpyAsync(off, offh.data(), sizeof(long long) * offh.size(), cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpyAsync(desc_dev + m, &d, sizeof(d), cudaMemcpyHostToDevice, st) != cudaSuccess) {
    *err = "sparse copy: writing the tile offsets failed";
    return LAQ_ECUDA;
  }
  sparse_fill_kernel<<<(unsigned)T, kSpRows, 0, st>>>(X, n, F, d.off_r, d.off_c, val, idx);
  if (cudaStreamSynchronize(st) != cudaSuccess || cudaGetLastError() != cudaSuccess) {   // offh and d go out of scope
    *err = "sparse copy: the fill kernel failed";
    return LAQ_ECUDA;
  }
  return LAQ_OK;
}

int launch_grad_softmax_sparse(const Params& P, int gbpw, cudaStream_t st) {
  const int Cp = (P.C + 1) & ~1;                      // classes rounded up to even (a zero class is added)
  const size_t sm = sizeof(float) * ((size_t)P.F * Cp + (size_t)kSpRows * Cp);
  const dim3 grid(gbpw, P.M);
  auto launch = [&](auto kernel) {
    if (sm > 40 * 1024) cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    kernel<<<grid, kSpRows, sm, st>>>(P, gbpw);
  };
  switch (Cp) {
    case 2: launch(grad_softmax_sparse_kernel<2>); break;
    case 4: launch(grad_softmax_sparse_kernel<4>); break;
    case 6: launch(grad_softmax_sparse_kernel<6>); break;
    case 8: launch(grad_softmax_sparse_kernel<8>); break;
    default: launch(grad_softmax_sparse_kernel<10>); break;
  }
  return 1;
}

}  // namespace laq
