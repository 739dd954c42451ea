// Steps 2-5 of the LAQ iteration as three streaming kernels over the per-worker vectors:
//   radius_kernel     R_m = || g_m - Q_m(theta_hat^{k-1}) ||_inf                       (Sec. 2.1)
//   quantize_kernel   codes of Eq. (5), ||dQ_m||^2 and ||eps_m||^2; its last block evaluates the
//                     skip rule (7a)/(7b), advances the clocks and lists the uploaders    (Sec. 2.2)
//   aggregate_kernel  for uploaders only: Q_m += dQ_m decoded from (R_m, codes) as the server
//                     does after Eq. (6); grad += sum dQ_m; theta -= alpha grad; its last block
//                     pushes ||alpha grad||^2 onto the ring of stored differences        (Eq. (4))
// All three are bound by HBM bandwidth: a lane reads 16 B of a row per load, a warp 512 B
// contiguous, with several independent loads in flight per thread.  Reductions are two-stage with
// a fixed order (no floating-point atomics), so a run is reproducible bit for bit.
//
// Compiled with -fmad=false: every fp32 operation below is a single IEEE round-to-nearest
// operation, in the order documented in laq.h; fused multiply-adds appear only where written.
#include <cuda_bf16.h>

#include "laq_internal.cuh"

namespace laq {

namespace {

// Synthetic gradient stream (definition in laq.h).  One strong hash per group of four coordinates,
// a cheap second word from it, and two near-Gaussian byte sums per word.
struct Synth {
  uint32_t key;
  float cz, drift;
  __device__ __forceinline__ void init(const Params& P, int m, unsigned long long k_iter) {
    const int gid = P.m_first + P.m_stride * m;     // the worker's global index
    key = fmix32(P.seed_lo ^ fmix32(P.seed_hi + 0x9e3779b9u * (uint32_t)(gid + 1)));
    cz = P.cz;
    float eta_m = (float)((double)P.eta0 * (double)(gid + 1) / (double)P.M_total);
    drift = __fmul_rn((float)k_iter, eta_m);
  }
  // coordinates 4v .. 4v+3
  __device__ __forceinline__ float4 at4(uint32_t v) const {
    const uint32_t h0 = fmix32(v ^ key);
    uint32_t h1 = h0 * 0x9e3779b1u;
    h1 ^= h1 >> 15;
    // b0+b2 and b1+b3 of each word; the even sums land directly on the bit pattern of 1.5 * 2^23 (the dot
    // product's addend), so that one integer add or subtract per value gives 1.5 * 2^23 + (a small integer)
    const int e0 = (int)__dp4a(h0, 0x00010001u, 0x4b400000u), o0 = (int)__dp4a(h0, 0x01000100u, 0u);
    const int e1 = (int)__dp4a(h1, 0x00010001u, 0x4b400000u), o1 = (int)__dp4a(h1, 0x01000100u, 0u);
    // exact int -> float through the mantissa of 1.5 * 2^23 (the -510 offset folds into the constant)
    const float z0 = __int_as_float(e0 + o0) - (12582912.0f + 510.0f);
    const float z1 = __int_as_float(e0 - o0) - 12582912.0f;
    const float z2 = __int_as_float(e1 + o1) - (12582912.0f + 510.0f);
    const float z3 = __int_as_float(e1 - o1) - 12582912.0f;
    float4 r;
    r.x = __fmul_rn(__fmaf_rn(drift, z2, z0), cz);
    r.y = __fmul_rn(__fmaf_rn(drift, z3, z1), cz);
    r.z = __fmul_rn(__fmaf_rn(drift, z0, z2), cz);
    r.w = __fmul_rn(__fmaf_rn(drift, z1, z3), cz);
    return r;
  }
  // the same with zeros at coordinates >= p (last group of a row)
  __device__ __forceinline__ float4 at4_masked(uint32_t v, long long p) const {
    float4 r = at4(v);
    const long long i = 4ll * v;
    if (i >= p) r.x = 0.f;
    if (i + 1 >= p) r.y = 0.f;
    if (i + 2 >= p) r.z = 0.f;
    if (i + 3 >= p) r.w = 0.f;
    return r;
  }
};

// asks for the line of ptr to be brought into L2; no register waits for it
__device__ __forceinline__ void prefetch_l2(const void* ptr) { asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr)); }

__device__ __forceinline__ uint32_t abs_bits(float x) { return __float_as_uint(x) & 0x7fffffffu; }

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Fixed-order block sum of one double per thread; result valid in thread 0.
__device__ __forceinline__ double block_sum(double v, double* sh /* >= 32 doubles */) {
  v = warp_sum(v);
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  __syncthreads();
  if (lane == 0) sh[w] = v;
  __syncthreads();
  double t = 0.0;
  if (threadIdx.x == 0)
    for (int i = 0; i < nw; ++i) t += sh[i];
  return t;
}

#ifndef LAQ_SWEEP_UNROLL
#define LAQ_SWEEP_UNROLL 2
#endif
#ifndef LAQ_QUANT_MAX_THREADS
#define LAQ_QUANT_MAX_THREADS 512
#endif
#ifndef LAQ_QUANT_MIN_BLOCKS
#define LAQ_QUANT_MIN_BLOCKS 2   // caps the quantize kernel at 64 registers (measured best)
#endif
#ifndef LAQ_QUANT_CHAINS
#define LAQ_QUANT_CHAINS 1       // independent fp64 accumulation chains per sum and thread (more: registers spill)
#endif
constexpr int kUnroll = LAQ_SWEEP_UNROLL;  // 16-byte groups in flight per thread

// ||theta||^2 of the iterate in memory (set by the caller: theta^0, or a restored state) into DevScalars::theta_sq,
// which the kernels otherwise keep up to date themselves.  One block, fp64, fixed order.
__global__ void __launch_bounds__(1024) theta_sq_kernel(const Params P) {
  __shared__ double sh[32];
  double t = 0.0;
  for (long long i = threadIdx.x; i < P.p; i += blockDim.x) t = fma((double)P.theta[i], (double)P.theta[i], t);
  t = block_sum(t, sh);
  if (threadIdx.x == 0) P.sc->theta_sq = t;
}

// ------------------------------------------------------------------------------------------------
// LAQ_FLAG_STORE_G with LAQ_MODEL_SYNTH: the workers' gradients of the iteration are written to memory first
// (this kernel is then step 1 of the iteration) and the sweeps read them from there, as they do downstream of
// a real gradient kernel.  Padding coordinates are written as zeros.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) synth_fill_kernel(const Params P) {
  if (*(volatile uint32_t*)&P.sc->err) return;
  const int m = blockIdx.y;
  Synth sy;
  sy.init(P, m, P.sc->k + 1);
  float4* __restrict__ g4 = reinterpret_cast<float4*>(P.g + (long long)m * P.ps);
  const uint32_t nv = (uint32_t)P.nv, v_full = (uint32_t)(P.p >> 2), stride = gridDim.x * blockDim.x;
  for (uint32_t v = blockIdx.x * blockDim.x + threadIdx.x; v < nv; v += stride)
    g4[v] = v < v_full ? sy.at4(v) : sy.at4_masked(v, P.p);
}

// ------------------------------------------------------------------------------------------------
// radius
// ------------------------------------------------------------------------------------------------
template <bool SYNTH>
__global__ void __launch_bounds__(512) radius_kernel(const Params P) {
  if (*(volatile uint32_t*)&P.sc->err) return;
  const int m = blockIdx.y;
  const unsigned long long k = P.sc->k;
  Synth sy;
  if (SYNTH) sy.init(P, m, k + 1);
  const float4* __restrict__ q4 = reinterpret_cast<const float4*>(P.qp + (long long)m * P.ps);
  const float4* __restrict__ g4 = SYNTH ? nullptr : reinterpret_cast<const float4*>(P.g + (long long)m * P.ps);
  // groups [0, nv_main) lie wholly inside the row; the (at most five) groups after them may contain
  // padding coordinates and take the masked path.  p < 2^32, so group indices fit 32 bits.
  const uint32_t nv = (uint32_t)P.nv, nv_main = (uint32_t)((P.p / 4) & ~1ll), stride = gridDim.x * blockDim.x;
  uint32_t mx = 0;
  // the ordering of |d| as unsigned bit patterns equals its ordering as floats, and puts inf and nan
  // above every finite value, so a non-finite entry surfaces in R
  uint32_t v = blockIdx.x * blockDim.x + threadIdx.x;
  for (; (unsigned long long)v + (kUnroll - 1) * (unsigned long long)stride < nv_main; v += kUnroll * stride) {
    float4 q[kUnroll], g[kUnroll];
#pragma unroll
    for (int j = 0; j < kUnroll; ++j) {
      q[j] = __ldg(q4 + (v + j * stride));
      g[j] = SYNTH ? sy.at4(v + j * stride) : __ldg(g4 + (v + j * stride));
    }
#pragma unroll
    for (int j = 0; j < kUnroll; ++j) {
      mx = max(mx, abs_bits(__fsub_rn(g[j].x, q[j].x)));
      mx = max(mx, abs_bits(__fsub_rn(g[j].y, q[j].y)));
      mx = max(mx, abs_bits(__fsub_rn(g[j].z, q[j].z)));
      mx = max(mx, abs_bits(__fsub_rn(g[j].w, q[j].w)));
    }
  }
  for (; v < nv_main; v += stride) {
    const float4 q = __ldg(q4 + v);
    const float4 g = SYNTH ? sy.at4(v) : __ldg(g4 + v);
    mx = max(mx, abs_bits(__fsub_rn(g.x, q.x)));
    mx = max(mx, abs_bits(__fsub_rn(g.y, q.y)));
    mx = max(mx, abs_bits(__fsub_rn(g.z, q.z)));
    mx = max(mx, abs_bits(__fsub_rn(g.w, q.w)));
  }
  if (blockIdx.x == 0 && nv_main + threadIdx.x < nv) {
    const uint32_t v = nv_main + threadIdx.x;
    const float4 q = __ldg(q4 + v);                      // padding of Q_prev and of a stored g is zero
    const float4 g = SYNTH ? sy.at4_masked(v, P.p) : __ldg(g4 + v);
    mx = max(mx, abs_bits(__fsub_rn(g.x, q.x)));
    mx = max(mx, abs_bits(__fsub_rn(g.y, q.y)));
    mx = max(mx, abs_bits(__fsub_rn(g.z, q.z)));
    mx = max(mx, abs_bits(__fsub_rn(g.w, q.w)));
  }
  mx = __reduce_max_sync(0xffffffffu, mx);
  __shared__ uint32_t sh[32];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  if (lane == 0) sh[w] = mx;
  __syncthreads();
  if (w == 0) {
    mx = (lane < ((blockDim.x + 31) >> 5)) ? sh[lane] : 0u;
    mx = __reduce_max_sync(0xffffffffu, mx);
    if (lane == 0) atomicMax(&P.Rbits[(k & 1ull) * P.M + m], mx);  // max is order independent
  }
}

// ------------------------------------------------------------------------------------------------
// code packing: the 4 codes of coordinates 4v..4v+3 form one 4b-bit field at bit 4vb of the row
// ------------------------------------------------------------------------------------------------
// All 32 lanes of a warp call this together with v = (a multiple of 32) + lane (the 1-bit and 3-bit packings
// combine neighbouring lanes); cw is the number of words of the row.
template <int B>
__device__ __forceinline__ void store_codes(uint32_t* row, uint32_t v, uint32_t y0, uint32_t y1, uint32_t y2,
                                            uint32_t y3, bool valid, long long cw) {
  // y_e = 0x4b000000 + code_e: the code sits in the low bits
  if (B == 3) {
    // eight neighbouring groups (32 coordinates) fill three words.  Lane pairs first join their 12-bit fields into
    // 24 bits A_0..A_3 (held by the even lanes of the octet); word j of the chunk is then cut out of A_j and A_j+1:
    // W0 = A0 | A1 << 24, W1 = A1 >> 8 | A2 << 16, W2 = A2 >> 16 | A3 << 8.
    const uint32_t field = valid ? ((y0 & 7u) | ((y1 & 7u) << 3) | ((y2 & 7u) << 6) | ((y3 & 7u) << 9)) : 0u;
    const uint32_t lane = threadIdx.x & 31u, r = lane & 7u, base = lane & 24u;
    const uint32_t pair = field | (__shfl_down_sync(0xffffffffu, field, 1) << 12);     // valid in even lanes
    const uint32_t j = r < 3u ? r : 0u;
    const uint32_t lo = __shfl_sync(0xffffffffu, pair, base + 2u * j);
    const uint32_t hi = __shfl_sync(0xffffffffu, pair, base + 2u * j + 2u);
    // (lo + hi 2^24) >> 8 j, 32 bits of it
    const uint32_t word_bits = __funnelshift_r(lo | (hi << 24), hi >> 8, 8u * j);
    const bool any_valid = __ballot_sync(0xffffffffu, valid) & (0xffu << base);
    const long long word = 3ll * (v >> 3) + r;
    if (any_valid && r < 3u && word < cw) row[word] = word_bits;
  } else if (B == 16) {
    if (valid) reinterpret_cast<uint2*>(row)[v] = make_uint2(__byte_perm(y0, y1, 0x5410), __byte_perm(y2, y3, 0x5410));
  } else if (B == 8) {
    if (valid) row[v] = __byte_perm(__byte_perm(y0, y1, 0x0040), __byte_perm(y2, y3, 0x0040), 0x5410);
  } else if (B == 4) {
    if (valid)
      reinterpret_cast<uint16_t*>(row)[v] =
          (uint16_t)((y0 & 15u) | ((y1 & 15u) << 4) | ((y2 & 15u) << 8) | ((y3 & 15u) << 12));
  } else if (B == 2) {
    if (valid) reinterpret_cast<uint8_t*>(row)[v] = (uint8_t)((y0 & 3u) | ((y1 & 3u) << 2) | ((y2 & 3u) << 4) | ((y3 & 3u) << 6));
  } else {  // B == 1: two neighbouring lanes share a byte; v and the lane index have the same parity
    uint32_t nib = valid ? ((y0 & 1u) | ((y1 & 1u) << 1) | ((y2 & 1u) << 2) | ((y3 & 1u) << 3)) : 0u;
    uint32_t hi = __shfl_down_sync(0xffffffffu, nib, 1);
    if (valid && !(v & 1)) reinterpret_cast<uint8_t*>(row)[v >> 1] = (uint8_t)(nib | (hi << 4));
  }
}

template <int B>
__device__ __forceinline__ void load_codes(const uint32_t* row, long long v, uint32_t c[4]) {
  if (B == 16) {
    uint2 w = __ldg(reinterpret_cast<const uint2*>(row) + v);
    c[0] = w.x & 0xffffu; c[1] = w.x >> 16; c[2] = w.y & 0xffffu; c[3] = w.y >> 16;
  } else if (B == 8) {
    uint32_t w = __ldg(row + v);
    c[0] = w & 255u; c[1] = (w >> 8) & 255u; c[2] = (w >> 16) & 255u; c[3] = w >> 24;
  } else if (B == 3) {
    const long long bit = 12ll * v;
    const uint32_t sh = (uint32_t)bit & 31u;
    const uint32_t lo = __ldg(row + (bit >> 5));
    const uint32_t hi = sh > 20u ? __ldg(row + (bit >> 5) + 1) : 0u;   // the field ends in the next word
    const uint32_t w = __funnelshift_r(lo, hi, sh);
    c[0] = w & 7u; c[1] = (w >> 3) & 7u; c[2] = (w >> 6) & 7u; c[3] = (w >> 9) & 7u;
  } else if (B == 4) {
    uint32_t w = __ldg(reinterpret_cast<const uint16_t*>(row) + v);
    c[0] = w & 15u; c[1] = (w >> 4) & 15u; c[2] = (w >> 8) & 15u; c[3] = (w >> 12) & 15u;
  } else if (B == 2) {
    uint32_t w = __ldg(reinterpret_cast<const uint8_t*>(row) + v);
    c[0] = w & 3u; c[1] = (w >> 2) & 3u; c[2] = (w >> 4) & 3u; c[3] = (w >> 6) & 3u;
  } else {
    uint32_t w = __ldg(reinterpret_cast<const uint8_t*>(row) + (v >> 1)) >> (4 * (int)(v & 1));
    c[0] = w & 1u; c[1] = (w >> 1) & 1u; c[2] = (w >> 2) & 1u; c[3] = (w >> 3) & 1u;
  }
}

// IEEE quotient x / s from y = RN(1/s): one product and two residual corrections (each residual is an
// exact fused multiply-add).  The second correction starts from a faithful quotient, which makes the
// result the correctly rounded one (Markstein's theorem); valid while nothing under- or overflows,
// which the caller guarantees by using it only for 2^-60 <= s <= 2^60.
__device__ __forceinline__ float div_by_reciprocal(float x, float s, float y) {
  float q = __fmul_rn(x, y);
  float r = __fmaf_rn(-s, q, x);
  q = __fmaf_rn(r, y, q);
  r = __fmaf_rn(-s, q, x);
  return __fmaf_rn(r, y, q);
}

// One coordinate of Eq. (5)/(6).  Returns 2^23 + code as a float bit pattern (code in the low bits);
// updates the two fp64 sums.
// FAST (2^-60 <= s <= 2^60): no clamp, |d| <= R bounds floor(t) by 2^b - 1 (t <= 2^b - 1/2 + rounding).
// Otherwise the grid step s = 2 tau R may be subnormal or zero although R > 0: the quotient then loses bits (or
// is x / 0) and floor(t) can leave [0, 2^b - 1], so the code is clamped to that range as Eq. (5) defines it, and
// s = 0 gives code 0 (the 0/0 reading used for R = 0).  Eq. (6) is applied as printed in every case.
template <bool FAST>
__device__ __forceinline__ uint32_t quantize_one(float g, float q, float R, float s, float y, float levels,
                                                 double& sdq, double& seps) {
  const float d = __fsub_rn(g, q);
  const float x = __fadd_rn(d, R);
  float fl, f;
  if (FAST) {
    const float t = __fadd_rn(div_by_reciprocal(x, s, y), 0.5f);
    fl = __fadd_rd(t, 8388608.0f);                  // 2^23 + floor(t): rounding down at unit spacing
    f = __fsub_rn(fl, 8388608.0f);                  // floor(t), exact
  } else {
    f = 0.f;
    if (s > 0.f) f = fminf(fmaxf(floorf(__fadd_rn(__fdiv_rn(x, s), 0.5f)), 0.f), levels);
    fl = __fadd_rn(f, 8388608.0f);
  }
  const float dq = __fsub_rn(__fmul_rn(s, f), R);   // Eq. (6): multiply, then subtract
  const float qn = __fadd_rn(q, dq);
  const float e = __fsub_rn(g, qn);
  sdq = fma((double)dq, (double)dq, sdq);           // the product of two fp32 values is exact in fp64
  seps = fma((double)e, (double)e, seps);
  return __float_as_uint(fl);
}

// Four coordinates of Eq. (5)/(6) with the code taken from a cheap candidate wherever that provably is the code of
// the exact evaluation, and from the exact evaluation otherwise.  Exact (reading of Eq. (5) used throughout):
// x = RN(d + R), u = RN(x / s), code = floor(RN(u + 1/2)).  Candidate: u' = RN(d y + c) in one fused operation,
// y = RN(1 / s), c = RN(R y).  With v = (d + R) / s <= 2 R / s =: L' (L' = (2^B - 1)(1 + O(2^-23))) and rho = 2^-24:
//   |u' - v| <= 2 rho v + rho L' / 2 + O(rho^2),   |u - v| <= 2 rho v + O(rho^2),   so   |u' - u| < 1.125 * 2^(B-22).
// Let f be the integer nearest to u' (one add of 2^23 in round-to-nearest) and w = u' - f.  When
// |w| <= 1/2 - 2^(B-21), u + 1/2 lies in [f + 0.875 * 2^(B-22), f + 1 - 0.875 * 2^(B-22)], several ulps of 2^B away
// from both integers, so floor(RN(u + 1/2)) = f.  Otherwise (for b = 8 about one coordinate in 4000) the whole group
// is redone with the exact quotient.  Codes, dQ and eps are those of quantize_one<true>, bit for bit.
// Acc = double: fp64 sums of exact products; Acc = float: the caller adds short runs of fp32 sums (see there).
template <int B, typename Acc>
__device__ __forceinline__ void quantize_group(const float4& g4, const float4& q4, float R, float s, float y, float c,
                                               Acc& adq, Acc& aeps, uint32_t (&yy)[4]) {
  static_assert(B <= 8, "the margin 2^(B-21) is only small for few levels");
  constexpr float kSafe = 0.5f - (float)(1u << B) * 0x1p-21f;
  const float g[4] = {g4.x, g4.y, g4.z, g4.w}, q[4] = {q4.x, q4.y, q4.z, q4.w};
  float fl[4], f[4];
  float worst = 0.f;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float u = __fmaf_rn(__fsub_rn(g[e], q[e]), y, c);
    fl[e] = __fadd_rn(u, 8388608.0f);          // 2^23 + (integer nearest to u')
    f[e] = __fsub_rn(fl[e], 8388608.0f);
    worst = fmaxf(worst, fabsf(__fsub_rn(u, f[e])));
  }
  if (worst > kSafe) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float x = __fadd_rn(__fsub_rn(g[e], q[e]), R);
      const float u = div_by_reciprocal(x, s, y);
      fl[e] = __fadd_rd(__fadd_rn(u, 0.5f), 8388608.0f);
      f[e] = __fsub_rn(fl[e], 8388608.0f);
    }
  }
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float dq = __fsub_rn(__fmul_rn(s, f[e]), R);   // Eq. (6): multiply, then subtract
    const float er = __fsub_rn(g[e], __fadd_rn(q[e], dq));
    if constexpr (sizeof(Acc) == 8) {
      adq = fma((double)dq, (double)dq, adq);           // the product of two fp32 values is exact in fp64
      aeps = fma((double)er, (double)er, aeps);
    } else {
      adq = __fmaf_rn(dq, dq, adq);
      aeps = __fmaf_rn(er, er, aeps);
    }
    yy[e] = __float_as_uint(fl[e]);
  }
}

// Skip rule (7a)+(7b), clocks, uploader list, counters: run by the last block of quantize_kernel.
// scratch: kTriggerScratchBytes of shared memory, 8-byte aligned, free for this block to use.
constexpr size_t kTriggerScratchBytes = 2 * 512 * sizeof(double) + kMaxWorkers * sizeof(uint32_t);
__device__ void trigger_stage(const Params& P, int bpw, unsigned char* scratch) {
  DevScalars* sc = P.sc;
  const unsigned long long k = sc->k;
  const int par = (int)(k & 1ull);
  const bool tracing = P.trace_cap > 0 && sc->trace_pos < (uint32_t)P.trace_cap;
  const long long trow = (long long)sc->trace_pos * P.M;
  __shared__ int nonfinite;
  if (threadIdx.x == 0) nonfinite = 0;
  __syncthreads();
  for (int m = threadIdx.x; m < P.M; m += blockDim.x)
    if (P.Rbits[par * P.M + m] >= 0x7f800000u) atomicOr(&nonfinite, 1);
  __syncthreads();
  if (nonfinite) {  // freeze: nothing of this iteration is applied
    if (threadIdx.x == 0) {
      sc->n_up = 0;
      atomicOr(&sc->err, 1u);
    }
    return;
  }
  // Sum of the block partials of every worker, in a fixed order.  This block runs alone at the end of the sweep,
  // so what counts is the number of dependent round trips to L2: with fewer workers than threads a worker's partials
  // are cut into strips summed by neighbouring threads (all loads of a strip independent), then the strips in order.
  double (*s_strip)[512] = reinterpret_cast<double (*)[512]>(scratch);                     // [2][512]
  uint32_t* s_Rb = reinterpret_cast<uint32_t*>(scratch + 2 * 512 * sizeof(double));       // radius bits, bit 31 = skip
  const int T = (int)blockDim.x;
  int tpw = 1;
  while (tpw < 16 && 2 * tpw * P.M <= T && 2 * tpw * P.M <= 512) tpw *= 2;
  if (tpw > 1) {
    const int len = (bpw + tpw - 1) / tpw;
    if ((int)threadIdx.x < P.M * tpw) {
      const int m = (int)threadIdx.x / tpw, j = (int)threadIdx.x % tpw;
      const double* pq = P.part_q + (long long)m * kMaxSweepBlocksPerWorker * 2;
      const int i1 = min(bpw, (j + 1) * len);
      double a = 0.0, e = 0.0;
#pragma unroll 16
      for (int i = j * len; i < i1; ++i) {
        a += __ldcg(pq + 2 * i);
        e += __ldcg(pq + 2 * i + 1);
      }
      s_strip[0][threadIdx.x] = a;
      s_strip[1][threadIdx.x] = e;
    }
    __syncthreads();
  }
  for (int m = threadIdx.x; m < P.M; m += blockDim.x) {
    double n_dq = 0.0, n_eps = 0.0;
    if (tpw > 1) {
      for (int j = 0; j < tpw; ++j) {
        n_dq += s_strip[0][m * tpw + j];
        n_eps += s_strip[1][m * tpw + j];
      }
    } else {
      const double* pq = P.part_q + (long long)m * kMaxSweepBlocksPerWorker * 2;
#pragma unroll 16
      for (int i = 0; i < bpw; ++i) {
        n_dq += __ldcg(pq + 2 * i);
        n_eps += __ldcg(pq + 2 * i + 1);
      }
    }
    double acc = 0.0;
    for (int d = 0; d < P.D; ++d) {
      const double term = (double)P.xi[d] * P.ring[(sc->ring_head + d) % P.D];
      acc = acc + term;
    }
    const double rhs = acc / P.trig_c + 3.0 * (n_eps + P.n_epshat[m]);
    const int t = P.clock[m];
    const bool crit_a = n_dq <= rhs;
    const bool crit_b = (P.clock_mode == 0) ? (t <= P.tbar) : (t + 2 <= P.tbar);
    const bool skip = crit_a && crit_b && !(P.flags & LAQ_FLAG_TRIGGER_OFF);
    if (skip) {
      P.clock[m] = t + 1;
    } else {
      P.clock[m] = 0;
      P.n_epshat[m] = n_eps;
    }
    P.skip[m] = skip ? 1 : 0;
    P.norms[3 * m + 0] = n_dq;
    P.norms[3 * m + 1] = n_eps;
    P.norms[3 * m + 2] = rhs;
    if (tracing) {
      P.t_skip[trow + m] = skip ? 1 : 0;
      P.t_R[trow + m] = __uint_as_float(P.Rbits[par * P.M + m]);
      P.t_ndq[trow + m] = n_dq;
      P.t_neps[trow + m] = n_eps;
      P.t_rhs[trow + m] = rhs;
    }
    P.Rbits[(par ^ 1) * P.M + m] = 0u;  // clear the other parity for the next iteration's max
    s_Rb[m] = P.Rbits[par * P.M + m] | (skip ? 0x80000000u : 0u);   // finite, so bit 31 is free
  }
  __syncthreads();
  if (threadIdx.x == 0) {   // uploader list in ascending worker order, from shared memory (no global round trips)
    const float levels = (float)((1u << P.b) - 1u);
    const float two_tau = __fmul_rn(2.0f, __fdiv_rn(1.0f, levels));
    int n = 0;
    for (int m = 0; m < P.M; ++m) {
      if (!(s_Rb[m] & 0x80000000u)) {
        const float R = __uint_as_float(s_Rb[m]);
        P.up_m[n] = m;
        P.up_q[n] = m;
        P.up_R[n] = R;
        P.up_s[n] = __fmul_rn(two_tau, R);
        ++n;
      }
    }
    sc->n_up = n;
    sc->uploads += (unsigned long long)n;
    sc->bits += (unsigned long long)n * ((P.flags & LAQ_FLAG_QUANT_OFF)
                                             ? 32ull * (unsigned long long)P.p
                                             : 32ull + (unsigned long long)P.b * (unsigned long long)P.p);
    if (tracing) P.t_up[sc->trace_pos] = n;
  }
}

// ---- asynchronous staging of a row through shared memory (quantize sweep over long rows) -----------------------
// Every warp owns a ring of kRingStages stages; a stage holds one tile of kRingGroups 16-byte groups of the warp's
// row of Q_prev and, when the gradients are read from memory, the same tile of g behind it.  One lane asks the
// copy engine for a stage's tiles (cp.async.bulk, completion counted in bytes on the stage's mbarrier) kRingStages
// tiles ahead of the one being worked on, so the loads in flight live in shared memory instead of in registers and
// no warp waits on a load it has just issued.  A stage is refilled after __syncwarp(): every lane has then read
// its groups.
#ifndef LAQ_RING_STAGES
#define LAQ_RING_STAGES 2
#endif
#ifndef LAQ_RING_U
#define LAQ_RING_U 8
#endif
constexpr int kRingStages = LAQ_RING_STAGES;
constexpr int kRingU = LAQ_RING_U;                 // groups per lane and tile
constexpr uint32_t kRingGroups = 32 * kRingU;      // 16-byte groups per tile (4 KB)
constexpr uint32_t kRingTileBytes = kRingGroups * 16;
constexpr int kRingMaxWarps = 16;                  // warps per block that can own a ring
// rows read from memory take the ring from this many coordinates on (shorter rows: the plain loop), in blocks of
// up to 8 warps (two tiles per stage: more warps would not fit the shared memory of an SM)
constexpr long long kRingMinStoredP = 1ll << 20;
__host__ __device__ constexpr bool stored_rows_take_ring(long long p, int threads) {
  return p >= kRingMinStoredP && threads <= 256;
}

// The per-worker sweep of quantize_kernel (R > 0).  FAST selects the reciprocal-based exact division.
// Groups [0, nv_main) lie wholly inside the row and run without masks; the few groups after them are
// handled by the first warp of the worker's first block with per-coordinate masks.  nv_main is even (a multiple
// of 8 for b = 3), so the lane pairs of the 1-bit packing (the lane octets of the 3-bit packing) never straddle
// the two parts.
// RING (FAST; rows generated in the kernel, or long rows read from memory): the full tiles of the row come through
// the warp's shared-memory ring (ring = the block's dynamic shared memory, bars = kRingStages mbarriers per warp);
// what is left of the main part (less than one tile) goes through the plain loop below.
template <bool SYNTH, int B, bool FAST, bool RING>
__device__ __forceinline__ void quantize_sweep(const Params& P, int m, unsigned long long k, float R, float s,
                                               double& sdq, double& seps, unsigned char* ring = nullptr,
                                               unsigned long long* bars = nullptr) {
  Synth sy;
  if (SYNTH) sy.init(P, m, k + 1);
  const float y = __fdiv_rn(1.0f, s), cy = __fmul_rn(R, y);
  const float levels = (float)((1u << B) - 1u);
  const float4* __restrict__ q4 = reinterpret_cast<const float4*>(P.qp + (long long)m * P.ps);
  const float4* __restrict__ g4 = SYNTH ? nullptr : reinterpret_cast<const float4*>(P.g + (long long)m * P.ps);
  uint32_t* row = P.codes + (long long)m * P.cw;
  const long long p = P.p;
  const uint32_t nv = (uint32_t)P.nv, nv_main = (uint32_t)((p / 4) & (B == 3 ? ~7ll : ~1ll)),
                 stride = gridDim.x * blockDim.x;
  const uint32_t lane = threadIdx.x & 31;
  uint32_t v = blockIdx.x * blockDim.x + threadIdx.x;
  constexpr int NC = LAQ_QUANT_CHAINS;
  double adq[NC], aeps[NC];
#pragma unroll
  for (int c = 0; c < NC; ++c) adq[c] = aeps[c] = 0.0;
  if constexpr (RING) {
    constexpr uint32_t NS = SYNTH ? 1u : 2u;                              // tiles per stage: Q_prev (and g)
    constexpr uint32_t kStageBytes = NS * kRingTileBytes;
    const uint32_t w = threadIdx.x >> 5, wpb = blockDim.x >> 5;
    const uint32_t gw = blockIdx.x * wpb + w, nw = gridDim.x * wpb;      // this warp among the worker's warps
    const uint32_t n_tiles = nv_main / kRingGroups;
    const uint32_t n_my = n_tiles > gw ? (n_tiles - gw + nw - 1) / nw : 0u;  // tiles gw, gw + nw, ...
    const float4* stage0 = reinterpret_cast<const float4*>(ring) + (size_t)w * kRingStages * NS * kRingGroups;
    const uint32_t stage_a = smem_addr(stage0), bar_a = smem_addr(bars + w * kRingStages);
    // test hook: this one warp issues no copies and polls with a short limit, so its waits run out with
    // nothing in flight (see laq_tune "starve_copies")
    const bool starved = P.starve != 0u && m == 0 && gw == 0;
    const uint32_t wait_limit = starved ? kStarvedWaitLimit : kRingWaitLimit;
    auto fetch = [&](uint32_t stage, size_t first_group) {
      const uint32_t dst = stage_a + stage * kStageBytes, bar = bar_a + 8 * stage;
      ring_expect(bar, kStageBytes);
      ring_copy(dst, q4 + first_group, kRingTileBytes, bar);
      if constexpr (!SYNTH) ring_copy(dst + kRingTileBytes, g4 + first_group, kRingTileBytes, bar);
    };
    if (lane == 0) {
      for (int st = 0; st < kRingStages; ++st) ring_bar_init(bar_a + 8 * st);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      if (!starved)
        for (uint32_t i = 0; i < (uint32_t)kRingStages && i < n_my; ++i) fetch(i, (size_t)(gw + i * nw) * kRingGroups);
    }
    __syncwarp();
    // per-lane state that advances by a constant per tile: first group of the tile for this lane, first group of
    // the tile kRingStages ahead, the current stage
    uint32_t v0 = gw * kRingGroups + lane;
    size_t ahead = (size_t)(gw + (uint32_t)kRingStages * nw) * kRingGroups;
    const uint32_t step_groups = nw * kRingGroups;
    uint32_t st = 0, parity = 0, done = 0;
    for (; done < n_my; ++done) {
      if (!__all_sync(0xffffffffu, ring_wait(bar_a + 8 * st, parity, wait_limit))) break;
      const float4* tile = stage0 + st * (NS * kRingGroups) + lane;
      uint32_t* out = row + v0;
      // the 4 kRingU coordinates of a lane in this tile are summed in fp32 (fused multiply-adds, 4 kRingU - 1
      // roundings: relative error of the run below 4 kRingU * 2^-24) and the run is then added in fp64; with
      // hundreds of thousands of runs per row the sums agree with the fp64 sums of exact products to ~1e-9
      float rdq = 0.f, reps = 0.f;
#pragma unroll
      for (int j = 0; j < kRingU; ++j) {
        const float4 q = tile[32 * j];
        float4 g;
        if constexpr (SYNTH) g = sy.at4(v0 + 32 * j);
        else g = tile[kRingGroups + 32 * j];
        uint32_t yy[4];
        if constexpr (B <= 8) {
          quantize_group<B>(g, q, R, s, y, cy, rdq, reps, yy);
        } else {
          yy[0] = quantize_one<true>(g.x, q.x, R, s, y, levels, adq[0 % NC], aeps[0 % NC]);
          yy[1] = quantize_one<true>(g.y, q.y, R, s, y, levels, adq[1 % NC], aeps[1 % NC]);
          yy[2] = quantize_one<true>(g.z, q.z, R, s, y, levels, adq[2 % NC], aeps[2 % NC]);
          yy[3] = quantize_one<true>(g.w, q.w, R, s, y, levels, adq[3 % NC], aeps[3 % NC]);
        }
        if constexpr (B == 8) out[32 * j] = __byte_perm(__byte_perm(yy[0], yy[1], 0x0040), __byte_perm(yy[2], yy[3], 0x0040), 0x5410);
        else store_codes<B>(row, v0 + 32 * j, yy[0], yy[1], yy[2], yy[3], true, P.cw);
      }
      if constexpr (B <= 8) {
        adq[0] += (double)rdq;
        aeps[0] += (double)reps;
      }
      __syncwarp();                                // every lane has read its groups: the stage may be refilled
      if (lane == 0 && done + kRingStages < n_my) fetch(st, ahead);
      ahead += step_groups;
      v0 += step_groups;
      if (++st == (uint32_t)kRingStages) {
        st = 0;
        parity ^= 1u;
      }
    }
    if (done < n_my) {
      // a wait ran out: record it, and before leaving give the copies still in flight (at most kRingStages stages,
      // this one included) the same bounded time to land, so that none writes into shared memory of a later block
      if (lane == 0) atomicOr(&P.sc->err, kErrRingWait);
      const uint32_t issued = min(n_my, done + (uint32_t)kRingStages);
      for (uint32_t i = done; i < issued; ++i) {
        ring_wait(bar_a + 8 * st, parity, wait_limit);
        if (++st == (uint32_t)kRingStages) {
          st = 0;
          parity ^= 1u;
        }
      }
    }
    v = n_tiles * kRingGroups + blockIdx.x * blockDim.x + threadIdx.x;   // what is left of the main part
  }
  // hot loop: every group of every lane of the warp is valid, no predicates
  for (; !RING && (unsigned long long)(v - lane + 31) + (kUnroll - 1) * (unsigned long long)stride < nv_main;
       v += kUnroll * stride) {
    float4 q[kUnroll], g[kUnroll];
#pragma unroll
    for (int j = 0; j < kUnroll; ++j) {
      q[j] = __ldg(q4 + (v + j * stride));
      g[j] = SYNTH ? sy.at4(v + j * stride) : __ldg(g4 + (v + j * stride));
    }
#pragma unroll
    for (int j = 0; j < kUnroll; ++j) {  // four independent accumulation chains per sum
      if constexpr (FAST && B <= 8) {
        uint32_t yy[4];
        quantize_group<B>(g[j], q[j], R, s, y, cy, adq[0], aeps[0], yy);
        store_codes<B>(row, v + j * stride, yy[0], yy[1], yy[2], yy[3], true, P.cw);
      } else {
        const uint32_t y0 = quantize_one<FAST>(g[j].x, q[j].x, R, s, y, levels, adq[0 % NC], aeps[0 % NC]);
        const uint32_t y1 = quantize_one<FAST>(g[j].y, q[j].y, R, s, y, levels, adq[1 % NC], aeps[1 % NC]);
        const uint32_t y2 = quantize_one<FAST>(g[j].z, q[j].z, R, s, y, levels, adq[2 % NC], aeps[2 % NC]);
        const uint32_t y3 = quantize_one<FAST>(g[j].w, q[j].w, R, s, y, levels, adq[3 % NC], aeps[3 % NC]);
        store_codes<B>(row, v + j * stride, y0, y1, y2, y3, true, P.cw);
      }
    }
  }
  if constexpr (NC == 4) {
    sdq += (adq[0] + adq[1]) + (adq[2] + adq[3]);
    seps += (aeps[0] + aeps[1]) + (aeps[2] + aeps[3]);
  } else {
#pragma unroll
    for (int c = 0; c < NC; ++c) {
      sdq += adq[c];
      seps += aeps[c];
    }
  }
  // remainder of the main part: all lanes of a warp run the same number of trips (the 1-bit packing
  // shuffles between lanes), invalid lanes compute on harmless operands and store nothing
  for (; v - lane < nv_main; v += stride) {
    const bool ok = v < nv_main;
    float4 q = make_float4(0.f, 0.f, 0.f, 0.f), g = q;
    if (ok) {
      q = __ldg(q4 + v);
      g = SYNTH ? sy.at4(v) : __ldg(g4 + v);
    }
    double a = 0.0, c = 0.0;
    const uint32_t y0 = quantize_one<FAST>(g.x, q.x, R, s, y, levels, a, c);
    const uint32_t y1 = quantize_one<FAST>(g.y, q.y, R, s, y, levels, a, c);
    const uint32_t y2 = quantize_one<FAST>(g.z, q.z, R, s, y, levels, a, c);
    const uint32_t y3 = quantize_one<FAST>(g.w, q.w, R, s, y, levels, a, c);
    if (ok) {
      sdq += a;
      seps += c;
    }
    store_codes<B>(row, v, y0, y1, y2, y3, ok, P.cw);
  }
  if (blockIdx.x == 0 && threadIdx.x < 32) {  // groups that may contain padding coordinates
    const uint32_t v = nv_main + threadIdx.x;
    const bool ok = v < nv;
    uint32_t yy[4] = {0x4b000000u, 0x4b000000u, 0x4b000000u, 0x4b000000u};
    if (ok) {
      const float4 q = __ldg(q4 + v);
      const float4 g = SYNTH ? sy.at4_masked(v, p) : __ldg(g4 + v);
      const float gg[4] = {g.x, g.y, g.z, g.w}, qq[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if (4ll * v + e < p) yy[e] = quantize_one<FAST>(gg[e], qq[e], R, s, y, levels, sdq, seps);
    }
    store_codes<B>(row, v, yy[0], yy[1], yy[2], yy[3], ok, P.cw);
  }
}

// R = 0: every code is zero (and so are dQ and eps)
template <int B>
__device__ __forceinline__ void zero_codes(const Params& P, int m) {
  uint32_t* row = P.codes + (long long)m * P.cw;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long w = (long long)blockIdx.x * blockDim.x + threadIdx.x; w < P.cw; w += stride) row[w] = 0u;
}

template <bool SYNTH, int B>
__global__ void __launch_bounds__(LAQ_QUANT_MAX_THREADS, LAQ_QUANT_MIN_BLOCKS) quantize_kernel(const Params P) {
  __shared__ double sh[32];
  __shared__ bool is_last;
  __shared__ __align__(8) unsigned long long ring_bars[kRingMaxWarps * kRingStages];
  // dynamic shared memory: the trigger stage's scratch and the warps' staging rings (the larger of both)
  extern __shared__ __align__(128) unsigned char ring_smem[];
  const int m = blockIdx.y;
  const bool frozen = *(volatile uint32_t*)&P.sc->err != 0;
  const unsigned long long k = P.sc->k;
  const uint32_t Rb = P.Rbits[(k & 1ull) * P.M + m];
  const float R = __uint_as_float(Rb);
  const bool finite = Rb < 0x7f800000u;
  double sdq = 0.0, seps = 0.0;
  if (!frozen && finite) {
    const float levels = (float)((1u << B) - 1u);
    const float s = __fmul_rn(__fmul_rn(2.0f, __fdiv_rn(1.0f, levels)), R);
    if (!(R > 0.f))
      zero_codes<B>(P, m);
    else if (s >= 0x1p-60f && s <= 0x1p60f) {
      if (SYNTH || stored_rows_take_ring(P.p, (int)blockDim.x))
        quantize_sweep<SYNTH, B, true, true>(P, m, k, R, s, sdq, seps, ring_smem, ring_bars);
      else if constexpr (!SYNTH)
        quantize_sweep<SYNTH, B, true, false>(P, m, k, R, s, sdq, seps);
    } else
      quantize_sweep<SYNTH, B, false, false>(P, m, k, R, s, sdq, seps);
  }
  const double tdq = block_sum(sdq, sh);
  const double teps = block_sum(seps, sh);
  if (threadIdx.x == 0) {
    double* pq = P.part_q + ((long long)m * kMaxSweepBlocksPerWorker + blockIdx.x) * 2;
    __stcg(pq, tdq);
    __stcg(pq + 1, teps);
    __threadfence();
    const uint32_t total = gridDim.x * gridDim.y;
    const uint32_t ticket = atomicAdd(&P.sc->cnt_quant, 1u);
    is_last = (ticket == total - 1);
    if (is_last) P.sc->cnt_quant = 0;
  }
  __syncthreads();
  if (is_last && !frozen) {
    __threadfence();
    if (*(volatile uint32_t*)&P.sc->err == 0) trigger_stage(P, gridDim.x, ring_smem);   // no block gave up on a tile
  }
}

// ------------------------------------------------------------------------------------------------
// Quantizer off (lazily aggregated gradients without quantization, the LAG baseline of Sec. 4; with the skip
// rule off as well: plain gradient descent, Eq. (2)).  The innovation g_m - Q_prev is sent as it is, so one
// sweep gives both its largest magnitude (kept for the report and the non-finite check) and its squared norm;
// eps is zero.  The last block applies the same skip rule.
// ------------------------------------------------------------------------------------------------
template <bool SYNTH>
__global__ void __launch_bounds__(512) innovation_kernel(const Params P) {
  __shared__ double sh[32];
  __shared__ uint32_t shm[32];
  __shared__ bool is_last;
  __shared__ __align__(8) unsigned char trig_scratch[kTriggerScratchBytes];
  const int m = blockIdx.y;
  const bool frozen = *(volatile uint32_t*)&P.sc->err != 0;
  const unsigned long long k = P.sc->k;
  double sdq = 0.0;
  uint32_t mx = 0;
  if (!frozen) {
    Synth sy;
    if (SYNTH) sy.init(P, m, k + 1);
    const float4* __restrict__ q4 = reinterpret_cast<const float4*>(P.qp + (long long)m * P.ps);
    const float4* __restrict__ g4 = SYNTH ? nullptr : reinterpret_cast<const float4*>(P.g + (long long)m * P.ps);
    const uint32_t nv = (uint32_t)P.nv, nv_main = (uint32_t)((P.p / 4) & ~1ll), stride = gridDim.x * blockDim.x;
    double acc[4] = {0.0, 0.0, 0.0, 0.0};
    auto take = [&](const float4& g, const float4& q) {
      const float d0 = __fsub_rn(g.x, q.x), d1 = __fsub_rn(g.y, q.y), d2 = __fsub_rn(g.z, q.z), d3 = __fsub_rn(g.w, q.w);
      mx = max(max(mx, abs_bits(d0)), max(abs_bits(d1), max(abs_bits(d2), abs_bits(d3))));
      acc[0] = fma((double)d0, (double)d0, acc[0]);
      acc[1] = fma((double)d1, (double)d1, acc[1]);
      acc[2] = fma((double)d2, (double)d2, acc[2]);
      acc[3] = fma((double)d3, (double)d3, acc[3]);
    };
    uint32_t v = blockIdx.x * blockDim.x + threadIdx.x;
    for (; (unsigned long long)v + (kUnroll - 1) * (unsigned long long)stride < nv_main; v += kUnroll * stride) {
      float4 q[kUnroll], g[kUnroll];
#pragma unroll
      for (int j = 0; j < kUnroll; ++j) {
        q[j] = __ldg(q4 + (v + j * stride));
        g[j] = SYNTH ? sy.at4(v + j * stride) : __ldg(g4 + (v + j * stride));
      }
#pragma unroll
      for (int j = 0; j < kUnroll; ++j) take(g[j], q[j]);
    }
    for (; v < nv_main; v += stride) take(SYNTH ? sy.at4(v) : __ldg(g4 + v), __ldg(q4 + v));
    if (blockIdx.x == 0 && nv_main + threadIdx.x < nv) {   // padding of Q_prev and of a stored g is zero
      const uint32_t vt = nv_main + threadIdx.x;
      take(SYNTH ? sy.at4_masked(vt, P.p) : __ldg(g4 + vt), __ldg(q4 + vt));
    }
    sdq = (acc[0] + acc[1]) + (acc[2] + acc[3]);
  }
  mx = __reduce_max_sync(0xffffffffu, mx);
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  if (lane == 0) shm[w] = mx;
  const double tdq = block_sum(sdq, sh);   // its barriers also publish shm
  if (w == 0) {
    mx = (lane < ((blockDim.x + 31) >> 5)) ? shm[lane] : 0u;
    mx = __reduce_max_sync(0xffffffffu, mx);
  }
  if (threadIdx.x == 0) {
    if (!frozen) atomicMax(&P.Rbits[(k & 1ull) * P.M + m], mx);
    double* pq = P.part_q + ((long long)m * kMaxSweepBlocksPerWorker + blockIdx.x) * 2;
    __stcg(pq, tdq);
    __stcg(pq + 1, 0.0);
    __threadfence();
    const uint32_t total = gridDim.x * gridDim.y;
    const uint32_t ticket = atomicAdd(&P.sc->cnt_quant, 1u);
    is_last = (ticket == total - 1);
    if (is_last) P.sc->cnt_quant = 0;
  }
  __syncthreads();
  if (is_last && !frozen) {
    __threadfence();
    trigger_stage(P, gridDim.x, trig_scratch);
  }
}

// ------------------------------------------------------------------------------------------------
// lazy aggregate + theta step
// ------------------------------------------------------------------------------------------------
#ifndef LAQ_AGG_AHEAD
#define LAQ_AGG_AHEAD 4
#endif
#ifndef LAQ_AGG_MIN_BLOCKS
#define LAQ_AGG_MIN_BLOCKS 5   // 48 registers, no spills
#endif
constexpr int kAggAhead = LAQ_AGG_AHEAD;  // uploaders whose row and code lines are requested into L2 ahead of use

// exact float of a code < 2^23 through the mantissa of 2^23
__device__ __forceinline__ float code_to_float(uint32_t c) { return __uint_as_float(0x4b000000u | c) - 8388608.0f; }

// grad^k is complete for group v: store it, take the step theta -= alpha grad (Eq. (4)) and add to the fp64 sums
// of ||alpha grad||^2 and ||theta||^2.
__device__ __forceinline__ void theta_step(const Params& P, uint32_t v, const float4& a, double& dsum, double& tsum) {
  reinterpret_cast<float4*>(P.agg)[v] = a;
  float4* th4 = reinterpret_cast<float4*>(P.theta);
  float4 th = th4[v];
  const float alpha = P.alpha;
  const float u0 = __fmul_rn(alpha, a.x), u1 = __fmul_rn(alpha, a.y), u2 = __fmul_rn(alpha, a.z),
              u3 = __fmul_rn(alpha, a.w);
  th.x = __fsub_rn(th.x, u0);
  th.y = __fsub_rn(th.y, u1);
  th.z = __fsub_rn(th.z, u2);
  th.w = __fsub_rn(th.w, u3);
  th4[v] = th;
  if (P.w1b != nullptr && 4ll * v < P.w1b_n) {   // the network's first-layer weights, as the tensor cores read them
    const __nv_bfloat162 lo = __floats2bfloat162_rn(th.x, th.y), hi = __floats2bfloat162_rn(th.z, th.w);
    uint2 pk;
    pk.x = *reinterpret_cast<const uint32_t*>(&lo);
    pk.y = *reinterpret_cast<const uint32_t*>(&hi);
    reinterpret_cast<uint2*>(P.w1b)[v] = pk;
  }
  dsum = fma((double)u0, (double)u0, dsum);
  dsum = fma((double)u1, (double)u1, dsum);
  dsum = fma((double)u2, (double)u2, dsum);
  dsum = fma((double)u3, (double)u3, dsum);
  tsum = fma((double)th.x, (double)th.x, tsum);
  tsum = fma((double)th.y, (double)th.y, tsum);
  tsum = fma((double)th.z, (double)th.z, tsum);
  tsum = fma((double)th.w, (double)th.w, tsum);
}

// Block partials of the two sums; the last block to arrive adds them in a fixed order, pushes ||alpha grad||^2 onto
// the ring of stored differences, writes the trace row and advances k.
__device__ __forceinline__ void aggregate_finish(const Params& P, double dsum, double tsum, double* sh, bool* is_last_sh) {
  const double bs = block_sum(dsum, sh);
  const double bt = block_sum(tsum, sh);
  if (threadIdx.x == 0) {
    __stcg(P.part_d + blockIdx.x, bs);
    __stcg(P.part_t + blockIdx.x, bt);
    __threadfence();
    const uint32_t ticket = atomicAdd(&P.sc->cnt_agg, 1u);
    *is_last_sh = (ticket == gridDim.x - 1);
    if (*is_last_sh) P.sc->cnt_agg = 0;
  }
  __syncthreads();
  if (!*is_last_sh) return;
  __threadfence();
  // ||theta^{k+1} - theta^k||^2 = ||alpha grad^k||^2 : fixed-order sum of the block partials
  double t = 0.0, t2 = 0.0;
  for (int i = threadIdx.x; i < (int)gridDim.x; i += blockDim.x) {
    t += __ldcg(P.part_d + i);
    t2 += __ldcg(P.part_t + i);
  }
  const double d2 = block_sum(t, sh);
  const double th2 = block_sum(t2, sh);
  if (threadIdx.x == 0) {
    DevScalars* sc = P.sc;
    sc->theta_sq = th2;
    const uint32_t head = (sc->ring_head + (uint32_t)P.D - 1u) % (uint32_t)P.D;
    P.ring[head] = d2;
    sc->ring_head = head;
    if (P.trace_cap > 0 && sc->trace_pos < (uint32_t)P.trace_cap) {
      P.t_d2[sc->trace_pos] = d2;
      double loss = 0.0;
      for (int m = 0; m < P.M; ++m) loss += P.loss_m[m];
      P.t_loss[sc->trace_pos] = loss;
      sc->trace_pos += 1;
    }
    sc->k += 1ull;
  }
}

template <int B>
__device__ __forceinline__ const void* code_address(const uint32_t* row, uint32_t v) {
  return reinterpret_cast<const uint8_t*>(row) +
         ((B == 1) ? (size_t)(v >> 1) : (B == 3) ? ((size_t)v * 3 / 2) & ~(size_t)3 : (size_t)v * (size_t)(B / 2));
}

// A thread owns groups v, v + stride, ...  Per group it holds only the aggregate in registers and walks the
// uploaders in ascending worker order; latency is covered by occupancy (few registers) and by requesting the
// lines of the uploaders ahead, and of theta, into L2 before they are needed.
template <int B>
__global__ void __launch_bounds__(256, LAQ_AGG_MIN_BLOCKS) aggregate_kernel(const Params P) {
  __shared__ int s_m[kMaxWorkers];     // row of the code buffer
  __shared__ int s_q[kMaxWorkers];     // row of Q_prev, -1: the uploader's Q_m lives in another context
  __shared__ float s_R[kMaxWorkers];
  __shared__ float s_s[kMaxWorkers];
  __shared__ double sh[32];
  __shared__ bool is_last;
  if (*(volatile uint32_t*)&P.sc->err) return;
  const int n_up = (int)P.sc->n_up;
  for (int u = threadIdx.x; u < n_up; u += blockDim.x) {
    s_m[u] = P.up_m[u];
    s_q[u] = P.up_q[u];
    s_R[u] = P.up_R[u];
    s_s[u] = P.up_s[u];
  }
  __syncthreads();
  // p < 2^32, so group indices fit 32 bits; groups >= v_full contain padding coordinates
  const uint32_t nv = (uint32_t)P.nv, v_full = (uint32_t)(P.p >> 2), stride = gridDim.x * blockDim.x;
  double dsum = 0.0, tsum = 0.0;
  for (uint32_t v = blockIdx.x * blockDim.x + threadIdx.x; v < nv; v += stride) {
    float4 a = reinterpret_cast<const float4*>(P.agg)[v];
    prefetch_l2(reinterpret_cast<const float4*>(P.theta) + v);
#pragma unroll
    for (int j = 0; j < kAggAhead; ++j)
      if (j < n_up) {
        if (s_q[j] >= 0) prefetch_l2(reinterpret_cast<const float4*>(P.qp + (long long)s_q[j] * P.ps) + v);
        prefetch_l2(code_address<B>(P.codes + (long long)s_m[j] * P.cw, v));
      }
    for (int u = 0; u < n_up; ++u) {
      if (u + kAggAhead < n_up) {
        const int qa = s_q[u + kAggAhead];
        if (qa >= 0) prefetch_l2(reinterpret_cast<const float4*>(P.qp + (long long)qa * P.ps) + v);
        prefetch_l2(code_address<B>(P.codes + (long long)s_m[u + kAggAhead] * P.cw, v));
      }
      const int qrow = s_q[u];
      uint32_t c[4];
      load_codes<B>(P.codes + (long long)s_m[u] * P.cw, v, c);
      const float R = s_R[u], s = s_s[u];
      // the server's recovery of the innovation from the message: dQ = 2 tau R q - R
      float d0 = __fsub_rn(__fmul_rn(s, code_to_float(c[0])), R);
      float d1 = __fsub_rn(__fmul_rn(s, code_to_float(c[1])), R);
      float d2 = __fsub_rn(__fmul_rn(s, code_to_float(c[2])), R);
      float d3 = __fsub_rn(__fmul_rn(s, code_to_float(c[3])), R);
      if (v >= v_full) {  // padding coordinates carry no innovation
        const long long i = 4ll * v;
        if (i >= P.p) d0 = 0.f;
        if (i + 1 >= P.p) d1 = 0.f;
        if (i + 2 >= P.p) d2 = 0.f;
        d3 = 0.f;
      }
      if (qrow >= 0) {    // the worker's own copy of Q_m moves with the server's (text after Eq. (6))
        float4* qptr = reinterpret_cast<float4*>(P.qp + (long long)qrow * P.ps) + v;
        float4 q = *qptr;
        q.x = __fadd_rn(q.x, d0);
        q.y = __fadd_rn(q.y, d1);
        q.z = __fadd_rn(q.z, d2);
        q.w = __fadd_rn(q.w, d3);
        *qptr = q;
      }
      a.x = __fadd_rn(a.x, d0);  // uploads are applied in ascending worker order
      a.y = __fadd_rn(a.y, d1);
      a.z = __fadd_rn(a.z, d2);
      a.w = __fadd_rn(a.w, d3);
    }
    theta_step(P, v, a, dsum, tsum);
  }
  aggregate_finish(P, dsum, tsum, sh, &is_last);
}

// Workers spread over several contexts: the list of ALL uploaders of the iteration (global indices, ascending, with
// their radii) replaces the list of local uploaders that the skip-rule stage left; the counters take the uploads of
// the other contexts.  Local uploaders read their code row and own a row of Q_prev; remote ones read the mailbox row
// of their global index.  One block.
__global__ void __launch_bounds__(256) merge_uploads_kernel(const Params P, int n, const int32_t* __restrict__ m_global,
                                                            const float* __restrict__ R) {
  DevScalars* sc = P.sc;
  if (*(volatile uint32_t*)&sc->err) return;
  const float levels = (float)((1u << P.b) - 1u);
  const float two_tau = __fmul_rn(2.0f, __fdiv_rn(1.0f, levels));
  for (int u = threadIdx.x; u < n; u += blockDim.x) {
    const int g = m_global[u];
    const int off = g - P.m_first;
    const bool local = off >= 0 && off % P.m_stride == 0 && off / P.m_stride < P.M;
    P.up_m[u] = local ? off / P.m_stride : P.M + g;     // mailbox rows follow the local rows
    P.up_q[u] = local ? off / P.m_stride : -1;
    P.up_R[u] = R[u];
    P.up_s[u] = __fmul_rn(two_tau, R[u]);
  }
  if (threadIdx.x == 0) {
    const unsigned long long extra = (unsigned long long)n - (unsigned long long)sc->n_up;   // the remote uploads
    sc->uploads += extra;
    sc->bits += extra * (32ull + (unsigned long long)P.b * (unsigned long long)P.p);
    sc->n_up = (uint32_t)n;
  }
}

// Quantizer off: an uploader's innovation is g_m - Q_prev itself and Q_prev becomes g_m.
template <bool SYNTH>
__global__ void __launch_bounds__(256, LAQ_AGG_MIN_BLOCKS) aggregate_raw_kernel(const Params P) {
  __shared__ int s_m[kMaxWorkers];
  __shared__ double sh[32];
  __shared__ bool is_last;
  if (*(volatile uint32_t*)&P.sc->err) return;
  const int n_up = (int)P.sc->n_up;
  const unsigned long long k = P.sc->k;
  __shared__ Synth s_sy[SYNTH ? kMaxWorkers : 1];
  for (int u = threadIdx.x; u < n_up; u += blockDim.x) {
    s_m[u] = P.up_m[u];
    if (SYNTH) s_sy[u].init(P, s_m[u], k + 1);
  }
  __syncthreads();
  const uint32_t nv = (uint32_t)P.nv, v_full = (uint32_t)(P.p >> 2), stride = gridDim.x * blockDim.x;
  double dsum = 0.0, tsum = 0.0;
  for (uint32_t v = blockIdx.x * blockDim.x + threadIdx.x; v < nv; v += stride) {
    float4 a = reinterpret_cast<const float4*>(P.agg)[v];
    prefetch_l2(reinterpret_cast<const float4*>(P.theta) + v);
#pragma unroll
    for (int j = 0; j < kAggAhead; ++j)
      if (j < n_up) {
        const int m1 = s_m[j];
        prefetch_l2(reinterpret_cast<const float4*>(P.qp + (long long)m1 * P.ps) + v);
        if (!SYNTH) prefetch_l2(reinterpret_cast<const float4*>(P.g + (long long)m1 * P.ps) + v);
      }
    for (int u = 0; u < n_up; ++u) {
      if (u + kAggAhead < n_up) {
        const int m1 = s_m[u + kAggAhead];
        prefetch_l2(reinterpret_cast<const float4*>(P.qp + (long long)m1 * P.ps) + v);
        if (!SYNTH) prefetch_l2(reinterpret_cast<const float4*>(P.g + (long long)m1 * P.ps) + v);
      }
      const int m = s_m[u];
      float4* qptr = reinterpret_cast<float4*>(P.qp + (long long)m * P.ps) + v;
      const float4 q = *qptr;
      float4 g;
      if (SYNTH) {
        const Synth sy = s_sy[u];
        g = (v >= v_full) ? sy.at4_masked(v, P.p) : sy.at4(v);
      } else {
        g = __ldg(reinterpret_cast<const float4*>(P.g + (long long)m * P.ps) + v);
      }
      {
        // Q_prev := g exactly.  The stored value is made to depend on the loaded one (AND with a kernel parameter
        // that is zero): a store issued while the load of the same address is still in flight was measured 3.6
        // times slower per uploader than one that waits for it.
        float4 t = g;
        t.x = __uint_as_float(__float_as_uint(g.x) | (__float_as_uint(q.x) & P.zero));
        *qptr = t;
      }
      a.x = __fadd_rn(a.x, __fsub_rn(g.x, q.x));  // uploads are applied in ascending worker order
      a.y = __fadd_rn(a.y, __fsub_rn(g.y, q.y));
      a.z = __fadd_rn(a.z, __fsub_rn(g.z, q.z));
      a.w = __fadd_rn(a.w, __fsub_rn(g.w, q.w));
    }
    theta_step(P, v, a, dsum, tsum);
  }
  aggregate_finish(P, dsum, tsum, sh, &is_last);
}

// ------------------------------------------------------------------------------------------------
// Small problems (M p up to 8192 padded coordinates): steps 2-5 of one iteration in ONE block, so that the
// iteration is not a chain of launches and cross-block hand-overs.  A warp owns a worker in the radius and
// quantize phases; the arithmetic and its order are those of the three sweep kernels.  With gbpw > 0 the block
// first combines the gbpw block partials of the linear-model gradient kernels (what grad_finalize_kernel does).
// ------------------------------------------------------------------------------------------------
constexpr int kSmallThreads = 1024;

template <int B>
__global__ void __launch_bounds__(kSmallThreads) small_iteration_kernel(const Params P, int gbpw) {
  __shared__ uint32_t s_Rb[kMaxWorkers];
  __shared__ double s_ndq[kMaxWorkers], s_neps[kMaxWorkers];
  __shared__ int s_m[kMaxWorkers];
  __shared__ float s_R[kMaxWorkers], s_s[kMaxWorkers];
  __shared__ uint8_t s_skip[kMaxWorkers];
  __shared__ double sh[32];
  __shared__ int s_nup, s_bad;
  DevScalars* sc = P.sc;
  if (*(volatile uint32_t*)&sc->err) return;
  const int t = threadIdx.x, lane = t & 31, w = t >> 5, nw = kSmallThreads / 32, M = P.M;
  const long long p = P.p;
  const uint32_t nv = (uint32_t)P.nv;
  const unsigned long long k = sc->k;
  const int par = (int)(k & 1ull);
  if (t == 0) s_bad = 0;
  // ---- step 1 (tail): block partials of the gradient kernels -> g_m, loss_m
  if (gbpw > 0) {
    const double inv_N = 1.0 / (double)P.Ntot;
    for (long long idx = t; idx < (long long)M * p; idx += kSmallThreads) {
      const int m = (int)(idx / p);
      const long long i = idx - (long long)m * p;
      const float* gp = P.gpart + (long long)m * gbpw * P.ps + i;
      double s = 0.0;
      for (int blk = 0; blk < gbpw; ++blk) s += (double)gp[(long long)blk * P.ps];
      const double share = (double)P.N[m] / (double)P.Ntot;
      P.g[(long long)m * P.ps + i] =
          (float)(s * (inv_N * batch_scale(P, m)) + share * (double)P.lambda * (double)P.theta[i]);
    }
    for (int m = t; m < M; m += kSmallThreads) {
      double l = 0.0;
      for (int blk = 0; blk < gbpw; ++blk) l += P.lpart[(long long)m * gbpw + blk];
      const double share = (double)P.N[m] / (double)P.Ntot;
      P.loss_m[m] = l * (inv_N * batch_scale(P, m)) + share * 0.5 * (double)P.lambda * sc->theta_sq;
    }
  }
  __syncthreads();
  // ---- radius: a warp per worker
  for (int m = w; m < M; m += nw) {
    const float4* q4 = reinterpret_cast<const float4*>(P.qp + (long long)m * P.ps);
    const float4* g4 = reinterpret_cast<const float4*>(P.g + (long long)m * P.ps);
    uint32_t mx = 0;
    for (uint32_t v = lane; v < nv; v += 32) {   // padding of Q_prev and g is zero
      const float4 q = q4[v], g = g4[v];
      mx = max(mx, abs_bits(__fsub_rn(g.x, q.x)));
      mx = max(mx, abs_bits(__fsub_rn(g.y, q.y)));
      mx = max(mx, abs_bits(__fsub_rn(g.z, q.z)));
      mx = max(mx, abs_bits(__fsub_rn(g.w, q.w)));
    }
    mx = __reduce_max_sync(0xffffffffu, mx);
    if (lane == 0) {
      s_Rb[m] = mx;
      if (mx >= 0x7f800000u) s_bad = 1;
    }
  }
  __syncthreads();
  if (s_bad) {  // freeze: nothing of this iteration is applied
    if (t == 0) {
      sc->n_up = 0;
      atomicOr(&sc->err, 1u);
    }
    return;
  }
  // ---- codes and the two norms: a warp per worker
  for (int m = w; m < M; m += nw) {
    const float R = __uint_as_float(s_Rb[m]);
    const float levels = (float)((1u << B) - 1u);
    const float s = __fmul_rn(__fmul_rn(2.0f, __fdiv_rn(1.0f, levels)), R);
    const bool fast = s >= 0x1p-60f && s <= 0x1p60f;
    const float y = __fdiv_rn(1.0f, s);
    const float4* q4 = reinterpret_cast<const float4*>(P.qp + (long long)m * P.ps);
    const float4* g4 = reinterpret_cast<const float4*>(P.g + (long long)m * P.ps);
    uint32_t* row = P.codes + (long long)m * P.cw;
    double sdq = 0.0, seps = 0.0;
    if (R > 0.f) {
      for (uint32_t v0 = 0; v0 < nv; v0 += 32) {   // all lanes make the same number of trips
        const uint32_t v = v0 + lane;
        const bool ok = v < nv;
        uint32_t yy[4] = {0x4b000000u, 0x4b000000u, 0x4b000000u, 0x4b000000u};
        if (ok) {
          const float4 q = q4[v], g = g4[v];
          const float gg[4] = {g.x, g.y, g.z, g.w}, qq[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
          for (int e = 0; e < 4; ++e)
            if (4ll * v + e < p)
              yy[e] = fast ? quantize_one<true>(gg[e], qq[e], R, s, y, levels, sdq, seps)
                           : quantize_one<false>(gg[e], qq[e], R, s, y, levels, sdq, seps);
        }
        store_codes<B>(row, v, yy[0], yy[1], yy[2], yy[3], ok, P.cw);
      }
    } else {
      for (long long wd = lane; wd < P.cw; wd += 32) row[wd] = 0u;
    }
    sdq = warp_sum(sdq);
    seps = warp_sum(seps);
    if (lane == 0) {
      s_ndq[m] = sdq;
      s_neps[m] = seps;
    }
  }
  __syncthreads();
  // ---- skip rule (7a) + clock (7b)
  const bool tracing = P.trace_cap > 0 && sc->trace_pos < (uint32_t)P.trace_cap;
  const long long trow = (long long)sc->trace_pos * M;
  for (int m = t; m < M; m += kSmallThreads) {
    const double n_dq = s_ndq[m], n_eps = s_neps[m];
    double acc = 0.0;
    for (int d = 0; d < P.D; ++d) {
      const double term = (double)P.xi[d] * P.ring[(sc->ring_head + d) % P.D];
      acc = acc + term;
    }
    const double rhs = acc / P.trig_c + 3.0 * (n_eps + P.n_epshat[m]);
    const int clk = P.clock[m];
    const bool crit_a = n_dq <= rhs;
    const bool crit_b = (P.clock_mode == 0) ? (clk <= P.tbar) : (clk + 2 <= P.tbar);
    const bool skip = crit_a && crit_b && !(P.flags & LAQ_FLAG_TRIGGER_OFF);
    if (skip) {
      P.clock[m] = clk + 1;
    } else {
      P.clock[m] = 0;
      P.n_epshat[m] = n_eps;
    }
    s_skip[m] = skip ? 1 : 0;
    P.skip[m] = skip ? 1 : 0;
    P.norms[3 * m + 0] = n_dq;
    P.norms[3 * m + 1] = n_eps;
    P.norms[3 * m + 2] = rhs;
    P.Rbits[par * M + m] = s_Rb[m];
    P.Rbits[(par ^ 1) * M + m] = 0u;
    if (tracing) {
      P.t_skip[trow + m] = skip ? 1 : 0;
      P.t_R[trow + m] = __uint_as_float(s_Rb[m]);
      P.t_ndq[trow + m] = n_dq;
      P.t_neps[trow + m] = n_eps;
      P.t_rhs[trow + m] = rhs;
    }
  }
  __syncthreads();
  if (t == 0) {
    const float levels = (float)((1u << B) - 1u);
    const float two_tau = __fmul_rn(2.0f, __fdiv_rn(1.0f, levels));
    int n = 0;
    for (int m = 0; m < M; ++m) {
      if (!s_skip[m]) {
        const float R = __uint_as_float(s_Rb[m]);
        s_m[n] = m;
        s_R[n] = R;
        s_s[n] = __fmul_rn(two_tau, R);
        ++n;
      }
    }
    s_nup = n;
    sc->n_up = n;
    sc->uploads += (unsigned long long)n;
    sc->bits += (unsigned long long)n * (32ull + (unsigned long long)B * (unsigned long long)p);
    if (tracing) P.t_up[sc->trace_pos] = n;
  }
  __syncthreads();
  // ---- lazy aggregate + theta step
  const int n_up = s_nup;
  float4* agg4 = reinterpret_cast<float4*>(P.agg);
  float4* th4 = reinterpret_cast<float4*>(P.theta);
  const float alpha = P.alpha;
  double dsum = 0.0, tsum = 0.0;
  for (uint32_t v = t; v < nv; v += kSmallThreads) {
    float4 a = agg4[v];
    const long long i = 4ll * v;
    for (int u = 0; u < n_up; ++u) {
      const int m = s_m[u];
      const float R = s_R[u], s = s_s[u];
      float4* qrow = reinterpret_cast<float4*>(P.qp + (long long)m * P.ps) + v;
      float4 q = *qrow;
      uint32_t c[4];
      load_codes<B>(P.codes + (long long)m * P.cw, v, c);
      float d0 = __fsub_rn(__fmul_rn(s, code_to_float(c[0])), R);
      float d1 = __fsub_rn(__fmul_rn(s, code_to_float(c[1])), R);
      float d2 = __fsub_rn(__fmul_rn(s, code_to_float(c[2])), R);
      float d3 = __fsub_rn(__fmul_rn(s, code_to_float(c[3])), R);
      if (i >= p) d0 = 0.f;        // padding coordinates carry no innovation
      if (i + 1 >= p) d1 = 0.f;
      if (i + 2 >= p) d2 = 0.f;
      if (i + 3 >= p) d3 = 0.f;
      q.x = __fadd_rn(q.x, d0);
      q.y = __fadd_rn(q.y, d1);
      q.z = __fadd_rn(q.z, d2);
      q.w = __fadd_rn(q.w, d3);
      *qrow = q;
      a.x = __fadd_rn(a.x, d0);
      a.y = __fadd_rn(a.y, d1);
      a.z = __fadd_rn(a.z, d2);
      a.w = __fadd_rn(a.w, d3);
    }
    agg4[v] = a;
    float4 th = th4[v];
    const float u0 = __fmul_rn(alpha, a.x), u1 = __fmul_rn(alpha, a.y), u2 = __fmul_rn(alpha, a.z),
                u3 = __fmul_rn(alpha, a.w);
    th.x = __fsub_rn(th.x, u0);
    th.y = __fsub_rn(th.y, u1);
    th.z = __fsub_rn(th.z, u2);
    th.w = __fsub_rn(th.w, u3);
    th4[v] = th;
    dsum = fma((double)u0, (double)u0, dsum);
    dsum = fma((double)u1, (double)u1, dsum);
    dsum = fma((double)u2, (double)u2, dsum);
    dsum = fma((double)u3, (double)u3, dsum);
    tsum = fma((double)th.x, (double)th.x, tsum);
    tsum = fma((double)th.y, (double)th.y, tsum);
    tsum = fma((double)th.z, (double)th.z, tsum);
    tsum = fma((double)th.w, (double)th.w, tsum);
  }
  const double d2 = block_sum(dsum, sh);
  const double th2 = block_sum(tsum, sh);
  if (t == 0) {
    sc->theta_sq = th2;
    const uint32_t head = (sc->ring_head + (uint32_t)P.D - 1u) % (uint32_t)P.D;
    P.ring[head] = d2;
    sc->ring_head = head;
    if (tracing) {
      P.t_d2[sc->trace_pos] = d2;
      double loss = 0.0;
      for (int m = 0; m < M; ++m) loss += P.loss_m[m];
      P.t_loss[sc->trace_pos] = loss;
      sc->trace_pos += 1;
    }
    sc->k += 1ull;
  }
}

template <bool SYNTH, int B>
void launch_quant_one(const Params& P, dim3 grid, int threads, size_t smem, cudaStream_t st) {
  // more than the default 48 KB of dynamic shared memory has to be asked for (a failure shows up in the launch)
  if (smem > 40 * 1024)
    cudaFuncSetAttribute(quantize_kernel<SYNTH, B>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  quantize_kernel<SYNTH, B><<<grid, threads, smem, st>>>(P);
}

template <bool SYNTH>
void launch_quant_b(const Params& P, dim3 grid, int threads, cudaStream_t st) {
  // rows generated in the kernel, long rows read from memory: every warp stages its tiles of Q_prev (and of g)
  // through a ring in dynamic shared memory
  const size_t ring = SYNTH ? (size_t)(threads / 32) * kRingStages * kRingTileBytes
                            : (stored_rows_take_ring(P.p, threads) ? (size_t)(threads / 32) * kRingStages * 2 * kRingTileBytes : 0);
  const size_t smem = ring > kTriggerScratchBytes ? ring : kTriggerScratchBytes;
  switch (P.b) {
    case 1: launch_quant_one<SYNTH, 1>(P, grid, threads, smem, st); break;
    case 2: launch_quant_one<SYNTH, 2>(P, grid, threads, smem, st); break;
    case 3: launch_quant_one<SYNTH, 3>(P, grid, threads, smem, st); break;
    case 4: launch_quant_one<SYNTH, 4>(P, grid, threads, smem, st); break;
    case 8: launch_quant_one<SYNTH, 8>(P, grid, threads, smem, st); break;
    default: launch_quant_one<SYNTH, 16>(P, grid, threads, smem, st); break;
  }
}

}  // namespace

int sweep_blocks_per_worker(const Params& P, const LaunchShape& ls) {
  // one resident wave: M x bpw blocks ~ SMs x blocks per SM, never more blocks than 16-byte groups
  long long want = ((long long)kNumSMs * ls.sweep_blocks_per_sm + P.M - 1) / P.M;
  // a thread should have at least 8 groups of 16 bytes: below that the per-block reductions dominate
  long long need = (P.nv + 8ll * ls.sweep_threads - 1) / (8ll * ls.sweep_threads);
  long long bpw = want < need ? want : need;
  if (bpw < 1) bpw = 1;
  if (bpw > kMaxSweepBlocksPerWorker) bpw = kMaxSweepBlocksPerWorker;
  return (int)bpw;
}

int aggregate_blocks(const Params& P, const LaunchShape& ls) {
  long long want = (long long)kNumSMs * ls.agg_blocks_per_sm;
  long long need = (P.nv + ls.agg_threads - 1) / ls.agg_threads;
  long long nb = want < need ? want : need;
  return (int)(nb < 1 ? 1 : nb);
}

int sweep_tile_groups() { return (int)kRingGroups; }

int launch_theta_sq(const Params& P, cudaStream_t st) {
  theta_sq_kernel<<<1, 1024, 0, st>>>(P);
  return 1;
}

bool generated_in_sweeps(const Params& P) { return P.model == LAQ_MODEL_SYNTH && !(P.flags & LAQ_FLAG_STORE_G); }

int launch_synth_fill(const Params& P, cudaStream_t st) {
  long long nb = (P.nv + 256 * 8 - 1) / (256 * 8);
  const long long cap = ((long long)kNumSMs * 16 + P.M - 1) / P.M;
  if (nb > cap) nb = cap;
  synth_fill_kernel<<<dim3((unsigned)(nb < 1 ? 1 : nb), P.M), 256, 0, st>>>(P);
  return 1;
}

bool small_iteration_applies(const Params& P) {
  return P.model != LAQ_MODEL_SYNTH && !(P.flags & LAQ_FLAG_QUANT_OFF) && (long long)P.M * P.ps <= 8192 &&
         P.M_total == P.M;
}

int launch_small_iteration(const Params& P, int gbpw_finalize, cudaStream_t st) {
  switch (P.b) {
    case 1: small_iteration_kernel<1><<<1, kSmallThreads, 0, st>>>(P, gbpw_finalize); break;
    case 2: small_iteration_kernel<2><<<1, kSmallThreads, 0, st>>>(P, gbpw_finalize); break;
    case 3: small_iteration_kernel<3><<<1, kSmallThreads, 0, st>>>(P, gbpw_finalize); break;
    case 4: small_iteration_kernel<4><<<1, kSmallThreads, 0, st>>>(P, gbpw_finalize); break;
    case 8: small_iteration_kernel<8><<<1, kSmallThreads, 0, st>>>(P, gbpw_finalize); break;
    default: small_iteration_kernel<16><<<1, kSmallThreads, 0, st>>>(P, gbpw_finalize); break;
  }
  return 1;
}

int launch_radius(const Params& P, const LaunchShape& ls, cudaStream_t st) {
  dim3 grid(sweep_blocks_per_worker(P, ls), P.M);
  if (generated_in_sweeps(P))
    radius_kernel<true><<<grid, ls.sweep_threads, 0, st>>>(P);
  else
    radius_kernel<false><<<grid, ls.sweep_threads, 0, st>>>(P);
  return 1;
}

int launch_innovation_trigger(const Params& P, const LaunchShape& ls, cudaStream_t st) {
  dim3 grid(sweep_blocks_per_worker(P, ls), P.M);
  if (generated_in_sweeps(P))
    innovation_kernel<true><<<grid, ls.sweep_threads, 0, st>>>(P);
  else
    innovation_kernel<false><<<grid, ls.sweep_threads, 0, st>>>(P);
  return 1;
}

int launch_quantize_trigger(const Params& P, const LaunchShape& ls, cudaStream_t st) {
  dim3 grid(sweep_blocks_per_worker(P, ls), P.M);
  if (generated_in_sweeps(P))
    launch_quant_b<true>(P, grid, ls.sweep_threads, st);
  else
    launch_quant_b<false>(P, grid, ls.sweep_threads, st);
  return 1;
}

int launch_merge_uploads(const Params& P, int n, const int32_t* d_m, const float* d_R, cudaStream_t st) {
  merge_uploads_kernel<<<1, 256, 0, st>>>(P, n, d_m, d_R);
  return 1;
}

int launch_aggregate(const Params& P, const LaunchShape& ls, cudaStream_t st) {
  const int nb = aggregate_blocks(P, ls);
  if (P.flags & LAQ_FLAG_QUANT_OFF) {
    if (generated_in_sweeps(P))
      aggregate_raw_kernel<true><<<nb, ls.agg_threads, 0, st>>>(P);
    else
      aggregate_raw_kernel<false><<<nb, ls.agg_threads, 0, st>>>(P);
    return 1;
  }
  switch (P.b) {
    case 1: aggregate_kernel<1><<<nb, ls.agg_threads, 0, st>>>(P); break;
    case 2: aggregate_kernel<2><<<nb, ls.agg_threads, 0, st>>>(P); break;
    case 3: aggregate_kernel<3><<<nb, ls.agg_threads, 0, st>>>(P); break;
    case 4: aggregate_kernel<4><<<nb, ls.agg_threads, 0, st>>>(P); break;
    case 8: aggregate_kernel<8><<<nb, ls.agg_threads, 0, st>>>(P); break;
    default: aggregate_kernel<16><<<nb, ls.agg_threads, 0, st>>>(P); break;
  }
  return 1;
}

}  // namespace laq
