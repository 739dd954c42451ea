// laq_quantize_worker_static: the quantizer of one worker (radius, codes, the two squared norms)
// for callers that are not allowed to allocate device memory.
//
// Who needs this: a host application that has handed the whole GPU to its own memory pool (so a
// cudaMalloc made on its behalf either fails or steals from that pool), or one that runs the
// quantizer inside a latency-critical loop where cudaMalloc/cudaFree are banned because they
// synchronise the device.  Such a caller can provide inputs and outputs, but has nowhere to put
// the few kilobytes of reduction scratch that the kernels need (the running maximum, the
// per-block partial sums and the "last block" ticket).
//
// Here that scratch lives in a file-scope __device__ array.  Every GPU that loads this library
// holds the array (kStaticScratchBytes) until the process exits.  All calls share it, and it keeps
// whatever the previous call left, so each call first clears the words that must start at zero.
// Two calls whose kernels overlap on the same GPU (different streams, or different host threads)
// race on the scratch and produce garbage: serialise them.
//
// In host code the array's name is only a handle, not a device address.  The first call on each
// device asks the runtime for the real address (cudaGetSymbolAddress with that device current),
// checks the result, caches it, and passes it to the kernels.  That first call also loads the
// module onto the device, so make it once during start-up, before any stream capture begins.
// The cached address belongs to the device's primary context: a host that destroys that context
// (cudaDeviceReset) must not call this entry point on the device again in the same process.
#include <cuda_runtime.h>
#include <stdint.h>

#include <cstdio>
#include <mutex>

#include "laq.h"

namespace {

constexpr int kThreads = 256;
constexpr int kMaxBlocks = 2048;                 // partial-sum slots in the static scratch
constexpr long long kMaxP = 1ll << 31;           // coordinates per call
constexpr int kMaxDevices = 64;

struct StaticScratch {
  uint32_t r_bits;        // running max |g - Q_prev| as float bits      (cleared per call)
  uint32_t ticket;        // blocks finished                              (cleared per call)
  uint32_t pad[62];
  double part[kMaxBlocks][2];   // per-block partial ||dQ||^2, ||eps||^2 (fully rewritten per call)
};
constexpr size_t kStaticScratchBytes = sizeof(StaticScratch);  // 33 024 bytes

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ double block_sum(double v, double* sh) {
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

// R = max_i |g_i - q_i| into scratch->r_bits (unsigned order of |x| bit patterns = float order).
__global__ void __launch_bounds__(kThreads) static_radius_kernel(const float* __restrict__ g,
                                                                  const float* __restrict__ q, long long p,
                                                                  StaticScratch* sc) {
  uint32_t mx = 0;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < p; i += stride)
    mx = max(mx, __float_as_uint(__fsub_rn(__ldg(g + i), __ldg(q + i))) & 0x7fffffffu);
  mx = __reduce_max_sync(0xffffffffu, mx);
  __shared__ uint32_t sh[32];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  if (lane == 0) sh[w] = mx;
  __syncthreads();
  if (w == 0) {
    mx = (lane < kThreads / 32) ? sh[lane] : 0u;
    mx = __reduce_max_sync(0xffffffffu, mx);
    if (lane == 0) atomicMax(&sc->r_bits, mx);
  }
}

// Codes of Eq. (5), packed b bits each (code i at bit i b of the stream), and the two fp64 sums.
// One thread handles 32/B consecutive coordinates, i.e. exactly one 32-bit word of the stream.
template <int B>
__global__ void __launch_bounds__(kThreads) static_quantize_kernel(const float* __restrict__ g,
                                                                    const float* __restrict__ q, long long p,
                                                                    uint32_t* __restrict__ codes, float* R_out,
                                                                    double* norms_out, StaticScratch* sc) {
  constexpr int PER = 32 / B;
  __shared__ double sh[32];
  __shared__ bool is_last;
  const uint32_t rb = sc->r_bits;
  const float R = __uint_as_float(rb);
  const bool finite = rb < 0x7f800000u, live = finite && R > 0.f;   // R = 0: all codes 0, both norms 0
  const float levels = (float)((1u << B) - 1u);
  const float s = __fmul_rn(__fmul_rn(2.0f, __fdiv_rn(1.0f, levels)), R);
  double sdq = 0.0, seps = 0.0;
  const long long n_words = (p * B + 31) / 32, stride = (long long)gridDim.x * blockDim.x;
  for (long long wd = (long long)blockIdx.x * blockDim.x + threadIdx.x; wd < n_words; wd += stride) {
    uint32_t word = 0;
#pragma unroll
    for (int e = 0; e < PER; ++e) {
      const long long i = wd * PER + e;
      if (live && i < p) {
        const float gi = __ldg(g + i), qi = __ldg(q + i);
        const float d = __fsub_rn(gi, qi);
        // a grid step that underflowed to zero makes Eq. (5) x / 0: code 0, as for R = 0
        const float f = s > 0.f ? fminf(fmaxf(floorf(__fadd_rn(__fdiv_rn(__fadd_rn(d, R), s), 0.5f)), 0.f), levels) : 0.f;
        const float dq = __fsub_rn(__fmul_rn(s, f), R);
        const float e_ = __fsub_rn(gi, __fadd_rn(qi, dq));
        sdq = fma((double)dq, (double)dq, sdq);
        seps = fma((double)e_, (double)e_, seps);
        word |= (uint32_t)f << (e * B);
      }
    }
    if (finite) codes[wd] = word;
  }
  const double tdq = block_sum(sdq, sh);
  const double teps = block_sum(seps, sh);
  if (threadIdx.x == 0) {
    __stcg(&sc->part[blockIdx.x][0], tdq);
    __stcg(&sc->part[blockIdx.x][1], teps);
    __threadfence();
    is_last = atomicAdd(&sc->ticket, 1u) == gridDim.x - 1;
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  double a = 0.0, c = 0.0;
  if (threadIdx.x == 0) {  // fixed order over the block partials
    for (unsigned i = 0; i < gridDim.x; ++i) {
      a += __ldcg(&sc->part[i][0]);
      c += __ldcg(&sc->part[i][1]);
    }
    *R_out = R;
    norms_out[0] = a;
    norms_out[1] = c;
  }
}

std::mutex g_mutex;
StaticScratch* g_scratch_addr[kMaxDevices] = {nullptr};

laq_status set_err(char* errbuf, size_t errlen, laq_status st, const char* msg) {
  if (errbuf && errlen) snprintf(errbuf, errlen, "%s", msg);
  return st;
}

}  // namespace

extern "C" laq_status laq_quantize_worker_static(const float* d_g, const float* d_qprev, int64_t p, int32_t b,
                                                 uint32_t* d_codes, float* d_R, double* d_norms,
                                                 void* cuda_stream, char* errbuf, size_t errbuf_len) {
  if (errbuf && errbuf_len) errbuf[0] = 0;
  if (!d_g || !d_qprev || !d_codes || !d_R || !d_norms) return set_err(errbuf, errbuf_len, LAQ_EINVAL, "null pointer");
  if (!(b == 1 || b == 2 || b == 4 || b == 8 || b == 16)) return set_err(errbuf, errbuf_len, LAQ_EINVAL, "b must be 1, 2, 4, 8 or 16");
  if (p < 1) return set_err(errbuf, errbuf_len, LAQ_EINVAL, "p must be positive");
  if (p > kMaxP) return set_err(errbuf, errbuf_len, LAQ_EINVAL, "p exceeds the static-scratch variant's limit of 2^31 coordinates per call");
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices)
    return set_err(errbuf, errbuf_len, LAQ_ECUDA, "no current CUDA device (or device ordinal >= 64)");
  // the scratch used is the current device's: inputs that live on another GPU would make the kernels run there
  // against this device's scratch address
  cudaPointerAttributes attr;
  if (cudaPointerGetAttributes(&attr, d_g) != cudaSuccess) {
    cudaGetLastError();
    return set_err(errbuf, errbuf_len, LAQ_EINVAL, "d_g is not a pointer the CUDA runtime knows");
  }
  if ((attr.type == cudaMemoryTypeDevice || attr.type == cudaMemoryTypeManaged) && attr.device != dev)
    return set_err(errbuf, errbuf_len, LAQ_EINVAL, "the buffers live on another GPU than the current device: make their device current for the call");
  StaticScratch* sc = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_scratch_addr[dev]) {  // once per device, with that device current
      void* ptr = nullptr;
      cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
      if (e != cudaSuccess || !ptr) {
        cudaGetLastError();
        return set_err(errbuf, errbuf_len, LAQ_ECUDA, "cudaGetSymbolAddress failed for the static scratch");
      }
      g_scratch_addr[dev] = (StaticScratch*)ptr;
    }
    sc = g_scratch_addr[dev];
  }
  cudaStream_t st = (cudaStream_t)cuda_stream;
  // the array keeps the previous call's contents: clear the running max and the ticket
  if (cudaMemsetAsync(sc, 0, 256, st) != cudaSuccess) return set_err(errbuf, errbuf_len, LAQ_ECUDA, "cudaMemsetAsync failed");
  long long want = (p + kThreads - 1) / kThreads;
  const int nb_r = (int)(want < kMaxBlocks ? want : kMaxBlocks);
  static_radius_kernel<<<nb_r, kThreads, 0, st>>>(d_g, d_qprev, p, sc);
  const long long n_words = (p * b + 31) / 32;
  want = (n_words + kThreads - 1) / kThreads;
  const int nb_q = (int)(want < kMaxBlocks ? want : kMaxBlocks);
  switch (b) {
    case 1: static_quantize_kernel<1><<<nb_q, kThreads, 0, st>>>(d_g, d_qprev, p, d_codes, d_R, d_norms, sc); break;
    case 2: static_quantize_kernel<2><<<nb_q, kThreads, 0, st>>>(d_g, d_qprev, p, d_codes, d_R, d_norms, sc); break;
    case 4: static_quantize_kernel<4><<<nb_q, kThreads, 0, st>>>(d_g, d_qprev, p, d_codes, d_R, d_norms, sc); break;
    case 8: static_quantize_kernel<8><<<nb_q, kThreads, 0, st>>>(d_g, d_qprev, p, d_codes, d_R, d_norms, sc); break;
    default: static_quantize_kernel<16><<<nb_q, kThreads, 0, st>>>(d_g, d_qprev, p, d_codes, d_R, d_norms, sc); break;
  }
  if (cudaGetLastError() != cudaSuccess) return set_err(errbuf, errbuf_len, LAQ_ECUDA, "kernel launch failed");
  return LAQ_OK;
}
