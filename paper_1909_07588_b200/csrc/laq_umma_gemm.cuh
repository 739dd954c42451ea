// A bf16 x bf16 -> fp32 "TN" product on the 5th-generation tensor cores (tcgen05), used by the two large
// products of the ReLU-network gradient:
//     D[i][j] = sum_k A[i][k] * B[j][k]        A: [rows_a][K] row-major, B: [rows_b][K] row-major (both K-major)
// One CTA computes one 128 x NT tile of D (NT a multiple of 16, 16 <= NT <= 256):
//   warp 0     one lane issues the TMA loads (cp.async.bulk.tensor, 128-byte swizzle; every block fetches its own tiles) of the
//              128 x 64 tile of A and the NT x 64 tile of B into a ring of kStages shared-memory stages;
//   warp 1     allocates tensor memory; one lane issues tcgen05.mma (M = 128, N = NT, K = 16, four per stage) with
//              the accumulator in tensor memory, and commits each stage back to the loader through an mbarrier;
//   warps 2-5  epilogue: tcgen05.ld moves the accumulator to registers (a thread owns one row of the tile) and
//              hands 32-column chunks to the caller's functor.
// Rows or columns of a tile that lie outside the tensors are filled with zeros by the TMA unit.
// Every mbarrier wait is bounded: when a wait runs out, the thread records it in *err_flag, stops waiting, and the
// block still reaches its final barrier and frees its tensor memory.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace laq {
namespace umma {

constexpr int kTileM = 128;
constexpr int kBlockK = 64;        // bf16 elements per stage along K: 128 bytes, one swizzle row
constexpr int kStages = 4;          // default depth of the stage ring (gemm_tn_tile<STAGES>)
constexpr int kThreads = 192;      // 6 warps
constexpr uint32_t kWaitLimit = 1u << 22;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
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
// Bounded wait; returns false (and records the failure) when the limit is reached.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint32_t* err_flag, uint32_t code) {
  for (uint32_t it = 0; it < kWaitLimit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if (it > 128) __nanosleep(64);
  }
  atomicOr(err_flag, code);
  return false;
}

// The same for kernels whose warps run long loops of dependent waits: `abort` is a flag in shared memory that the
// first thread whose wait runs out sets, so that the other roles stop polling at once instead of running out one
// after the other.  Returns false when the limit is reached (recorded in *err_flag) or the flag is seen.
__device__ __forceinline__ bool mbar_wait_abortable(uint32_t bar, uint32_t parity, uint32_t limit, volatile int* abort,
                                                    uint32_t* err_flag, uint32_t code) {
  for (uint32_t it = 0; it < limit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if (it > 128) {
      __nanosleep(64);
      if ((it & 255u) == 0u && *abort) return false;
    }
  }
  atomicOr(err_flag, code);
  *abort = 1;
  return false;
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
      "l"(map), "r"(bar), "r"(x), "r"(y)
      : "memory");
}

// Shared-memory matrix descriptor of a K-major tile stored with the 128-byte swizzle: rows of 128 bytes,
// groups of 8 rows 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3ffffu) >> 4);   // start address
  d |= (uint64_t)1 << 16;                    // leading-dimension byte offset (unused for this layout)
  d |= (uint64_t)(1024 >> 4) << 32;          // stride-dimension byte offset: 8 rows x 128 bytes
  d |= (uint64_t)1 << 46;                    // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                    // 128-byte swizzle
  return d;
}

// Instruction descriptor: D fp32, A and B bf16, both K-major, M = 128, N = nt.
__device__ __forceinline__ uint32_t instr_desc_bf16(int nt) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(nt >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
}

__device__ __forceinline__ void mma_bf16_ss(uint32_t d_tmem, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
      "}\n" ::"r"(d_tmem),
      "l"(da), "l"(db), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_load_32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
        "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
        "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void tmem_load_16(uint32_t taddr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

__host__ __device__ constexpr size_t stage_bytes(int nt) { return (size_t)(kTileM + nt) * kBlockK * 2; }
__host__ __device__ constexpr size_t smem_bytes(int nt, int stages = kStages) { return stages * stage_bytes(nt) + 1024 + 256; }
__host__ __device__ constexpr uint32_t tmem_cols(int nt) { return nt <= 32 ? 32u : nt <= 64 ? 64u : nt <= 128 ? 128u : 256u; }

// Which part of the problem a CTA works on: tile origin in A rows (i0) and B rows (j0), and the K range
// [k0, k0 + 64 nkb) in elements.  With nkb_first < nkb the range is in two pieces: the first nkb_first blocks
// start at k0, the remaining ones at k1 (a row window that wraps around the end of a shard).
// a_rpk / b_rpk > 0: the operand is stored in K blocks, element (row r, column k) at
// ((k / 64) rpk + r) 64 + k mod 64, so that a tile of a K block is one contiguous piece of memory; its tensor map
// then has 64 columns and (K / 64) rpk rows.
struct TileCoord {
  int i0, j0, k0, nkb;
  int k1 = 0, nkb_first = 0x7fffffff;
  int a_rpk = 0, b_rpk = 0;
  __device__ __forceinline__ int k_of(int kb) const {
    return kb < nkb_first ? k0 + kb * kBlockK : k1 + (kb - nkb_first) * kBlockK;
  }
};

// Epi::run(tmem_base, q, lane, set) is executed by the epilogue warps once the accumulator is complete; warp
// quarter q (0..3) may read TMEM lanes 32 q .. 32 q + 31, i.e. accumulator rows 32 q + lane.  The epilogue warps
// are threads 64.. of the block: four of them (EPI_WARPS = 4, set = 0), or eight (EPI_WARPS = 8: two sets of four,
// set = 0 or 1, both sets see all rows and may share the columns between them).  They may synchronise among
// themselves with named barrier 1 over 32 EPI_WARPS threads.
__device__ __forceinline__ void epilogue_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
// Named barrier ID (1..15) over COUNT threads (a multiple of 32); every participating warp names the same count.
template <int ID, int COUNT>
__device__ __forceinline__ void named_sync() {
  asm volatile("bar.sync %0, %1;" ::"n"(ID), "n"(COUNT) : "memory");
}

// Shared memory that follows the stage ring (for an epilogue's own buffers); pass the extra bytes at launch.
__device__ __forceinline__ unsigned char* extra_smem(int nt) {
  extern __shared__ unsigned char umma_smem_raw[];
  const uint32_t base = smem_u32(umma_smem_raw);
  const uint32_t aligned = (base + 1023u) & ~1023u;
  return umma_smem_raw + (aligned - base) + kStages * stage_bytes(nt);
}

// The stage ring itself.  Once the accumulator barrier has completed every tensor-core read of the ring is done and
// no copy is in flight, so an epilogue may use the ring as its scratch: the block then needs no shared memory beyond
// the ring, and two blocks fit on an SM (one computes while the other runs its epilogue).
__device__ __forceinline__ unsigned char* ring_smem() {
  extern __shared__ unsigned char umma_smem_raw[];
  const uint32_t base = smem_u32(umma_smem_raw);
  return umma_smem_raw + (((base + 1023u) & ~1023u) - base);
}

// Adapter: f(row_in_tile, col0, const float (&acc)[32]) is called by the thread that owns accumulator row
// `row_in_tile` (0..127) for the 32-column chunks col0 = 0, 32, ... < NT.  The last chunk may reach past NT:
// entries at columns >= NT are undefined and f must ignore them.
template <class F>
struct ChunkEpilogue {
  F f;
  int nt;
  __device__ __forceinline__ void run(uint32_t tmem_base, int q, int lane, int /*set*/) {
    for (int c0 = 0; c0 < nt; c0 += 32) {
      uint32_t v[32];
      tmem_load_32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, v);
      float acc[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) acc[i] = __uint_as_float(v[i]);
      f(q * 32 + lane, c0, acc);
    }
  }
};

template <int STAGES = kStages, int EPI_WARPS = 4, class Epi>
__device__ __forceinline__ void gemm_tn_tile(const CUtensorMap* tmA, const CUtensorMap* tmB, int nt, TileCoord tc,
                                             uint32_t* err_flag, Epi& epi) {
  extern __shared__ unsigned char umma_smem_raw[];
  __shared__ uint64_t bars[2 * STAGES + 1];
  __shared__ uint32_t tmem_base_sh;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t smem0 = (smem_u32(umma_smem_raw) + 1023u) & ~1023u;   // stages are 1024-byte aligned
  const uint32_t a_bytes = kTileM * kBlockK * 2, st_bytes = (uint32_t)stage_bytes(nt);
  const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[STAGES]), accum = smem_u32(&bars[2 * STAGES]);
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(empty0 + 8 * s, 1);
    }
    mbar_init(accum, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {  // tensor memory for the accumulator (whole warp)
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_sh)),
                 "r"(tmem_cols(nt))
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = tmem_base_sh;

  if (warp == 0) {
    if (lane == 0) {
      for (int kb = 0; kb < tc.nkb; ++kb) {
        const int s = kb % STAGES;
        const uint32_t par = ((uint32_t)(kb / STAGES) & 1u) ^ 1u;
        if (!mbar_wait(empty0 + 8 * s, par, err_flag, 2u)) break;
        mbar_expect_tx(full0 + 8 * s, st_bytes);
        const uint32_t sa = smem0 + s * st_bytes;
        const int k = tc.k_of(kb);
        tma_load_2d(sa, tmA, full0 + 8 * s, tc.a_rpk ? 0 : k, tc.a_rpk ? (k / kBlockK) * tc.a_rpk + tc.i0 : tc.i0);
        tma_load_2d(sa + a_bytes, tmB, full0 + 8 * s, tc.b_rpk ? 0 : k, tc.b_rpk ? (k / kBlockK) * tc.b_rpk + tc.j0 : tc.j0);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = instr_desc_bf16(nt);
      bool ok = true;
      for (int kb = 0; kb < tc.nkb && ok; ++kb) {
        const int s = kb % STAGES;
        ok = mbar_wait(full0 + 8 * s, (uint32_t)(kb / STAGES) & 1u, err_flag, 4u);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t sa = smem0 + s * st_bytes;
        const uint64_t da = smem_desc_sw128(sa), db = smem_desc_sw128(sa + a_bytes);
#pragma unroll
        for (int kk = 0; kk < kBlockK / 16; ++kk)   // 16 elements = 32 bytes = 2 descriptor address units
          mma_bf16_ss(tmem_base, da + 2 * kk, db + 2 * kk, idesc, (kb | kk) != 0 ? 1u : 0u);
        mma_commit(empty0 + 8 * s);                 // the stage is free once these MMAs have read it
      }
      mma_commit(accum);                            // accumulator complete (also reached after a failed wait)
    }
  } else {
    const int q = warp & 3;                         // the TMEM lane quarter this warp may read
    const bool ok = __all_sync(0xffffffffu, mbar_wait(accum, 0u, err_flag, 8u));
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    // all epilogue warps take the same branch (the outcomes are combined), so an epilogue may use
    // its named barriers
    __shared__ int epi_ok[EPI_WARPS];
    if (lane == 0) epi_ok[warp - 2] = (ok && tc.nkb > 0) ? 1 : 0;
    named_sync<1, 32 * EPI_WARPS>();
    int all_ok = 1;
#pragma unroll
    for (int e = 0; e < EPI_WARPS; ++e) all_ok &= epi_ok[e];
    if (all_ok) epi.run(tmem_base, q, lane, (warp - 2) >> 2);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols(nt)) : "memory");
  }
}

// Host: a 2-D tensor map over a row-major bf16 matrix [rows][cols] with the given row pitch (bytes, a multiple of
// 16), boxes of 64 columns x box_rows rows, 128-byte swizzle, zero fill outside the matrix.
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}

inline bool make_map_bf16_2d(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint64_t pitch_bytes,
                             uint32_t box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {pitch_bytes};
  const cuuint32_t box[2] = {(cuuint32_t)kBlockK, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace umma
}  // namespace laq
