// Skinny weight-streaming GEMM on the 5th-generation tensor cores.
//
//   part[z][n][m] = sum_{k in K-range z} W[m, k] * A[n, k]        (bf16 operands, fp32 in TMEM)
//
// The weight matrix sits on the MMA's M axis (tiles of 128 output features), the few token rows
// on its N axis (16..256, padded), so a [128 x 64] weight slab is consumed by four
// tcgen05.mma (K = 16 each) however few rows there are.  Both operands are K-major and are
// brought in by TMA with the 128-byte swizzle into a ring of shared-memory stages; one thread
// issues the MMAs, accumulators live in tensor memory and are read back with tcgen05.ld.
// The work is bandwidth bound: the grid is (M/128 tiles) x (K split) so that all SMs stream
// weights; every CTA stores its partial tile, and the (row-wise) consumer kernel adds the
// partials in split order -- a fixed order, so results do not depend on the number of rows.
#pragma once
#include "fm_common.cuh"
#include "fm_ptx.cuh"

namespace tc {

constexpr int BM = 128;          // output features per CTA
constexpr int BK = 64;           // K elements per slab (128 bytes of bf16)
constexpr int STAGES = 4;

struct Args {
  const CUtensorMap* tmW;        // [Mpad, K] bf16, box 128 x 64
  const CUtensorMap* tmA;        // [rows, K] bf16, box N x 64
  float* part;                   // [split][n_rows_ld][ldm]
  int M, K, N;                   // N = padded rows in the box (multiple of 16, <= 256)
  int n_store;                   // rows actually stored (<= N)
  int ldm;                       // leading dimension of part rows (>= M)
  long long split_stride;        // elements between splits
  int split;                     // K splits = gridDim.y
  int w_row0, a_row0;            // row offsets into the tensor maps (stacked weights / row groups)
  const int* n_active;           // skip when *n_active == 0 (may be null)
  int* status;
};

__device__ inline uint64_t smem_desc_sw128(uint32_t addr) {
  // K-major operand, 128-byte swizzle: start address, leading offset 1 (unused), stride between
  // 8-row groups = 1024 bytes, descriptor version 1, layout type 2
  return (uint64_t)((addr >> 4) & 0x3FFF) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) |
         ((uint64_t)2 << 61);
}
__device__ inline uint32_t instr_desc_bf16(int n) {
  // fp32 accumulate, bf16 x bf16, both K-major, M = 128, N = n
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}
__device__ inline void mma_ss(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ inline void commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(ptx::smem_u32(bar))
               : "memory");
}
__device__ inline void fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ inline void fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ inline void ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

inline int smem_bytes(int N) { return STAGES * (BM * 128 + ((N * 128 + 1023) / 1024) * 1024) + 1024 + 256; }

// grid (M/128 tiles, split); block 128.  Warp 0 lane 0 feeds TMA, warp 1 lane 0 issues MMAs,
// all four warps read the accumulator back (warp w owns TMEM lanes 32w..32w+31).
__global__ void __launch_bounds__(128) gemm_tc_kernel(const Args g) {
  if (g.n_active != nullptr && *g.n_active == 0) return;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int b_bytes = ((g.N * 128 + 1023) / 1024) * 1024;
  const int stage_bytes = BM * 128 + b_bytes;
  uint64_t* full = reinterpret_cast<uint64_t*>(sm + STAGES * stage_bytes);
  uint64_t* empty = full + STAGES;
  uint64_t* accum = empty + STAGES;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(accum + 1);
  __shared__ int s_fail;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile_m = blockIdx.x, z = blockIdx.y;
  const int slabs = g.K / BK;
  const int s0 = (int)((long long)slabs * z / g.split), s1 = (int)((long long)slabs * (z + 1) / g.split);
  const int n_slabs = s1 - s0;
  uint32_t ncols = 32;
  while ((int)ncols < g.N) ncols <<= 1;

  if (threadIdx.x == 0) {
    s_fail = 0;
    for (int i = 0; i < STAGES; ++i) { ptx::mbar_init(full + i, 1); ptx::mbar_init(empty + i, 1); }
    ptx::mbar_init(accum, 1);
    ptx::fence_mbar_init();
    ptx::prefetch_tmap(g.tmW);
    ptx::prefetch_tmap(g.tmA);
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(ptx::smem_u32(tmem_slot)), "r"(ncols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_before();
  __syncthreads();
  fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0 && lane == 0) {
    // ---- producer: stream this CTA's K range through the stage ring
    for (int i = 0; i < n_slabs; ++i) {
      const int st = i % STAGES;
      if (i >= STAGES && !ptx::mbar_wait(empty + st, ((i / STAGES) - 1) & 1)) { s_fail = 1; break; }
      unsigned char* a_dst = sm + st * stage_bytes;
      ptx::mbar_expect_tx(full + st, BM * 128 + g.N * 128);
      ptx::tma_load_2d(a_dst, g.tmW, (s0 + i) * BK, g.w_row0 + tile_m * BM, full + st);
      ptx::tma_load_2d(a_dst + BM * 128, g.tmA, (s0 + i) * BK, g.a_row0, full + st);
    }
  } else if (warp == 1 && lane == 0) {
    // ---- MMA issuer
    const uint32_t idesc = instr_desc_bf16(g.N);
    for (int i = 0; i < n_slabs; ++i) {
      const int st = i % STAGES;
      if (!ptx::mbar_wait(full + st, (i / STAGES) & 1)) { s_fail = 1; break; }
      fence_after();
      const uint32_t a_addr = ptx::smem_u32(sm + st * stage_bytes);
      const uint64_t da = smem_desc_sw128(a_addr), db = smem_desc_sw128(a_addr + BM * 128);
#pragma unroll
      for (int k = 0; k < BK / 16; ++k)                    // +32 bytes along K per step (encoded >> 4)
        mma_ss(tmem, da + 2 * k, db + 2 * k, idesc, (i > 0 || k > 0) ? 1u : 0u);
      commit(empty + st);                                  // stage reusable once these MMAs retire
    }
    commit(accum);                                         // accumulator complete
  }
  __syncwarp();
  // ---- epilogue: everyone waits for the accumulator, then stores the partial tile
  bool ok = n_slabs > 0 ? ptx::mbar_wait(accum, 0) : true;
  __syncwarp();
  fence_after();
  if (!ok || s_fail) {
    if (threadIdx.x == 0) atomicExch(g.status, -5);
  } else {
    const int m = tile_m * BM + warp * 32 + lane;
    float* dst = g.part + (size_t)z * g.split_stride + m;
    for (int n0 = 0; n0 < g.N; n0 += 16) {
      uint32_t r[16];
      if (n_slabs > 0) ld16(tmem + ((uint32_t)(warp * 32) << 16) + n0, r);
      else {
#pragma unroll
        for (int j = 0; j < 16; ++j) r[j] = 0u;
      }
      if (m < g.M) {
#pragma unroll
        for (int j = 0; j < 16; ++j)
          if (n0 + j < g.n_store) dst[(size_t)(n0 + j) * g.ldm] = __uint_as_float(r[j]);
      }
    }
  }
  fence_before();
  __syncthreads();
  fence_after();
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(ncols) : "memory");
  }
}

}  // namespace tc
