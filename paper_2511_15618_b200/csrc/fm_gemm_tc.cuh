// Skinny weight-streaming GEMM on the 5th-generation tensor cores, with the row-wise work that
// follows each projection fused into its tail.
//
//   y[n][m] = sum_k W[m, k] * A[n, k]        (bf16 operands, fp32 accumulation in tensor memory)
//
// The weight matrix sits on the MMA's M axis (tiles of 128 output features), the few token rows
// on its N axis (16..240, padded), so a [128 x 64] weight slab is consumed by four
// tcgen05.mma (K = 16 each) however few rows there are.  Both operands are K-major with the
// 128-byte swizzle.  Weights are stored in HBM slab by slab, each [128 x 64] slab as the 16 KB
// image the MMA reads from shared memory, so a CTA's K range is one contiguous stream fetched by
// 16 KB bulk copies; the token rows come through a TMA tensor map.  A ring of shared-memory stages
// decouples the copies from the one thread that issues the MMAs; accumulators live in tensor
// memory and are read back with tcgen05.ld.
// Operand rows may come as two bfloat16 terms per value, [hi | lo] side by side (hi = bf16(v),
// lo = bf16(v - hi)): the hi tile and the lo tile of a slab then sit one after the other in shared
// memory and form one operand of 2N rows, so each weight slab is still read once; the two
// products land in separate accumulator columns and are added when the accumulator is read.  This
// removes the rounding of the activations from the error budget at no cost in weight traffic.
// The work is bandwidth bound: the grid is (M/128 tiles) x (S splits of K) so that many SMs
// stream weights.  The S CTAs of one M tile form a thread-block cluster: every CTA owns 1/S of the
// tile's columns; each CTA sends the columns of its partial tile to their owners' shared memory
// with asynchronous distributed-shared-memory stores that count their bytes on an mbarrier of the
// owner, so an owner continues as soon as its own S partials are in, adds them in rank order (a
// fixed order, so a row's result does not depend on how many rows the launch holds) and applies
// the epilogue of the projection: RMSNorm scale of the operand rows, then one of
//   EPI_F32 / EPI_BF16   plain store,
//   EPI_GELU             bf16(gelu(y))                      (first FFN matrix),
//   EPI_RESID            x (+)= y; next operand bf16(x * gain); per-tile sums of squares
//                        (output projection, second FFN matrix, shorten),
//   EPI_QKV              rotary embedding, queries out, keys / values appended to the cache,
//   EPI_RESID_CAT        EPI_RESID of the last layer below a shortening: the new hiddens are also
//                        scattered into the concatenated operand rows of the shorten GEMM and into
//                        the level's carry ring, and rows whose parent was computed in an earlier
//                        pass receive that parent's stored upsampled slot at once,
//   EPI_UP               the upsampling projection [3d x d]: slot r of parent row u is added to the
//                        child row 3u + r of the level below (whose residual rows still hold the
//                        pre-shorten hiddens), with next operand and sums of squares for the child
//                        rows; the triple is stored for later passes.
// The kernel is written for programmatic dependent launch: weights do not depend on the
// previous kernel, so their first stages are requested before griddepcontrol.wait.
#pragma once
#include "fm_common.cuh"
#include "fm_ptx.cuh"

namespace tc {

constexpr int BM = 128;          // output features per CTA
constexpr int BK = 64;           // K elements per slab (128 bytes of bf16)
constexpr int MAX_STAGES = 8;
constexpr int MAX_SPLIT = 8;     // portable cluster size
constexpr int MAX_N = 240;       // token rows per launch: two stages + the receive buffer must fit in 227 KB

enum EpiMode { EPI_F32 = 0, EPI_BF16 = 1, EPI_GELU = 2, EPI_RESID = 3, EPI_QKV = 4, EPI_RESID_CAT = 5, EPI_UP = 6 };

struct Args {
  const bf16* W;                 // packed weight slabs: [M tile][K slab][128 x 64 swizzled image]
  const CUtensorMap* tmA;        // operand rows [rows, a_parts * K] bf16 as (K, rows, parts), box 64 x N x a_parts
  int M, K, N;                   // N = token rows per CTA = rows of the operand box (multiple of 16, <= MAX_N)
  int n_store;                   // rows of the launch; N tile z (= blockIdx.z) covers rows [z*N, z*N + N)
  int split;                     // K splits = gridDim.y = cluster size (1, 2, 4 or 8)
  int stages;                    // depth of the shared-memory ring (2..MAX_STAGES)
  int a_parts;                   // 1: plain bf16 operand rows, 2: hi + lo terms
  int w_tile0, a_row0;           // first M tile inside W (stacked matrices), first operand row
  int z_rows, z_w_tiles;         // z_rows > 0: blockIdx.z indexes stacked problems instead of N tiles: problem z
                                 // uses weight tiles from w_tile0 + z*z_w_tiles and rows from z*z_rows (n_store rows each)
  const int* n_active;           // skip when *n_active == 0 (may be null); must not change during a pass
  int* status;
};

struct Epi {
  int row0;                      // first output row of this launch (N tiles beyond the first)
  const float* ssq_in;           // [ssq_n][ld_ssq] partial sums of squares of the operand rows; null = no scale
  int ssq_n, ld_ssq;
  float inv_d_in, eps;
  void* out; int ldo;            // EPI_F32 / EPI_BF16 / EPI_GELU
  int lo_off;                    // bf16 outputs (out of EPI_BF16 / EPI_GELU, a_out of EPI_RESID): when > 0 the
                                 // lo term of every value is stored lo_off elements behind its hi term
  float* x; int ldx; int add;    // EPI_RESID: residual stream, add = 0 replaces it
  const float* gain;             //            gain of the next norm (null = 1)
  bf16* a_out; int lda;          //            next GEMM's operand rows (may be null)
  float* ssq_out; int ld_ssq_out;//            [M tiles * split][ld] partial sums of squares of the new x rows (may be null)
  Dims dm; SeqState st;          // EPI_QKV
  int batch, level;
  const float2* rope_tab;
  bf16* q_out;                   //            [rows, H*dh], rotated and scaled by qscale
  bf16* Kc; bf16* Vc;            //            caches [B, Hkv, slots, dh]
  float qscale;
  const float* stash_x;          //            when stash_ring is set: residual rows [rows, stash_d] that the CTAs
  float* stash_ring;             //            of K split 0 copy, column block by column block, into the carry ring
  int stash_d, stash_rs;         //            [B, stash_rs, stash_d] at entry pos mod stash_rs (split-node hiddens)
  // EPI_RESID_CAT (dm, st, batch, level = this level): shorten / carry side outputs
  bf16* cat_out;                 //            operand rows of the shorten GEMM [rows above, 6d] as [hi | lo], part k at k*d
  float* cat_ring;               //            carry ring of this level's hiddens [B, fm_ring(level), d]
  const float* cat_tri;          //            stored upsampled triples of the level above [B, fm_ring(level+1), 3d]
  // EPI_UP (dm, st, batch, level = the parent level; x / gain / a_out / ssq_out describe the child rows)
  float* tri_ring;               //            where the triples of this pass go [B, fm_ring(level), 3d]
  int d_model;
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

// ---- thread-block cluster: rank, barrier, stores into a peer CTA's shared memory
__device__ inline uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ inline void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// 16-byte store into a peer CTA's shared memory that reports its bytes to an mbarrier of that CTA
__device__ inline void st_async_peer4(uint32_t remote_addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d, uint32_t remote_bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];" ::"r"(remote_addr),
               "r"(a), "r"(b), "r"(c), "r"(d), "r"(remote_bar)
               : "memory");
}
__device__ inline bool mbar_try_wait_cluster(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(ptx::smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ inline bool mbar_wait_cluster(uint64_t* bar, uint32_t parity, long long limit_cycles = 200000000ll) {
  if (mbar_try_wait_cluster(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait_cluster(bar, parity))
    if (clock64() - t0 > limit_cycles) return false;
  return true;
}
__device__ inline uint32_t map_peer(uint32_t local_addr, uint32_t rank) {
  uint32_t ra;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(local_addr), "r"(rank));
  return ra;
}

// Shared memory: ring of `stages` x ([128 x 64] weight slab + [N x 64] operand slab), then the
// receive buffer of the cluster reduction [split][64/split][2][N + 4] fp32 = (N + 4) * 512 bytes
// (peers write into it while this CTA may still be multiplying, so it never aliases the ring;
// the 4 floats of padding spread the readers over the banks), then the side rows [N][512 bytes]
// (what the epilogue reads per row besides the product: the residual rows of the tile's 128
// columns, or the rows' rotary angles; brought in by bulk copies while the MMAs run), then barriers.
inline int stage_bytes(int N, int parts) { return BM * 128 + parts * (((N * 128 + 1023) / 1024) * 1024); }
// The side rows exist only when a thread may get more than two items of the epilogue (N rows x
// 64/split pair slots over 128 threads); otherwise the shared memory is better left to a
// neighbouring kernel's CTA.
__host__ __device__ inline int side_bytes(int N, int split) { return N * (64 / split) > 256 ? N * 512 : 0; }
// as many stages as the CTA has slabs (its whole K range is then requested at once), at most 8
// and what fits beside the receive buffer
inline int pick_stages(int N, int n_slabs, int parts, int side_b) {
  int st = (200 * 1024 - (N + 4) * 512 - side_b) / stage_bytes(N, parts);
  st = st > MAX_STAGES ? MAX_STAGES : st;
  st = st > n_slabs ? n_slabs : st;
  return st < 2 ? 2 : st;
}
inline int smem_bytes(int N, int stages, int parts, int side_b) {
  return stages * stage_bytes(N, parts) + (N + 4) * 512 + side_b + 1024 + 256;
}

inline int max_smem_bytes() {
  const int sb = side_bytes(32, 1);
  const int a = smem_bytes(32, pick_stages(32, MAX_STAGES, 1, sb), 1, sb), b = smem_bytes(32, pick_stages(32, MAX_STAGES, 2, sb), 2, sb);
  return a > b ? a : b;
}

// (The differences below use __fsub_rn so that the compiler cannot fold a product that the caller
// passes in into a fused multiply-subtract: a value must split the same way at every call site.)
__device__ inline void store_hi_lo(bf16* p, float v, int lo_off) {
  const bf16 hi = __float2bfloat16(v);
  p[0] = hi;
  if (lo_off > 0) p[lo_off] = __float2bfloat16(__fsub_rn(v, __bfloat162float(hi)));
}

// two neighbouring values as [hi, hi] and [lo, lo] pairs: one 4-byte store each
__device__ inline void store_hi_lo2(bf16* p, float a, float b, int lo_off) {
  const __nv_bfloat162 hi = __floats2bfloat162_rn(a, b);
  *reinterpret_cast<__nv_bfloat162*>(p) = hi;
  if (lo_off > 0)
    *reinterpret_cast<__nv_bfloat162*>(p + lo_off) = __floats2bfloat162_rn(__fsub_rn(a, __bfloat162float(hi.x)), __fsub_rn(b, __bfloat162float(hi.y)));
}

__device__ inline float gelu_erf_f(float x) { return 0.5f * x * (1.f + erff(x * 0.70710678118654752f)); }

// Pair slot q (0..63) of a 128-column tile -> its two columns.  Rotary pairs are (i, i + dh/2)
// inside a head, so with heads of 64 a tile holds two heads with 32 pairs each, with heads of
// 128 one head with 64 pairs.  The other epilogues use the same map (any bijection would do).
// Epilogues without rotation pair neighbouring columns (2q, 2q + 1), so that a thread's two values
// leave in one store.
template <bool ROT>
__device__ inline void pair_cols(int q, bool head128, int& ca, int& cb) {
  if (!ROT) { ca = 2 * q; cb = ca + 1; }
  else if (head128) { ca = q; cb = q + 64; }
  else { ca = (q >> 5) * 64 + (q & 31); cb = ca + 32; }
}

// grid (M/128 tiles, split, N tiles of the token rows), cluster (1, split, 1); block 128.  Warp 0 lane 0 feeds TMA, warp 1
// lane 0 issues MMAs, all four warps read the accumulator back (warp w owns TMEM lanes 32w..32w+31).
// SIDE: the launch has side rows (side_bytes(N, split) > 0); a separate instantiation, because the
// mere presence of that path costs the few-row launches 0.4 us each (measured).
template <int MODE, bool SIDE>
__global__ void __launch_bounds__(128) gemm_tc_kernel(const Args g, const Epi e) {
  constexpr int ROWS_AUX = (MODE == EPI_RESID_CAT || MODE == EPI_UP) ? 256 : 1;
  constexpr int CARRY_MAX = MODE == EPI_UP ? 128 : 1;
  if (g.n_active != nullptr && *g.n_active == 0) {   // the whole grid leaves; keep the launch chain ordered
    ptx::grid_dep_launch();
    ptx::grid_dep_wait();
    return;
  }
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int STAGES = g.stages;
  const int b_bytes = ((g.N * 128 + 1023) / 1024) * 1024;
  const int stage_bytes = BM * 128 + g.a_parts * b_bytes;
  const int NP = g.N + 4;
  float* recv = reinterpret_cast<float*>(sm + STAGES * stage_bytes);          // [S][PW][2][NP]
  float* side = recv + NP * 128;                                              // [N][128] fp32 (or [N][64] float2)
  uint64_t* full = reinterpret_cast<uint64_t*>(sm + STAGES * stage_bytes + NP * 512 + (SIDE ? g.N * 512 : 0));
  uint64_t* empty = full + MAX_STAGES;
  uint64_t* accum = empty + MAX_STAGES;
  uint64_t* rbar = accum + 1;                                                 // partials of all ranks have arrived
  uint64_t* sbar = rbar + 1;                                                  // side rows have arrived
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sbar + 1);
  __shared__ int s_fail;
  __shared__ float s_inv[256];
  __shared__ int s_rb[256], s_rp[256];
  __shared__ int s_ra[ROWS_AUX], s_rl[ROWS_AUX];             // EPI_RESID_CAT / EPI_UP: see the row maps below
  __shared__ int s_carry[CARRY_MAX], s_ncarry;               // EPI_UP: child rows whose parent is not in this pass

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tile_m = blockIdx.x;
  // token rows of this CTA: N tile blockIdx.z of the launch's rows
  const int row_lo = (int)blockIdx.z * (g.z_rows > 0 ? g.z_rows : g.N);
  const int ns = g.z_rows > 0 ? min(g.N, g.n_store) : min(g.N, g.n_store - row_lo);   // rows of this tile that exist
  const int w_tile = g.w_tile0 + (int)blockIdx.z * g.z_w_tiles;
  const int row0 = e.row0 + row_lo;                        // first output row
  const int a_row = g.a_row0 + row_lo;                     // first operand row
  const int S = g.split;
  const int z = (int)cluster_rank();                 // == blockIdx.y: the cluster spans the grid's y extent
  const int slabs = g.K / BK;
  const int s0 = (int)((long long)slabs * z / S), s1 = (int)((long long)slabs * (z + 1) / S);
  const int n_slabs = s1 - s0;
  uint32_t ncols = 32;
  while ((int)ncols < g.a_parts * g.N) ncols <<= 1;

  if (tid == 0) {
    s_fail = 0;
    for (int i = 0; i < STAGES; ++i) { ptx::mbar_init(full + i, 1); ptx::mbar_init(empty + i, 1); }
    ptx::mbar_init(accum, 1);
    ptx::mbar_init(rbar, 1);
    ptx::mbar_init(sbar, 1);
    ptx::fence_mbar_init();
    // rows are sent in groups of 16: groups x 16 rows x 128/S columns x S ranks x 4 bytes
    ptx::mbar_expect_tx(rbar, (uint32_t)((ns + 15) / 16) * 16u * 512u);
    ptx::prefetch_tmap(g.tmA);
    // The weight slabs of the first stages do not depend on the previous kernel: request them at
    // once, so that they travel while the rest of the prologue runs.
    const bf16* wsrc = g.W + ((size_t)(w_tile + tile_m) * slabs + s0) * (BM * BK);
    const int pre = n_slabs < STAGES ? n_slabs : STAGES;
    for (int i = 0; i < pre; ++i) {
      ptx::mbar_expect_tx(full + i, BM * 128 + g.a_parts * g.N * 128);
      ptx::bulk_load(sm + i * stage_bytes, wsrc + (size_t)i * (BM * BK), BM * 128, full + i);
    }
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
  // This CTA now holds its tensor memory and shared memory: the next kernel may start its own
  // prologue beside us.
  ptx::grid_dep_launch();
  // Peers will write into this CTA's receive buffer and count on its barrier: make sure every
  // CTA of the cluster runs and has initialised them.
  if (S > 1) cluster_sync();

  // side rows: residual rows of this tile's columns (EPI_RESID that adds), or the rows' rotary
  // angles (EPI_QKV tiles that hold query or key heads)
  // Only when a thread has more than two items: with fewer, loads straight into registers right
  // after the dependency wait are quicker than the round through the copy engine (measured).
  constexpr bool IS_RESID = MODE == EPI_RESID || MODE == EPI_RESID_CAT;
  constexpr bool ROW_MAPS = MODE == EPI_QKV || MODE == EPI_RESID_CAT || MODE == EPI_UP;
  const bool want_side = (IS_RESID && e.add != 0) ||
                         (MODE == EPI_QKV && e.dm.theta != 0.f && (tile_m * BM) / e.dm.dh < e.dm.H + e.dm.Hkv);
  const bool use_side = SIDE && want_side;
  if (warp == 0) {
    // ---- operand rows of the first stages (their weight slabs are already on their way): one
    // copy per slab brings the hi and the lo tile; lanes issue them side by side
    const int pre = n_slabs < STAGES ? n_slabs : STAGES;
    ptx::grid_dep_wait();
    if (lane < pre) ptx::tma_load_3d(sm + lane * stage_bytes + BM * 128, g.tmA, (s0 + lane) * BK, a_row, 0, full + lane);
  }
  if (warp == 0 && lane == 0) {
    // ---- producer: stream the rest of this CTA's K range through the stage ring
    const bf16* wsrc = g.W + ((size_t)(w_tile + tile_m) * slabs + s0) * (BM * BK);
    const int pre = n_slabs < STAGES ? n_slabs : STAGES;
    for (int i = pre; i < n_slabs; ++i) {
      const int st = i % STAGES;
      if (!ptx::mbar_wait(empty + st, ((i / STAGES) - 1) & 1)) { s_fail = 1; break; }
      unsigned char* a_dst = sm + st * stage_bytes;
      ptx::mbar_expect_tx(full + st, BM * 128 + g.a_parts * g.N * 128);
      ptx::bulk_load(a_dst, wsrc + (size_t)i * (BM * BK), BM * 128, full + st);
      ptx::tma_load_3d(a_dst + BM * 128, g.tmA, (s0 + i) * BK, a_row, 0, full + st);
    }
  } else if (warp == 1 && lane == 0) {
    // ---- MMA issuer
    const uint32_t idesc = instr_desc_bf16(g.a_parts * g.N);   // hi and lo tiles: one operand of 2N rows
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
  else if (warp >= 2) {
    // ---- warps 2 and 3, while the operands arrive: operand-row scales (the partial sums of
    // squares of a row are gathered by 8 lanes, each adding its slots in slot order, then combined by
    // a fixed shuffle tree) and row maps
    if (ROW_MAPS && warp == 3) {
      // row maps, and the rows' rotary angles into the side buffer: positions are per-pass state
      // and the table is constant, so nothing here waits for the previous kernel
      const uint32_t row_bytes = (uint32_t)e.dm.dh * 4u;   // dh/2 (cos, sin) pairs
      uint32_t total = 0;
      for (int n0 = 0; n0 < ns; n0 += 32) {
        const int n = n0 + lane;
        int b = 0, p = 0;
        const bool valid = n < ns && fm_row_map(e.dm, e.st, e.batch, e.level, row0 + n, b, p);
        if (n < ns) { s_rb[n] = valid ? b : -1; s_rp[n] = p; }
        if ((MODE == EPI_RESID_CAT || MODE == EPI_UP) && n < ns && valid) {
          // first position of the sequence at the other level of the pair, last position at the lower one
          const int Lb = e.st.L[b], nr = e.st.nrow[b];
          const int rl = fm_ratio(MODE == EPI_UP ? e.level - 1 : e.level), ru = 3 * rl;
          s_ra[n] = MODE == EPI_UP ? (Lb + rl - 1) / rl : (Lb + ru - 1) / ru;
          s_rl[n] = (Lb + nr - 1) / rl;
        }
        total += (uint32_t)__popc(__ballot_sync(0xffffffffu, valid)) * row_bytes;
      }
      if (MODE == EPI_QKV && use_side) {
        if (lane == 0) ptx::mbar_expect_tx(sbar, total);
        __syncwarp();
        for (int n = lane; n < ns; n += 32)
          if (s_rb[n] >= 0) ptx::bulk_load(side + n * 128, e.rope_tab + (size_t)s_rp[n] * (e.dm.dh >> 1), row_bytes, sbar);
      }
    }
    if (MODE == EPI_UP && warp == 2 && lane == 0) {
      const int lvl = e.level - 1, rl = fm_ratio(lvl), m_low = fm_rows_per_seq(e.dm, lvl);
      const int slot = (tile_m * BM) / e.d_model;
      int cnt = 0;
      for (int b = 0; b < e.batch; ++b) {
        const int nr = e.st.nrow[b], Lb = e.st.L[b];
        if (nr <= 0) continue;
        const int p0l = (Lb + rl - 1) / rl, plast = (Lb + nr - 1) / rl, p0u = (Lb + 3 * rl - 1) / (3 * rl);
        for (int p = p0l; p < 3 * p0u && p <= plast; ++p)
          if (p % 3 == slot && cnt < CARRY_MAX) s_carry[cnt++] = b * m_low + (p - p0l);
      }
      s_ncarry = cnt;
    }
    ptx::grid_dep_wait();
    if (IS_RESID && use_side && warp == 2) {               // residual rows of this tile's columns
      const int cols = min(BM, g.M - tile_m * BM);
      if (lane == 0) ptx::mbar_expect_tx(sbar, (uint32_t)(ns * cols) * 4u);
      __syncwarp();
      for (int n = lane; n < ns; n += 32)
        ptx::bulk_load(side + n * 128, e.x + (size_t)(row0 + n) * e.ldx + tile_m * BM, (uint32_t)cols * 4u, sbar);
    }
    const int t = tid - 64;
    if (e.ssq_in != nullptr) {
      const int sub = t & 7;
      for (int n0 = 0; n0 < ns; n0 += 8) {
        const int n = n0 + (t >> 3);
        float v[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const int slot = sub + 8 * k;
          v[k] = (n < ns && slot < e.ssq_n) ? __ldcg(e.ssq_in + (size_t)slot * e.ld_ssq + row0 + n) : 0.f;
        }
        float ss = 0.f;
#pragma unroll
        for (int k = 0; k < 8; ++k) ss += v[k];
        for (int slot = sub + 64; slot < e.ssq_n; slot += 8)             // more than 64 slots: not expected
          ss += (n < ns) ? __ldcg(e.ssq_in + (size_t)slot * e.ld_ssq + row0 + n) : 0.f;
        ss += __shfl_xor_sync(0xffffffffu, ss, 1);
        ss += __shfl_xor_sync(0xffffffffu, ss, 2);
        ss += __shfl_xor_sync(0xffffffffu, ss, 4);
        if (sub == 0 && n < ns) s_inv[n] = rsqrtf(ss * e.inv_d_in + e.eps);
      }
    } else {
      for (int n = t; n < ns; n += 64) s_inv[n] = 1.f;
    }
  }
  __syncwarp();

  // ---- where this thread's accumulator column goes, and its first item of the epilogue.  Column
  // m of the tile is half h of pair slot q; slots [r*PW, (r+1)*PW) belong to rank r, which receives
  // [source rank][slot][half][row].  Everything that does not depend on the previous kernel
  // (indices, gains, rotary angles) is prepared here, before the wait.
  const int lgS = 31 - __clz(S);                           // S is 1, 2, 4 or 8
  const int lgPW = 6 - lgS, PW = 1 << lgPW;
  const bool head128 = MODE == EPI_QKV && e.dm.dh == 128;
  const int items = ns * PW;
  uint32_t dst0 = 0, dbar = 0;
  float* recv_own;                                         // S == 1: this thread's row run in the local buffer
  {
    const int q = MODE != EPI_QKV ? (tid >> 1) : (head128 ? (tid & 63) : ((tid >> 6) * 32 + (tid & 31)));
    const int h = MODE != EPI_QKV ? (tid & 1) : (head128 ? (tid >> 6) : ((tid >> 5) & 1));
    const int owner = q >> lgPW, cc = q & (PW - 1);
    recv_own = recv + (((size_t)z * PW + cc) * 2 + h) * NP;
    if (S > 1) {
      dst0 = map_peer(ptx::smem_u32(recv_own), (uint32_t)owner);
      dbar = map_peer(ptx::smem_u32(rbar), (uint32_t)owner);
    }
  }
  // A thread keeps its pair slot in every item (items advance by 128, a multiple of PW): its two
  // columns, and with them the gains, are fixed.
  float pre_ga = 1.f, pre_gb = 1.f;
  float2 pre_cs = make_float2(1.f, 0.f);                   // first item's rotary angle when the side rows are not used
  if (tid < items) {
    int ca, cb;
    pair_cols<MODE == EPI_QKV>(z * PW + (tid & (PW - 1)), head128, ca, cb);
    const int ma = tile_m * BM + ca, mb = tile_m * BM + cb;
    if (IS_RESID && e.gain != nullptr) {
      if (ma < g.M) pre_ga = e.gain[ma];
      if (mb < g.M) pre_gb = e.gain[mb];
    }
    if (MODE == EPI_UP && e.gain != nullptr) {             // gains of the child rows' next norm: column m mod d
      if (ma < g.M) pre_ga = e.gain[ma % e.d_model];
      if (mb < g.M) pre_gb = e.gain[mb % e.d_model];
    }
    if (MODE == EPI_QKV && want_side && !use_side) {
      int b, p;
      const bool valid = fm_row_map(e.dm, e.st, e.batch, e.level, row0 + (tid >> lgPW), b, p);
      const int head = ma / e.dm.dh, i = ma - head * e.dm.dh;
      if (valid && ma < g.M && head < e.dm.H + e.dm.Hkv) pre_cs = e.rope_tab[(size_t)p * (e.dm.dh >> 1) + i];
    }
  }
  // Kernel parameters the tail needs, read into registers now: a first touch of the parameter
  // bank after the wait would sit on the critical path.
  int k_row0 = row0, k_ldo = e.ldo, k_ldx = e.ldx, k_lda = e.lda, k_ldssq = e.ld_ssq_out;
  int k_M = g.M, k_ns = ns, k_lo = e.lo_off;
  void* k_out = e.out;
  float* k_x = e.x;
  bf16* k_aout = e.a_out;
  float* k_ssqo = e.ssq_out;
  bf16 *k_q = e.q_out, *k_K = e.Kc, *k_V = e.Vc;
  float k_qs = e.qscale;
  int k_H = e.dm.H, k_Hkv = e.dm.Hkv, k_dh = e.dm.dh, k_P = e.dm.P, k_cap = MODE == EPI_QKV ? e.dm.cap[e.level] : 1;
  int* k_status = g.status;

  asm volatile("" : "+r"(k_row0), "+r"(k_ldo), "+r"(k_ldx), "+r"(k_lda), "+r"(k_ldssq), "+r"(k_M), "+r"(k_ns), "+r"(k_lo));
  asm volatile("" : "+l"(k_out), "+l"(k_x), "+l"(k_aout), "+l"(k_ssqo), "+l"(k_q), "+l"(k_K), "+l"(k_V), "+l"(k_status));
  asm volatile("" : "+f"(k_qs), "+r"(k_H), "+r"(k_Hkv), "+r"(k_dh), "+r"(k_P), "+r"(k_cap));
  ptx::grid_dep_wait();                                    // everything below touches activations
  float pre_xa = 0.f, pre_xb = 0.f;                        // first item's residual values, same case
  if (IS_RESID && want_side && !use_side && tid < items) {
    int ca, cb;
    pair_cols<MODE == EPI_QKV>(z * PW + (tid & (PW - 1)), head128, ca, cb);
    const int ma = tile_m * BM + ca, mb = tile_m * BM + cb;
    const float* xr = k_x + (size_t)(k_row0 + (tid >> lgPW)) * k_ldx;
    if (ma < k_M) pre_xa = xr[ma];
    if (mb < k_M) pre_xb = xr[mb];
  }

  __syncthreads();                                         // s_inv / row maps are written (long before the MMAs end)
  if (MODE == EPI_QKV && e.stash_ring != nullptr && z == 0) {
    // the rows' residual values, as they enter this layer, go into the carry ring (the draft heads
    // read them after the pass); this CTA copies column tile_m*128 + tid
    const int col = tile_m * BM + tid;
    if (col < e.stash_d)
      for (int n = 0; n < ns; ++n)
        if (s_rb[n] >= 0)
          e.stash_ring[((size_t)s_rb[n] * e.stash_rs + s_rp[n] % e.stash_rs) * e.stash_d + col] = e.stash_x[(size_t)(row0 + n) * e.stash_d + col];
  }
  // ---- every warp waits for the accumulator and sends its 32 columns of the partial tile to
  // their owners.  A timeout is recorded; zeros are sent so that no owner waits in vain.
  bool ok = n_slabs > 0 ? ptx::mbar_wait(accum, 0) : true;
  ok = __all_sync(0xffffffffu, ok);
  fence_after();
  for (int n0 = 0; n0 < k_ns; n0 += 16) {
    uint32_t r[16];
    if (ok && n_slabs > 0) {
      ld16(tmem + ((uint32_t)(warp * 32) << 16) + n0, r);
      if (g.a_parts == 2) {                                // the lo products: columns N..2N-1
        uint32_t r2[16];
        ld16(tmem + ((uint32_t)(warp * 32) << 16) + g.N + n0, r2);
#pragma unroll
        for (int j = 0; j < 16; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) + __uint_as_float(r2[j]));
      }
    } else {
#pragma unroll
      for (int j = 0; j < 16; ++j) r[j] = 0u;
    }
    if (S > 1) {
#pragma unroll
      for (int j = 0; j < 16; j += 4) st_async_peer4(dst0 + (uint32_t)(n0 + j) * 4u, r[j], r[j + 1], r[j + 2], r[j + 3], dbar);
    } else {                                               // no split: the tile stays in this CTA
#pragma unroll
      for (int j = 0; j < 16; j += 4)
        *reinterpret_cast<uint4*>(recv_own + n0 + j) = make_uint4(r[j], r[j + 1], r[j + 2], r[j + 3]);
    }
  }
  bool arrived = true;
  if (S > 1) arrived = mbar_wait_cluster(rbar, 0);
  else __syncthreads();
  if (use_side) arrived = ptx::mbar_wait(sbar, 0) && arrived;
  if (!ok || !arrived || s_fail) {
    if (tid == 0) atomicExch(k_status, -5);
  }
  // ---- this rank's share of the tile: pair slots [z*PW, (z+1)*PW), all rows
  const int lgL = lgPW < 5 ? lgPW : 5, L = 1 << lgL;        // lanes that share a row
  for (int it0 = 0; it0 < items; it0 += 128) {
    const int it = it0 + tid;
    const bool active = it < items, first = it0 == 0;
    const int n = active ? it >> lgPW : 0, cc = active ? it & (PW - 1) : 0;
    int ca, cb;
    pair_cols<MODE == EPI_QKV>(z * PW + cc, head128, ca, cb);
    float va[MAX_SPLIT], vb[MAX_SPLIT];
#pragma unroll
    for (int r = 0; r < MAX_SPLIT; ++r) {                  // all loads first, then the sums in rank order
      const float* src = recv + ((r << lgPW) + cc) * 2 * NP + n;
      va[r] = (r < S && active) ? src[0] : 0.f;
      vb[r] = (r < S && active) ? src[NP] : 0.f;
    }
    float ya = 0.f, yb = 0.f;
#pragma unroll
    for (int r = 0; r < MAX_SPLIT; ++r)
      if (r < S) { ya += va[r]; yb += vb[r]; }
    const float inv = s_inv[n];
    ya *= inv;
    yb *= inv;
    const int ma = tile_m * BM + ca, mb = tile_m * BM + cb;
    const bool a_ok = active && ma < k_M, b_ok = active && mb < k_M;
    const size_t row = (size_t)(k_row0 + n);
    if (MODE == EPI_F32) {
      float* o = reinterpret_cast<float*>(k_out) + row * k_ldo;
      if (b_ok && (k_ldo & 1) == 0) *reinterpret_cast<float2*>(o + ma) = make_float2(ya, yb);
      else {
        if (a_ok) o[ma] = ya;
        if (b_ok) o[mb] = yb;
      }
    } else if (MODE == EPI_BF16) {
      bf16* o = reinterpret_cast<bf16*>(k_out) + row * k_ldo;
      if (b_ok) store_hi_lo2(o + ma, ya, yb, k_lo);
      else if (a_ok) store_hi_lo(o + ma, ya, k_lo);
    } else if (MODE == EPI_GELU) {
      bf16* o = reinterpret_cast<bf16*>(k_out) + row * k_ldo;
      if (b_ok) store_hi_lo2(o + ma, gelu_erf_f(ya), gelu_erf_f(yb), k_lo);
      else if (a_ok) store_hi_lo(o + ma, gelu_erf_f(ya), k_lo);
    } else if (IS_RESID) {
      float* xr = k_x + row * k_ldx;
      float xa = 0.f, xb = 0.f;
      if (b_ok) {                                          // both columns (M is even wherever the residual is used)
        float2 x0 = make_float2(0.f, 0.f);
        if (use_side) x0 = *reinterpret_cast<const float2*>(side + n * 128 + ca);
        else if (first) x0 = make_float2(pre_xa, pre_xb);
        else if (want_side) x0 = *reinterpret_cast<const float2*>(xr + ma);
        xa = x0.x + ya;
        xb = x0.y + yb;
        if (MODE == EPI_RESID_CAT && s_rb[n] >= 0) {
          // (xa, xb) is the level's final hidden of position p: into the carry ring, into the operand
          // row of the parent that pools it (if that parent is a row of this pass), and, where the
          // position's own parent p / 3 was computed in an earlier pass, that parent's stored slot
          // is added at once (the up-stack then finds h + upsampled slot in the residual row)
          const int b = s_rb[n], p = s_rp[n], dd = e.d_model, rs = fm_ring(e.level), rsu = fm_ring(e.level + 1);
          *reinterpret_cast<float2*>(e.cat_ring + ((size_t)b * rs + p % rs) * dd + ma) = make_float2(xa, xb);
          const int u = (p + 2) / 3, part = p - 3 * u + 2;
          if (3 * u <= s_rl[n])
            store_hi_lo2(e.cat_out + ((size_t)(b * fm_rows_per_seq(e.dm, e.level + 1) + u - s_ra[n]) * 6 + part) * dd + ma, xa, xb, 3 * dd);
          if (p < 3 * s_ra[n]) {
            const float2 t = __ldcg(reinterpret_cast<const float2*>(e.cat_tri + (((size_t)b * rsu + (p / 3) % rsu) * 3 + p % 3) * dd + ma));
            xa += t.x;
            xb += t.y;
          }
        }
        *reinterpret_cast<float2*>(xr + ma) = make_float2(xa, xb);
        if (k_aout != nullptr) store_hi_lo2(k_aout + row * k_lda + ma, __fmul_rn(xa, pre_ga), __fmul_rn(xb, pre_gb), k_lo);
      } else if (a_ok) {
        xa = (use_side ? side[n * 128 + ca] : (first ? pre_xa : (want_side ? xr[ma] : 0.f))) + ya;
        xr[ma] = xa;
        if (k_aout != nullptr) store_hi_lo(k_aout + row * k_lda + ma, __fmul_rn(xa, pre_ga), k_lo);
      }
      if (k_ssqo != nullptr) {
        // per-row sums of squares of this rank's columns: a fixed shuffle tree over the L lanes that
        // share the row; the next GEMM adds the (tile, rank, lane group) partials in slot order
        float sqv = __fmaf_rn(xa, xa, __fmul_rn(xb, xb));
        for (int o = L >> 1; o > 0; o >>= 1) sqv += __shfl_xor_sync(0xffffffffu, sqv, o);
        if (active && (cc & (L - 1)) == 0)
          k_ssqo[(size_t)((((tile_m << lgS) + z) << (lgPW - lgL)) + (cc >> lgL)) * k_ldssq + k_row0 + n] = sqv;
      }
    } else if (MODE == EPI_UP) {
      // (ya, yb): columns (ma, ma + 1) of the triple of parent row n = slot ma / d, column ma % d
      const int dd = e.d_model;
      float xa = 0.f, xb = 0.f;
      bool child = false;
      size_t crow = 0;
      if (b_ok && s_rb[n] >= 0) {
        const int b = s_rb[n], pu = s_rp[n], rsu = fm_ring(e.level);
        *reinterpret_cast<float2*>(e.tri_ring + ((size_t)b * rsu + pu % rsu) * 3 * dd + ma) = make_float2(ya, yb);
        const int slot = ma / dd, col = ma - slot * dd, p = 3 * pu + slot;
        if (p <= s_rl[n]) {                                // the child is a row of this pass
          child = true;
          crow = (size_t)b * fm_rows_per_seq(e.dm, e.level - 1) + (p - s_ra[n]);
          float* xr = k_x + crow * k_ldx + col;
          const float2 x0 = __ldcg(reinterpret_cast<const float2*>(xr));
          xa = x0.x + ya;
          xb = x0.y + yb;
          *reinterpret_cast<float2*>(xr) = make_float2(xa, xb);
          if (k_aout != nullptr) store_hi_lo2(k_aout + crow * k_lda + col, __fmul_rn(xa, pre_ga), __fmul_rn(xb, pre_gb), k_lo);
        }
      }
      if (k_ssqo != nullptr) {                             // as EPI_RESID, for the child row; tiles count within d
        float sqv = __fmaf_rn(xa, xa, __fmul_rn(xb, xb));
        for (int o = L >> 1; o > 0; o >>= 1) sqv += __shfl_xor_sync(0xffffffffu, sqv, o);
        if (active && child && (cc & (L - 1)) == 0)
          k_ssqo[(size_t)(((((tile_m % (dd / BM)) << lgS) + z) << (lgPW - lgL)) + (cc >> lgL)) * k_ldssq + crow] = sqv;
      }
    } else {  // EPI_QKV: (ya, yb) is the rotary pair (i, i + dh/2) of one head
      const int dh = k_dh, half = dh >> 1, H = k_H, Hkv = k_Hkv;
      const int head = ma / dh, i = ma - head * dh;
      if (a_ok && head < H + 2 * Hkv) {
        const int b = s_rb[n], p = s_rp[n];
        const bool valid = b >= 0;
        const int slots = k_P + k_cap;
        if (head < H + Hkv) {
          float2 cs = make_float2(1.f, 0.f);
          if (use_side) { if (valid) cs = reinterpret_cast<const float2*>(side)[n * 64 + i]; }
          else if (first) cs = pre_cs;
          else if (want_side && valid) cs = e.rope_tab[(size_t)p * half + i];
          const float y1 = ya * cs.x - yb * cs.y, y2 = yb * cs.x + ya * cs.y;
          if (head < H) {
            bf16* q = k_q + (row * H + head) * dh;
            q[i] = __float2bfloat16(valid ? y1 * k_qs : 0.f);
            q[half + i] = __float2bfloat16(valid ? y2 * k_qs : 0.f);
          } else if (valid) {
            bf16* dst = k_K + (((size_t)b * Hkv + (head - H)) * slots + k_P + (p % k_cap)) * dh;
            dst[i] = __float2bfloat16(y1);
            dst[half + i] = __float2bfloat16(y2);
          }
        } else if (valid) {
          bf16* dst = k_V + (((size_t)b * Hkv + (head - H - Hkv)) * slots + k_P + (p % k_cap)) * dh;
          dst[i] = __float2bfloat16(ya);
          dst[half + i] = __float2bfloat16(yb);
        }
      }
    }
  }
  if (MODE == EPI_UP) {
    // child rows of this tile's slot whose parent was computed in an earlier pass: their residual
    // rows are final already (the last layer below added the stored slot); what is missing is the
    // next operand and the sums of squares, for this rank's columns
    const int dd = e.d_model, nci = s_ncarry << lgPW;
    for (int it0 = 0; it0 < nci; it0 += 128) {
      const int it = it0 + tid;
      const bool active = it < nci;
      const int cc = it & (PW - 1);
      const size_t crow = active ? (size_t)s_carry[it >> lgPW] : 0;
      int ca, cb;
      pair_cols<false>(z * PW + cc, false, ca, cb);
      const int col = (tile_m * BM + ca) % dd;
      float2 x0 = make_float2(0.f, 0.f);
      if (active) x0 = __ldcg(reinterpret_cast<const float2*>(k_x + crow * k_ldx + col));
      if (active && k_aout != nullptr) {
        const float ga = e.gain != nullptr ? e.gain[col] : 1.f, gb = e.gain != nullptr ? e.gain[col + 1] : 1.f;
        store_hi_lo2(k_aout + crow * k_lda + col, __fmul_rn(x0.x, ga), __fmul_rn(x0.y, gb), k_lo);
      }
      if (k_ssqo != nullptr) {
        float sqv = __fmaf_rn(x0.x, x0.x, __fmul_rn(x0.y, x0.y));
        for (int o = L >> 1; o > 0; o >>= 1) sqv += __shfl_xor_sync(0xffffffffu, sqv, o);
        if (active && (cc & (L - 1)) == 0)
          k_ssqo[(size_t)(((((tile_m % (dd / BM)) << lgS) + z) << (lgPW - lgL)) + (cc >> lgL)) * k_ldssq + crow] = sqv;
      }
    }
  }
  fence_before();
  __syncthreads();
  fence_after();
  if (s_fail) ptx::drain_delay();                          // a wait gave up: stages already requested may still be landing
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(ncols) : "memory");
  }
}

}  // namespace tc
