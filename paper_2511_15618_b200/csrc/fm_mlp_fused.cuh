// The feed-forward half of a block, x += W2 gelu(W1 rms(x)), as ONE launch for passes with few
// token rows (a single sequence: up to 16 rows).  With so few rows the two projections are pure
// weight streaming and a launch is dominated by its fixed latencies (kernel boundary, operand
// fetch, cross-CTA reduction), so the chain W1 -> GELU -> W2 is cut along the hidden dimension
// instead of being run as two dependent launches:
//
//   * the d_ff hidden features are dealt out FB (16/32/64) per CTA; CTA (cluster c, rank r)
//     computes its FB features over the whole K = d with tcgen05.mma (features on the MMA's M
//     axis, token rows on N, hi and lo terms of the rows as one 2N-row operand), reads them back
//     from tensor memory, applies the RMSNorm scale of the rows and the GELU, and rounds them to
//     [hi | lo] bfloat16 terms;
//   * the CS CTAs of a cluster exchange those values through distributed shared memory (each CTA
//     pushes its FB columns into every peer's operand tile with st.async, counted on the peer's
//     mbarrier), so every CTA holds the cluster's HB = CS * FB hidden features as a K-major
//     operand;
//   * CTA r then multiplies its 128-column tile(s) of the output with the cluster's K range of W2
//     ([128 x HB], the standard slab layout) -- a partial sum over HB of the d_ff features;
//   * the partial tiles of the NC clusters go to global memory; the CTA that arrives last for an
//     output tile (ticket counter) adds them in cluster order to the residual rows, writes the new
//     residual, the next GEMM's operand rows bf16(x * gain) as [hi | lo] and the rows' partial sums
//     of squares (one slot per tile).  Nobody waits for anybody: every reduction order is fixed, so
//     a row's result does not depend on the number of rows in the launch.
// Both weight blocks of a CTA (FB x d of W1, 128 x HB of W2 per tile) are requested before
// griddepcontrol.wait; only the operand rows and the row statistics wait for the previous kernel.
#pragma once
#include "fm_common.cuh"
#include "fm_gemm_tc.cuh"
#include "fm_ptx.cuh"

namespace mlp {

constexpr int THREADS = 256;
constexpr int GROUPS = 4;          // W1 / operand slabs arrive in this many barrier groups

struct Args {
  const bf16* W1p;                 // [CTA g][K slab][FB rows x 64] 128-byte-swizzled images (FB*128 bytes each)
  const bf16* W2;                  // standard weight slabs [d/128 tiles][dff/64 slabs][128 x 64 image]
  const CUtensorMap* tmA;          // operand rows [rows_alloc, 2*d] as (K, rows, parts), box 64 x N x 2
  int d, dff, N, rows;             // N = 8 or 16: rows of the operand box; rows <= N
  int FB, CS, NC;                  // hidden features per CTA, cluster size, clusters (grid = CS x NC)
  const float* ssq_in;             // [ssq_n][ld_ssq] partial sums of squares of the operand rows
  int ssq_n, ld_ssq;
  float inv_d, eps;
  float* x;                        // residual rows [rows, d], updated in place
  const float* gain;               // gain of the next norm (null = 1)
  bf16* a_out;                     // next operand rows [rows, 2*d] as [hi | lo] (may be null)
  float* ssq_out; int ld_ssq_out;  // [d/128][ld] partial sums of squares of the new rows (may be null)
  float* part;                     // [NC][d/128][16][128] partial output tiles
  int* ticket;                     // [d/128], zero between launches
  const int* n_active;             // skip when *n_active == 0
  int* status;
};

// shared-memory plan (bytes), shared by host and device
struct Plan {
  int w1, w2, a, op2, stage, total;
};
__host__ __device__ inline Plan plan(int d, int N, int FB, int CS) {
  Plan p;
  const int slabs = d / 64, HB = CS * FB, tiles = (d / 128) / CS;
  p.w1 = slabs * FB * 128;
  p.w2 = tiles * (HB / 64) * 16384;
  p.a = slabs * 2 * N * 128;
  p.op2 = (HB / 64) * 2 * N * 128;
  p.stage = 2 * N * FB * 2;
  // the first MMA reads 128 rows from every W1 slab although only FB exist: what follows the last
  // slab must be mapped shared memory for another (128 - FB) * 128 bytes; the W2 block is
  const int tail = p.w2 + p.a + p.op2;
  const int pad = tail < (128 - FB) * 128 ? (128 - FB) * 128 - tail : 0;
  p.total = p.w1 + p.w2 + p.a + p.op2 + pad + ((p.stage + 1023) / 1024) * 1024 + 256 + 1024;
  return p;
}

// Hidden features per CTA and cluster size for a model, or FB = 0 when the fused form does not
// apply (then the two projections run as separate launches).
inline void shape(int d, int dff, int n_sm, int& FB, int& CS) {
  FB = 0; CS = 0;
  if (d % 128 != 0) return;
  const int OT = d / 128;
  if ((OT & (OT - 1)) != 0) return;
  const int cs = OT < 8 ? OT : 8;
  for (int fb = 16; fb <= 64; fb *= 2) {
    const int HB = cs * fb;
    if (HB % 64 != 0 || dff % HB != 0) continue;
    if (dff / fb > n_sm) continue;
    if (plan(d, 16, fb, cs).total > 220 * 1024) continue;
    FB = fb; CS = cs;
    return;
  }
}

__global__ void __launch_bounds__(THREADS) mlp_fused_kernel(const Args g) {
  if (g.n_active != nullptr && *g.n_active == 0) {
    ptx::grid_dep_launch();
    ptx::grid_dep_wait();
    return;
  }
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int N = g.N, N2 = 2 * g.N, FB = g.FB, CS = g.CS;
  const int slabs = g.d / 64, HB = CS * FB, hslabs = HB / 64, OT = g.d / 128, TPC = OT / CS;
  const int r = CS > 1 ? (int)tc::cluster_rank() : 0, c = blockIdx.y;
  const Plan pl = plan(g.d, N, FB, CS);
  unsigned char* w1s = sm;
  unsigned char* w2s = w1s + pl.w1;
  unsigned char* as = w2s + pl.w2;
  unsigned char* op2 = as + pl.a;
  const int pad_off = pl.total - (((pl.stage + 1023) / 1024) * 1024 + 256 + 1024);
  unsigned char* stage = sm + pad_off;
  uint64_t* bars = reinterpret_cast<uint64_t*>(stage + ((pl.stage + 1023) / 1024) * 1024);
  uint64_t* full = bars;                 // [GROUPS] W1 slabs + operand slabs of a group
  uint64_t* w2bar = bars + GROUPS;
  uint64_t* acc1 = w2bar + 1;
  uint64_t* acc2 = acc1 + 1;
  uint64_t* rbar = acc2 + 1;             // hidden features of the peers have arrived
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(rbar + 1);
  __shared__ int s_fail, s_last[2];
  __shared__ float s_inv[16];

  uint32_t ncols = 32;
  while ((int)ncols < N2 * (1 + TPC)) ncols <<= 1;
  const int per_group = (slabs + GROUPS - 1) / GROUPS;

  if (tid == 0) {
    s_fail = 0;
    for (int i = 0; i < GROUPS; ++i) ptx::mbar_init(full + i, 2);    // one arrival for the weights, one for the rows
    ptx::mbar_init(w2bar, 1);
    ptx::mbar_init(acc1, 1);
    ptx::mbar_init(acc2, 1);
    ptx::mbar_init(rbar, 1);
    ptx::fence_mbar_init();
    if (CS > 1) ptx::mbar_expect_tx(rbar, (uint32_t)((CS - 1) * N2 * FB * 2));
    ptx::prefetch_tmap(g.tmA);
    // weights do not depend on the previous kernel: request all of them now
    const bf16* w1src = g.W1p + (size_t)(c * CS + r) * slabs * (FB * 64);
    for (int q = 0; q < GROUPS; ++q) {
      const int k0 = q * per_group, k1 = min(slabs, k0 + per_group);
      if (k1 <= k0) { ptx::mbar_arrive(full + q); continue; }
      ptx::mbar_expect_tx(full + q, (uint32_t)((k1 - k0) * FB * 128));
      ptx::bulk_load(w1s + (size_t)k0 * FB * 128, w1src + (size_t)k0 * FB * 64, (uint32_t)((k1 - k0) * FB * 128), full + q);
    }
    ptx::mbar_expect_tx(w2bar, (uint32_t)(TPC * hslabs * 16384));
    for (int tt = 0; tt < TPC; ++tt) {
      const int T = r + tt * CS;
      const bf16* w2src = g.W2 + ((size_t)T * (g.dff / 64) + (size_t)c * hslabs) * (128 * 64);
      for (int j = 0; j < hslabs; ++j)
        ptx::bulk_load(w2s + (size_t)(tt * hslabs + j) * 16384, w2src + (size_t)j * (128 * 64), 16384, w2bar);
    }
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(ptx::smem_u32(tmem_slot)), "r"(ncols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc::fence_before();
  __syncthreads();
  tc::fence_after();
  const uint32_t tmem = *tmem_slot;
  ptx::grid_dep_launch();
  // peers will write into this CTA's operand tile and count on its barrier: every CTA of the
  // cluster must have initialised them before anybody sends (arrive now, wait before sending)
  if (CS > 1) asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");

  if (warp == 0) {
    // ---- operand rows, all K slabs: one copy per slab brings the hi and the lo tile
    if (lane < GROUPS) {
      const int k0 = lane * per_group, k1 = min(slabs, k0 + per_group);
      if (k1 > k0) ptx::mbar_expect_tx(full + lane, (uint32_t)((k1 - k0) * N2 * 128));
      else ptx::mbar_arrive(full + lane);
    }
    __syncwarp();
    ptx::grid_dep_wait();
    for (int k = lane; k < slabs; k += 32) {
      const int q = k / per_group;
      ptx::tma_load_3d(as + (size_t)k * N2 * 128, g.tmA, k * 64, 0, 0, full + q);
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---- first product: this CTA's FB hidden features over the whole K
      const uint32_t idesc = tc::instr_desc_bf16(N2);
      bool ok = true;
      for (int q = 0; q < GROUPS && ok; ++q) {
        const int k0 = q * per_group, k1 = min(slabs, k0 + per_group);
        if (!ptx::mbar_wait(full + q, 0)) { s_fail = 1; ok = false; break; }
        tc::fence_after();
        for (int k = k0; k < k1; ++k) {
          const uint64_t da = tc::smem_desc_sw128(ptx::smem_u32(w1s + (size_t)k * FB * 128));
          const uint64_t db = tc::smem_desc_sw128(ptx::smem_u32(as + (size_t)k * N2 * 128));
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) tc::mma_ss(tmem, da + 2 * kk, db + 2 * kk, idesc, (k > 0 || kk > 0) ? 1u : 0u);
        }
      }
      tc::commit(acc1);
    }
  } else if (warp == 2) {
    // ---- RMSNorm scale of the operand rows from the producer's partial sums of squares
    ptx::grid_dep_wait();
    if (g.ssq_in != nullptr) {
      const int sub = lane & 7;
      for (int n0 = 0; n0 < N; n0 += 4) {
        const int n = n0 + (lane >> 3);
        float ss = 0.f;
        for (int slot = sub; slot < g.ssq_n; slot += 8)
          ss += (n < g.rows) ? __ldcg(g.ssq_in + (size_t)slot * g.ld_ssq + n) : 0.f;
        ss += __shfl_xor_sync(0xffffffffu, ss, 1);
        ss += __shfl_xor_sync(0xffffffffu, ss, 2);
        ss += __shfl_xor_sync(0xffffffffu, ss, 4);
        if (sub == 0 && n < 16) s_inv[n] = n < g.rows ? rsqrtf(ss * g.inv_d + g.eps) : 0.f;
      }
    } else if (lane < 16) {
      s_inv[lane] = 1.f;
    }
  }
  ptx::grid_dep_wait();
  __syncthreads();                                         // s_inv is written

  // ---- hidden features back from tensor memory: lane f of the accumulator is feature f of this
  // CTA, columns [0, N) the product with the hi terms, [N, 2N) with the lo terms
  if (warp * 32 < FB) {
    bool ok = ptx::mbar_wait(acc1, 0);
    ok = __all_sync(0xffffffffu, ok);
    if (!ok && lane == 0) s_fail = 1;
    tc::fence_after();
    const int f = warp * 32 + lane;
    uint32_t a[16], b[16];
    float y[16];
    const uint32_t taddr = tmem + ((uint32_t)(warp * 32) << 16);
    if (ok) {
      tc::ld16(taddr, a);
      if (N == 16) {
        tc::ld16(taddr + 16, b);
#pragma unroll
        for (int n = 0; n < 16; ++n) y[n] = __uint_as_float(a[n]) + __uint_as_float(b[n]);
      } else {
#pragma unroll
        for (int n = 0; n < 8; ++n) { y[n] = __uint_as_float(a[n]) + __uint_as_float(a[8 + n]); y[8 + n] = 0.f; }
      }
    } else {
#pragma unroll
      for (int n = 0; n < 16; ++n) y[n] = 0.f;
    }
    bf16* st = reinterpret_cast<bf16*>(stage);             // [2N rows][FB features]
    if (f < FB) {
#pragma unroll
      for (int n = 0; n < 16; ++n) {
        if (n < N) {
          const float v = n < g.rows ? tc::gelu_erf_f(y[n] * s_inv[n]) : 0.f;
          const bf16 hi = __float2bfloat16(v);
          st[n * FB + f] = hi;
          st[(N + n) * FB + f] = __float2bfloat16(v - __bfloat162float(hi));
        }
      }
    }
  }
  if (CS > 1) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  __syncthreads();
  // ---- exchange: 16-byte chunks (8 features of one row) into every CTA's operand tile of the
  // second product, K-major with the 128-byte swizzle, feature r*FB + i at K index r*FB + i
  {
    const int cpr = FB / 8;                                 // chunks per row
    const uint32_t op2_u = ptx::smem_u32(op2);
    const uint32_t rbar_u = ptx::smem_u32(rbar);
    for (int it = tid; it < N2 * cpr; it += THREADS) {
      const int row = it / cpr, ch = it - row * cpr;
      const uint4 v = *reinterpret_cast<const uint4*>(stage + (size_t)(row * FB + ch * 8) * 2);
      const int fo = r * FB + ch * 8, j = fo >> 6, cj = (fo & 63) >> 3;
      const uint32_t off = (uint32_t)(j * N2 * 128 + row * 128 + ((cj ^ (row & 7)) << 4));
      *reinterpret_cast<uint4*>(op2 + off) = v;
      for (int p = 0; p < CS; ++p)
        if (p != r) tc::st_async_peer4(tc::map_peer(op2_u + off, (uint32_t)p), v.x, v.y, v.z, v.w, tc::map_peer(rbar_u, (uint32_t)p));
    }
  }
  ptx::fence_proxy_async();                                 // this CTA's own chunks: visible to the tensor core
  __syncthreads();
  if (warp == 1 && lane == 0) {
    // ---- second product: this CTA's output tile(s) over the cluster's HB hidden features
    bool ok = true;
    if (CS > 1) ok = tc::mbar_wait_cluster(rbar, 0);
    ok = ok && ptx::mbar_wait(w2bar, 0);
    if (!ok) s_fail = 1;
    ptx::fence_proxy_async();
    tc::fence_after();
    const uint32_t idesc = tc::instr_desc_bf16(N2);
    if (ok) {
      for (int tt = 0; tt < TPC; ++tt)
        for (int j = 0; j < hslabs; ++j) {
          const uint64_t da = tc::smem_desc_sw128(ptx::smem_u32(w2s + (size_t)(tt * hslabs + j) * 16384));
          const uint64_t db = tc::smem_desc_sw128(ptx::smem_u32(op2 + (size_t)j * N2 * 128));
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)
            tc::mma_ss(tmem + (uint32_t)(N2 * (1 + tt)), da + 2 * kk, db + 2 * kk, idesc, (j > 0 || kk > 0) ? 1u : 0u);
        }
    }
    tc::commit(acc2);
  }
  // ---- partial output tile(s) -> global memory: thread = output column
  if (warp < 4) {
    bool ok = ptx::mbar_wait(acc2, 0);
    ok = __all_sync(0xffffffffu, ok);
    if (!ok && lane == 0) s_fail = 1;
    tc::fence_after();
    for (int tt = 0; tt < TPC; ++tt) {
      const int T = r + tt * CS;
      uint32_t a[16], b[16];
      float y[16];
      const uint32_t taddr = tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)(N2 * (1 + tt));
      if (ok && !s_fail) {
        tc::ld16(taddr, a);
        if (N == 16) {
          tc::ld16(taddr + 16, b);
#pragma unroll
          for (int n = 0; n < 16; ++n) y[n] = __uint_as_float(a[n]) + __uint_as_float(b[n]);
        } else {
#pragma unroll
          for (int n = 0; n < 8; ++n) { y[n] = __uint_as_float(a[n]) + __uint_as_float(a[8 + n]); y[8 + n] = 0.f; }
        }
      } else {
#pragma unroll
        for (int n = 0; n < 16; ++n) y[n] = 0.f;
      }
      float* dst = g.part + ((size_t)(c * OT + T) * 16) * 128 + warp * 32 + lane;
#pragma unroll
      for (int n = 0; n < 16; ++n)
        if (n < g.rows) __stcg(dst + n * 128, y[n]);
    }
  }
  // ---- ticket per output tile: the CTA that arrives last adds the clusters' partial tiles
  __syncthreads();
  if (tid == 0) {
    if (s_fail) atomicExch(g.status, -5);
    for (int tt = 0; tt < TPC; ++tt) {
      int t;
      asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;" : "=r"(t) : "l"(g.ticket + r + tt * CS) : "memory");
      s_last[tt] = (t == g.NC - 1) ? 1 : 0;
    }
  }
  __syncthreads();
  for (int tt = 0; tt < TPC; ++tt) {
    if (!s_last[tt]) continue;
    const int T = r + tt * CS;
    // item = (row n, 4 columns): the 32 items of a row are one warp
    for (int it = tid; it < g.rows * 32; it += THREADS) {
      const int n = it >> 5, c4 = (it & 31) * 4;
      const float* src = g.part + ((size_t)T * 16 + n) * 128 + c4;
      const size_t cstride = (size_t)OT * 16 * 128;
      float* xr = g.x + (size_t)n * g.d + T * 128 + c4;
      float4 acc = *reinterpret_cast<const float4*>(xr);
      for (int c0 = 0; c0 < g.NC; c0 += 16) {
        float4 v[16];
#pragma unroll
        for (int k = 0; k < 16; ++k)
          v[k] = (c0 + k < g.NC) ? __ldcg(reinterpret_cast<const float4*>(src + (size_t)(c0 + k) * cstride)) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int k = 0; k < 16; ++k) { acc.x += v[k].x; acc.y += v[k].y; acc.z += v[k].z; acc.w += v[k].w; }
      }
      *reinterpret_cast<float4*>(xr) = acc;
      if (g.a_out != nullptr) {
        float4 gg = make_float4(1.f, 1.f, 1.f, 1.f);
        if (g.gain != nullptr) gg = *reinterpret_cast<const float4*>(g.gain + T * 128 + c4);
        bf16* ao = g.a_out + (size_t)n * 2 * g.d + T * 128 + c4;
        tc::store_hi_lo2(ao, acc.x * gg.x, acc.y * gg.y, g.d);
        tc::store_hi_lo2(ao + 2, acc.z * gg.z, acc.w * gg.w, g.d);
      }
      if (g.ssq_out != nullptr) {
        float sq = acc.x * acc.x + acc.y * acc.y + acc.z * acc.z + acc.w * acc.w;
        sq = warp_sum(sq);
        if (lane == 0) g.ssq_out[(size_t)T * g.ld_ssq_out + n] = sq;
      }
    }
    if (tid == 0) g.ticket[T] = 0;
  }
  tc::fence_before();
  __syncthreads();
  tc::fence_after();
  if (s_fail) ptx::drain_delay();
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(ncols) : "memory");
  }
}

}  // namespace mlp
