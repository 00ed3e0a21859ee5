// Few-row causal attention over one level's KV cache (Sec. 3.3: the candidates of a pass are
// masked causally among themselves; conditioning enters as prefix keys visible to every row).
//
// Split-KV design: one CTA per (sequence, kv-head, chunk of C cache slots).  The chunk's K and V
// tiles are staged in shared memory by TMA (2-D tensor maps over the cache, 128-byte swizzle);
// all query rows of the sequence that share the kv-head (rows of the pass x heads of the group)
// form the M axis of warp-level bf16 MMAs, so the cache is read once per pass, not once per row.
// Each warp owns a fixed quarter of the chunk's slots; softmax statistics are reduced with quad
// shuffles; the four warps and then the chunks are merged in a fixed order, so a row's result
// does not depend on how many other rows or sequences the launch holds.  The CTA that finishes
// last for a (sequence, kv-head) merges the chunk partials (ticket counter, no waiting).
#pragma once
#include "fm_common.cuh"
#include "fm_ptx.cuh"

struct AttnArgs {
  Dims dm;
  SeqState st;
  int batch, level;
  const bf16* q;              // [rows, H*dh] bf16, rotated and scaled by log2(e)/sqrt(dh)
  const CUtensorMap* tmK;     // cache as 2-D [B*Hkv*slots, dh], box 64 x 64
  const CUtensorMap* tmV;
  float* part;                // [B*Hkv, max_chunks, MROWS, dh + 2]
  int* ticket;                // [B*Hkv], zero between launches
  bf16* out;                  // [rows, H*dh]
  int max_chunks, mrows;      // mrows = rows_per_seq * group rounded up to 16
};

template <int DH, int C>
struct AttnSmem {
  static constexpr int HALVES = DH / 64;
  static constexpr int TILE = HALVES * C * 128;            // bytes of one K (or V) tile
  static constexpr int PART = 4 * 16 * (DH + 2) * 4;       // per-warp partials of one m-tile
  static constexpr int BYTES = 2 * TILE + PART + 64 + 1024; // + barrier + alignment slack
};

// position currently held by cache slot `slot` (-1: prefix entry, -2: nothing usable)
__device__ inline int attn_slot_pos(int slot, int P, int cap, int p_max) {
  if (slot < P) return -1;
  const int r = slot - P;
  if (r >= cap || r > p_max) return -2;
  return r + ((p_max - r) / cap) * cap;
}

template <int DH, int C>
__global__ void __launch_bounds__(128) attn_split_kernel(const AttnArgs a) {
  using SM = AttnSmem<DH, C>;
  constexpr int NT = C / 4 / 8;                 // 8-key n-tiles per warp
  constexpr int KS = DH / 16;                   // k-steps of Q K^T
  const Dims& dm = a.dm;
  const int chunk = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t4 = lane & 3;
  ptx::grid_dep_launch();
  ptx::grid_dep_wait();                            // queries and the new keys/values come from the previous kernel
  if (b >= a.batch) return;
  const int n = a.st.nrow[b];
  if (n <= 0) return;
  const int Lb = a.st.L[b], ratio = fm_ratio(a.level);
  const int p0 = (Lb + ratio - 1) / ratio;
  const int nq = (Lb + n - 1) / ratio - p0 + 1;
  if (nq <= 0) return;
  const int p_max = p0 + nq - 1;
  const int P = dm.P, cap = dm.cap[a.level], W = dm.window[a.level];
  const int slots = P + cap;
  const int used = P + min(cap, p_max + 1);
  const int n_chunks = (used + C - 1) / C;
  if (chunk >= n_chunks) return;
  const int group = dm.H / dm.Hkv;
  const int M = nq * group;
  const int m_rows = fm_rows_per_seq(dm, a.level);

  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  unsigned char* Ks = sm;
  unsigned char* Vs = sm + SM::TILE;
  float* pw = reinterpret_cast<float*>(sm + 2 * SM::TILE);            // [4][16][DH+2]
  uint64_t* bar = reinterpret_cast<uint64_t*>(sm + 2 * SM::TILE + SM::PART);
  __shared__ int s_last;

  if (threadIdx.x == 0) {
    ptx::mbar_init(bar, 1);
    ptx::fence_mbar_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    ptx::mbar_expect_tx(bar, 2 * SM::TILE);
    const int row0 = (b * dm.Hkv + hk) * slots + chunk * C;
#pragma unroll
    for (int h = 0; h < SM::HALVES; ++h)
#pragma unroll
      for (int kb = 0; kb < C / 64; ++kb) {
        ptx::tma_load_2d(Ks + (h * C + kb * 64) * 128, a.tmK, h * 64, row0 + kb * 64, bar);
        ptx::tma_load_2d(Vs + (h * C + kb * 64) * 128, a.tmV, h * 64, row0 + kb * 64, bar);
      }
  }
  // positions held by this thread's key columns: n-tile nt, element e -> key warp*C/4 + nt*8 + 2*t4 + e
  int kpos[NT][2];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt)
#pragma unroll
    for (int e = 0; e < 2; ++e)
      kpos[nt][e] = attn_slot_pos(chunk * C + warp * (C / 4) + nt * 8 + 2 * t4 + e, P, cap, p_max);

  const bool ready = ptx::mbar_wait(bar, 0);
  if (!ready) {                                    // never expected; leave without touching the tiles
    if (threadIdx.x == 0) atomicExch(a.st.status, -5);
    return;
  }
  const uint32_t Ks_u = ptx::smem_u32(Ks), Vs_u = ptx::smem_u32(Vs);
  float* gpart = a.part + ((size_t)(b * dm.Hkv + hk) * a.max_chunks + chunk) * a.mrows * (DH + 2);

  for (int mt = 0; mt * 16 < M; ++mt) {
    // ---- Q fragments of this m-tile (rows idx = mt*16 + g, +8; idx = r*group + gh)
    uint32_t qa[KS][4];
    int prow[2];
#pragma unroll
    for (int hrow = 0; hrow < 2; ++hrow) {
      const int idx = mt * 16 + g + hrow * 8;
      const bool ok = idx < M;
      const int r = ok ? idx / group : 0, gh = ok ? idx - r * group : 0;
      prow[hrow] = ok ? p0 + r : -100;
      const bf16* qp = a.q + ((size_t)(b * m_rows + r) * dm.H + hk * group + gh) * DH;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        qa[ks][hrow] = ok ? *reinterpret_cast<const uint32_t*>(qp + ks * 16 + 2 * t4) : 0u;
        qa[ks][2 + hrow] = ok ? *reinterpret_cast<const uint32_t*>(qp + ks * 16 + 8 + 2 * t4) : 0u;
      }
    }
    // ---- S = Q K^T over this warp's C/4 keys
    float s[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
      for (int np = 0; np < NT / 2; ++np) {
        const int key = warp * (C / 4) + np * 16 + (lane & 7) + (lane >> 4) * 8;
        const int ch = ks * 2 + ((lane >> 3) & 1);
        uint32_t r0, r1, r2, r3;
        ptx::ldmatrix_x4(r0, r1, r2, r3, Ks_u + (ch >> 3) * C * 128 + ptx::swz128(key, ch & 7));
        ptx::mma_bf16_16816(s[2 * np], qa[ks], r0, r1);
        ptx::mma_bf16_16816(s[2 * np + 1], qa[ks], r2, r3);
      }
    }
    // ---- mask, row max, exponentials, row sums (rows g and g+8; quad = the 4 lanes sharing g)
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int kp = kpos[nt][e & 1], pr = prow[e >> 1];
        const bool vis = kp == -1 || (kp >= 0 && kp <= pr && (W == 0 || kp >= pr - W + 1));
        s[nt][e] = (vis && pr >= 0) ? s[nt][e] : -INFINITY;
        mx[e >> 1] = fmaxf(mx[e >> 1], s[nt][e]);
      }
#pragma unroll
    for (int hrow = 0; hrow < 2; ++hrow) {
      mx[hrow] = fmaxf(mx[hrow], __shfl_xor_sync(0xffffffffu, mx[hrow], 1));
      mx[hrow] = fmaxf(mx[hrow], __shfl_xor_sync(0xffffffffu, mx[hrow], 2));
    }
    const float base[2] = {mx[0] == -INFINITY ? 0.f : mx[0], mx[1] == -INFINITY ? 0.f : mx[1]};
    float ls[2] = {0.f, 0.f};
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        s[nt][e] = exp2f(s[nt][e] - base[e >> 1]);
        ls[e >> 1] += s[nt][e];
      }
#pragma unroll
    for (int hrow = 0; hrow < 2; ++hrow) {
      ls[hrow] += __shfl_xor_sync(0xffffffffu, ls[hrow], 1);
      ls[hrow] += __shfl_xor_sync(0xffffffffu, ls[hrow], 2);
    }
    // ---- O = P V
    float o[DH / 8][4];
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
#pragma unroll
    for (int kk = 0; kk < NT / 2; ++kk) {
      uint32_t pa[4];
      pa[0] = ptx::pack_bf16(s[2 * kk][0], s[2 * kk][1]);
      pa[1] = ptx::pack_bf16(s[2 * kk][2], s[2 * kk][3]);
      pa[2] = ptx::pack_bf16(s[2 * kk + 1][0], s[2 * kk + 1][1]);
      pa[3] = ptx::pack_bf16(s[2 * kk + 1][2], s[2 * kk + 1][3]);
#pragma unroll
      for (int dp = 0; dp < DH / 16; ++dp) {
        const int key = warp * (C / 4) + kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
        const int ch = dp * 2 + (lane >> 4);
        uint32_t r0, r1, r2, r3;
        ptx::ldmatrix_x4_trans(r0, r1, r2, r3, Vs_u + (ch >> 3) * C * 128 + ptx::swz128(key, ch & 7));
        ptx::mma_bf16_16816(o[2 * dp], pa, r0, r1);
        ptx::mma_bf16_16816(o[2 * dp + 1], pa, r2, r3);
      }
    }
    // ---- the four warps' partials -> shared, merged in warp order -> chunk partial in global
    __syncthreads();                                // previous m-tile's readers are done with pw
    float* mine = pw + warp * 16 * (DH + 2);
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) {
      mine[g * (DH + 2) + i * 8 + 2 * t4] = o[i][0];
      mine[g * (DH + 2) + i * 8 + 2 * t4 + 1] = o[i][1];
      mine[(g + 8) * (DH + 2) + i * 8 + 2 * t4] = o[i][2];
      mine[(g + 8) * (DH + 2) + i * 8 + 2 * t4 + 1] = o[i][3];
    }
    if (t4 == 0) {
      mine[g * (DH + 2) + DH] = mx[0]; mine[g * (DH + 2) + DH + 1] = ls[0];
      mine[(g + 8) * (DH + 2) + DH] = mx[1]; mine[(g + 8) * (DH + 2) + DH + 1] = ls[1];
    }
    __syncthreads();
    for (int e = threadIdx.x; e < 16 * (DH + 2); e += 128) {
      const int i = e / (DH + 2), c = e - i * (DH + 2);
      if (mt * 16 + i >= M) continue;
      float mm = -INFINITY;
#pragma unroll
      for (int w = 0; w < 4; ++w) mm = fmaxf(mm, pw[(w * 16 + i) * (DH + 2) + DH]);
      float v;
      if (c == DH) v = mm;
      else {
        v = 0.f;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
          const float mw = pw[(w * 16 + i) * (DH + 2) + DH];
          const float sc = mw == -INFINITY ? 0.f : exp2f(mw - mm);
          v += sc * pw[(w * 16 + i) * (DH + 2) + (c == DH + 1 ? DH + 1 : c)];
        }
      }
      gpart[(size_t)(mt * 16 + i) * (DH + 2) + c] = v;
    }
  }

  // ---- ticket: the CTA that arrives last for this (sequence, kv-head) merges all chunk partials
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const int t = atomicAdd(a.ticket + b * dm.Hkv + hk, 1);
    s_last = (t == n_chunks - 1) ? 1 : 0;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  const float* base = a.part + (size_t)(b * dm.Hkv + hk) * a.max_chunks * a.mrows * (DH + 2);
  const size_t cstride = (size_t)a.mrows * (DH + 2);
  for (int e = threadIdx.x; e < M * DH; e += 128) {
    const int idx = e / DH, c = e - idx * DH;
    const float* pr = base + (size_t)idx * (DH + 2);
    float mm = -INFINITY;
    for (int ck = 0; ck < n_chunks; ++ck) mm = fmaxf(mm, __ldcg(pr + ck * cstride + DH));
    float acc = 0.f, lsum = 0.f;
    int ck = 0;
    for (; ck + 4 <= n_chunks; ck += 4) {          // loads first, then the sums in chunk order
      float m4[4], l4[4], v4[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const float* q = pr + (ck + u) * cstride;
        m4[u] = __ldcg(q + DH); l4[u] = __ldcg(q + DH + 1); v4[u] = __ldcg(q + c);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const float sc = m4[u] == -INFINITY ? 0.f : exp2f(m4[u] - mm);
        acc += sc * v4[u];
        lsum += sc * l4[u];
      }
    }
    for (; ck < n_chunks; ++ck) {
      const float* q = pr + ck * cstride;
      const float mc = __ldcg(q + DH);
      const float sc = mc == -INFINITY ? 0.f : exp2f(mc - mm);
      acc += sc * __ldcg(q + c);
      lsum += sc * __ldcg(q + DH + 1);
    }
    const int r = idx / group, gh = idx - r * group;
    a.out[((size_t)(b * m_rows + r) * dm.H + hk * group + gh) * DH + c] = __float2bfloat16(acc / lsum);
  }
  if (threadIdx.x == 0) a.ticket[b * dm.Hkv + hk] = 0;
}
