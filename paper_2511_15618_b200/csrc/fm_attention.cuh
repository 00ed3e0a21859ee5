// Few-row causal attention over one level's KV cache (Sec. 3.3: the candidates of a pass are
// masked causally among themselves; conditioning enters as prefix keys visible to every row).
//
// Streaming split-KV design.  The cache of a (sequence, kv-head) is cut into chunks of C slots and
// the chunks into groups of G consecutive chunks (G is fixed per level when the context is
// created).  One CTA streams one group: a producer warp brings the K and V tiles of its chunks in
// with TMA (2-D tensor maps over the cache, 128-byte swizzle) through a ring of shared-memory
// stages; NW compute warps each own a fixed 16-slot slice of every chunk and keep their own
// running softmax state (max, sum, output) across the group's chunks, so warps never wait for one
// another while streaming.  All query rows of the sequence that share the kv-head (rows of the
// pass x heads of the group, 16 per CTA) form the M axis of warp-level bf16 MMAs, so the cache is
// read once per pass, not once per row; softmax statistics are reduced with quad shuffles.
// At the end of the group the warps' states are merged in warp order; the groups' states go to a
// scratch buffer in global memory and are merged in group order by the CTA that finishes last
// (ticket counter, nobody waits).  (Merging through a thread-block cluster's shared memory was
// measured and is slower here: CTAs this large are gang-scheduled microseconds apart.)
// Slices, chunks and groups are fixed by slot index, so a row's result does not depend on how many
// other rows or sequences the launch holds, nor on the cache length at the time it is computed.
// Programmatic dependent launch: cache entries written by earlier passes do not depend on the
// previous kernel, so chunks that hold none of this pass's new slots are requested before
// griddepcontrol.wait.
#pragma once
#include "fm_common.cuh"
#include "fm_ptx.cuh"

struct AttnArgs {
  Dims dm;
  SeqState st;
  int batch, level;
  const bf16* q;              // [rows, H*dh] bf16, rotated and scaled by log2(e)/sqrt(dh)
  const CUtensorMap* tmK;     // cache as 2-D [B*Hkv*slots, dh], box C x 64
  const CUtensorMap* tmV;
  float* part;                // [B*Hkv*MT, max_groups, 16, dh + 2]
  int* ticket;                // [B*Hkv*MT], zero between launches
  bf16* out;                  // [rows, 2*H*dh]: the next GEMM's operand rows as [hi | lo] bfloat16 terms
  int G;                      // chunks per group
  int max_groups;             // groups the cache of this level can hold (= gridDim.x)
  int MT;                     // 16-row query tiles per (sequence, kv-head)
  // Draft mode (SP-Block / HF-Block queries, Sec. 3.1): draft_nq > 0 query rows per sequence, none of
  // them in the cache; every row sees what the last accepted position of the level sees (the prefix
  // and positions max(0, p - W + 1) .. p with p = floor((L - 1) / ratio)).  Row r of sequence b is
  // read at q[(b * draft_nq + r)] and written to out row r * out_row_stride + b.
  int draft_nq;
  int out_row_stride;
};

template <int DH, int C, int NW>
struct AttnCfg {
  static_assert(C == 16 * NW, "every compute warp owns 16 slots of a chunk");
  static constexpr int STAGES = 4;
  static constexpr int HALVES = DH / 64;
  static constexpr int TILE = C * DH * 2;                   // bytes of one K (or V) tile
  static constexpr int STAGE = 2 * TILE;
  static constexpr int RING = STAGES * STAGE;
  static constexpr int STATE = 16 * (DH + 2) * 4;           // one merged state: 16 rows x (output, max, sum)
  static constexpr int MERGE = (NW + 1) * STATE;            // the warps' states and the merged one, aliasing the ring
  static constexpr int WORK = RING > MERGE ? RING : MERGE;
  static constexpr int BYTES = WORK + 128 + 1024;           // + barriers + alignment slack
  // groups the last CTA can merge: their states plus 16 x (groups + 1) weights are staged in WORK
  static constexpr int MAX_GROUPS_FIT = (WORK - 64) / (STATE + 64);
  static constexpr int MAX_GROUPS = MAX_GROUPS_FIT < 24 ? MAX_GROUPS_FIT : 24;
  static constexpr int THREADS = (NW + 1) * 32;
};

namespace attn {
__device__ inline void store_out(bf16* out, size_t at, float v, int lo_off) {
  const bf16 hi = __float2bfloat16(v);
  out[at] = hi;
  out[at + lo_off] = __float2bfloat16(v - __bfloat162float(hi));
}
__device__ inline int div_ratio(int x, int level) { return level == 0 ? x : (level == 1 ? x / 3 : x / 9); }
}  // namespace attn

// grid (max_groups, Hkv * MT, batch); block (NW + 1) warps: NW compute warps and one producer warp.
template <int DH, int C, int NW>
__global__ void __launch_bounds__((NW + 1) * 32) attn_stream_kernel(const AttnArgs a) {
  using CF = AttnCfg<DH, C, NW>;
  constexpr int KS = DH / 16;                   // k-steps of Q K^T
  const Dims& dm = a.dm;
  const int u = blockIdx.x;
  const int hk = a.MT == 1 ? (int)blockIdx.y : (int)blockIdx.y / a.MT;
  const int mt = (int)blockIdx.y - hk * a.MT;
  const int b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t4 = lane & 3;
  ptx::grid_dep_launch();
  // ---- what this CTA has to do (per-pass state is final before the pass's first kernel starts)
  const int level = a.level;
  const int n = b < a.batch ? a.st.nrow[b] : 0;
  const int Lb = b < a.batch ? a.st.L[b] : 0;
  const int ratio = fm_ratio(level);
  const bool dmode = a.draft_nq > 0;
  const int p0 = dmode ? attn::div_ratio(Lb - 1, level) : attn::div_ratio(Lb + ratio - 1, level);
  const int nq = n > 0 ? (dmode ? a.draft_nq : attn::div_ratio(Lb + n - 1, level) - p0 + 1) : 0;
  const int p_max = dmode ? p0 : p0 + nq - 1;
  const int P = dm.P, cap = dm.cap[level], W = dm.window[level];
  const int slots = P + cap;
  const int used = P + min(cap, p_max + 1);
  const int n_chunks = (used + C - 1) / C;
  const int n_groups = (n_chunks + a.G - 1) / a.G;
  const int group = dm.H / dm.Hkv;
  const int M = nq * group;
  if (nq <= 0 || mt * 16 >= M || u >= n_groups || n_groups > CF::MAX_GROUPS) {
    // nothing of the cache falls into this group yet; or more groups than the merge can stage
    // (the host sizes G so that this never happens): report, write nothing
    if (n_groups > CF::MAX_GROUPS && threadIdx.x == 0) atomicExch(a.st.status, -3);   // capacity
    ptx::grid_dep_wait();                          // keep the launch chain ordered
    return;
  }
  const int c_lo = u * a.G, n_my = min(a.G, n_chunks - c_lo);
  const int m_rows = dmode ? a.draft_nq : fm_rows_per_seq(dm, level);

  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* full = reinterpret_cast<uint64_t*>(sm + CF::WORK);
  uint64_t* empty = full + CF::STAGES;
  __shared__ int s_last, s_fail, s_pre;

  // slots written by this pass: P + (p mod cap), p = p0..p_max: one run of nq slots from new_lo,
  // which may wrap around the end of the ring once
  const int new_lo = P + p0 % cap;
  const int n_new = dmode ? 0 : nq;                          // draft queries append nothing
  auto has_new = [&](int c) {
    const int lo = c * C, hi = lo + C;                       // [lo, hi)
    const int e1 = min(new_lo + n_new, slots);               // first part [new_lo, e1)
    const int n2 = new_lo + n_new - e1;                      // wrapped part [P, P + n2)
    return (new_lo < hi && e1 > lo) || (n2 > 0 && P < hi && P + n2 > lo);
  };
  const int row_base = (b * dm.Hkv + hk) * slots;
  auto issue = [&](int i) {
    const int st = i % CF::STAGES;
    unsigned char* Ks = sm + st * CF::STAGE;
    unsigned char* Vs = Ks + CF::TILE;
    ptx::mbar_expect_tx(full + st, CF::STAGE);
    const int row0 = row_base + (c_lo + i) * C;
#pragma unroll
    for (int h = 0; h < CF::HALVES; ++h) {
      ptx::tma_load_2d(Ks + h * C * 128, a.tmK, h * 64, row0, full + st);
      ptx::tma_load_2d(Vs + h * C * 128, a.tmV, h * 64, row0, full + st);
    }
  };
  if (threadIdx.x == 0) {
    s_fail = 0;
    for (int i = 0; i < CF::STAGES; ++i) { ptx::mbar_init(full + i, 1); ptx::mbar_init(empty + i, NW); }
    ptx::fence_mbar_init();
    // chunks that hold old entries only are requested at once, before the dependency wait
    int i = 0;
    const int pre = n_my < CF::STAGES ? n_my : CF::STAGES;
    while (i < pre && !has_new(c_lo + i)) { issue(i); ++i; }
    s_pre = i;
  }
  __syncthreads();

  // running state of this warp's slices: rows g and g+8 of the query tile
  float o[DH / 8][4];
  float mrun[2] = {-INFINITY, -INFINITY}, lrun[2] = {0.f, 0.f};
#pragma unroll
  for (int i = 0; i < DH / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;

  if (warp == NW) {
    // ---- producer
    if (lane == 0) {
      ptx::grid_dep_wait();
      for (int i = s_pre; i < n_my; ++i) {
        if (i >= CF::STAGES && !ptx::mbar_wait(empty + i % CF::STAGES, ((i / CF::STAGES) - 1) & 1)) { s_fail = 1; break; }
        issue(i);
      }
    }
    __syncwarp();
  } else {
    // ---- compute warps
    ptx::grid_dep_wait();                          // queries come from the previous kernel
    // Q fragments of this CTA's query tile (rows idx = mt*16 + g, +8; idx = r*group + gh)
    uint32_t qa[KS][4];
    int prow[2];
#pragma unroll
    for (int hrow = 0; hrow < 2; ++hrow) {
      const int idx = mt * 16 + g + hrow * 8;
      const bool ok = idx < M;
      const int r = ok ? (group == 1 ? idx : idx / group) : 0, gh = ok ? idx - r * group : 0;
      prow[hrow] = ok ? (dmode ? p0 : p0 + r) : -100;
      const bf16* qp = a.q + ((size_t)(b * m_rows + r) * dm.H + hk * group + gh) * DH;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        qa[ks][hrow] = ok ? *reinterpret_cast<const uint32_t*>(qp + ks * 16 + 2 * t4) : 0u;
        qa[ks][2 + hrow] = ok ? *reinterpret_cast<const uint32_t*>(qp + ks * 16 + 8 + 2 * t4) : 0u;
      }
    }
    // slot -> position: behind the prefix, slot P + r holds position r + k*cap with
    // k = floor((p_max - r) / cap) = wrap_q if r <= wrap_r else wrap_q - 1
    const int wrap_q = p_max / cap, wrap_r = p_max - wrap_q * cap;
    for (int i = 0; i < n_my; ++i) {
      const int st = i % CF::STAGES;
      // is every slot of the chunk visible to every row of the pass?  (the common case: prefix, or
      // old positions inside every row's window) -- then no masks are needed
      const int s_lo = (c_lo + i) * C, s_hi = s_lo + C - 1;
      bool all_vis = s_hi < P;
      if (!all_vis && s_lo >= P) {
        const int r_lo = s_lo - P, r_hi = s_hi - P;
        if (r_hi < cap && r_hi <= p_max && (r_hi <= wrap_r || r_lo > wrap_r)) {
          const int k = r_hi <= wrap_r ? wrap_q : wrap_q - 1;
          all_vis = r_hi + k * cap <= p0 && (W == 0 || r_lo + k * cap >= p_max - W + 1);
        }
      }
      if (!ptx::mbar_wait(full + st, (i / CF::STAGES) & 1)) { s_fail = 1; break; }
      const uint32_t Ks_u = ptx::smem_u32(sm + st * CF::STAGE), Vs_u = Ks_u + CF::TILE;
      // ---- S = Q K^T over this warp's 16 slots
      float s[2][4];
      s[0][0] = s[0][1] = s[0][2] = s[0][3] = s[1][0] = s[1][1] = s[1][2] = s[1][3] = 0.f;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        const int key = warp * 16 + (lane & 7) + (lane >> 4) * 8;
        const int ch = ks * 2 + ((lane >> 3) & 1);
        uint32_t r0, r1, r2, r3;
        ptx::ldmatrix_x4(r0, r1, r2, r3, Ks_u + (ch >> 3) * C * 128 + ptx::swz128(key, ch & 7));
        ptx::mma_bf16_16816(s[0], qa[ks], r0, r1);
        ptx::mma_bf16_16816(s[1], qa[ks], r2, r3);
      }
      if (!all_vis) {
        // positions of this thread's key columns: n-tile nt, element e -> slot base + nt*8 + 2*t4 + e
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int slot = s_lo + warp * 16 + nt * 8 + 2 * t4 + e;
            const int r = slot - P;
            const int kp = slot < P ? -1 : ((r >= cap || r > p_max) ? -2 : r + (r <= wrap_r ? wrap_q : wrap_q - 1) * cap);
#pragma unroll
            for (int hrow = 0; hrow < 2; ++hrow) {
              const int pr = prow[hrow];
              const bool vis = kp == -1 || (kp >= 0 && kp <= pr && (W == 0 || kp >= pr - W + 1));
              if (!(vis && pr >= 0)) s[nt][hrow * 2 + e] = -INFINITY;
            }
          }
      }
      // ---- running max, exponentials, running sums (rows g and g+8; quad = the 4 lanes sharing g)
      float mx[2];
      mx[0] = fmaxf(fmaxf(s[0][0], s[0][1]), fmaxf(s[1][0], s[1][1]));
      mx[1] = fmaxf(fmaxf(s[0][2], s[0][3]), fmaxf(s[1][2], s[1][3]));
      float scale[2], base[2];
#pragma unroll
      for (int hrow = 0; hrow < 2; ++hrow) {
        mx[hrow] = fmaxf(mx[hrow], __shfl_xor_sync(0xffffffffu, mx[hrow], 1));
        mx[hrow] = fmaxf(mx[hrow], __shfl_xor_sync(0xffffffffu, mx[hrow], 2));
        const float mnew = fmaxf(mrun[hrow], mx[hrow]);
        base[hrow] = mnew == -INFINITY ? 0.f : mnew;
        scale[hrow] = mnew == mrun[hrow] ? (mnew == -INFINITY ? 0.f : 1.f) : exp2f(mrun[hrow] - base[hrow]);
        mrun[hrow] = mnew;
      }
      float ls[2] = {0.f, 0.f};
#pragma unroll
      for (int nt = 0; nt < 2; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          s[nt][e] = exp2f(s[nt][e] - base[e >> 1]);
          ls[e >> 1] += s[nt][e];
        }
#pragma unroll
      for (int hrow = 0; hrow < 2; ++hrow) {
        ls[hrow] += __shfl_xor_sync(0xffffffffu, ls[hrow], 1);
        ls[hrow] += __shfl_xor_sync(0xffffffffu, ls[hrow], 2);
        lrun[hrow] = lrun[hrow] * scale[hrow] + ls[hrow];
      }
      // the running output only needs rescaling when a row's maximum moved (scale 1 changes nothing)
      if (__any_sync(0xffffffffu, scale[0] != 1.f || scale[1] != 1.f)) {
#pragma unroll
        for (int i2 = 0; i2 < DH / 8; ++i2) {
          o[i2][0] *= scale[0]; o[i2][1] *= scale[0];
          o[i2][2] *= scale[1]; o[i2][3] *= scale[1];
        }
      }
      // ---- O += P V
      uint32_t pa[4];
      pa[0] = ptx::pack_bf16(s[0][0], s[0][1]);
      pa[1] = ptx::pack_bf16(s[0][2], s[0][3]);
      pa[2] = ptx::pack_bf16(s[1][0], s[1][1]);
      pa[3] = ptx::pack_bf16(s[1][2], s[1][3]);
#pragma unroll
      for (int dp = 0; dp < DH / 16; ++dp) {
        const int key = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
        const int ch = dp * 2 + (lane >> 4);
        uint32_t r0, r1, r2, r3;
        ptx::ldmatrix_x4_trans(r0, r1, r2, r3, Vs_u + (ch >> 3) * C * 128 + ptx::swz128(key, ch & 7));
        ptx::mma_bf16_16816(o[2 * dp], pa, r0, r1);
        ptx::mma_bf16_16816(o[2 * dp + 1], pa, r2, r3);
      }
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(empty + st);           // this warp is done with the stage
    }
  }
  // ---- the warps' states -> shared (the ring is idle once every warp is here), merged in warp order
  __syncthreads();
  if (s_fail) {                                              // a bounded wait gave up: report, write nothing
    if (threadIdx.x == 0) atomicExch(a.st.status, -5);
    ptx::drain_delay();                                      // chunks already requested may still be landing
    return;
  }
  // Merge of the NW warps' states, in warp order.  First every warp publishes its row maxima and
  // sums; each thread then rescales its own registers to the common maximum of its rows, after
  // which the merged output is a plain sum over the warps.
  float* pw = reinterpret_cast<float*>(sm);                  // [NW][16][DH] rescaled outputs
  float* ml = pw + NW * 16 * DH;                             // [NW][16][2] maxima and sums
  if (warp < NW && t4 == 0) {
    ml[(warp * 16 + g) * 2] = mrun[0]; ml[(warp * 16 + g) * 2 + 1] = lrun[0];
    ml[(warp * 16 + g + 8) * 2] = mrun[1]; ml[(warp * 16 + g + 8) * 2 + 1] = lrun[1];
  }
  __syncthreads();
  if (warp < NW) {
    float sc[2];
#pragma unroll
    for (int hrow = 0; hrow < 2; ++hrow) {
      float mm = -INFINITY;
#pragma unroll
      for (int w = 0; w < NW; ++w) mm = fmaxf(mm, ml[(w * 16 + g + hrow * 8) * 2]);
      sc[hrow] = mrun[hrow] == -INFINITY ? 0.f : exp2f(mrun[hrow] - mm);
    }
    float* mine = pw + warp * 16 * DH;
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) {
      *reinterpret_cast<float2*>(mine + g * DH + i * 8 + 2 * t4) = make_float2(o[i][0] * sc[0], o[i][1] * sc[0]);
      *reinterpret_cast<float2*>(mine + (g + 8) * DH + i * 8 + 2 * t4) = make_float2(o[i][2] * sc[1], o[i][3] * sc[1]);
    }
  }
  __syncthreads();
  const size_t pt = ((size_t)(b * dm.Hkv + hk) * a.MT + mt);
  float* gpart = a.part + (pt * a.max_groups + u) * 16 * (DH + 2);
  const bool single = n_groups == 1;
  for (int e = threadIdx.x; e < 16 * (DH + 2); e += CF::THREADS) {
    const int i = e / (DH + 2), c = e - i * (DH + 2);
    const int idx = mt * 16 + i;
    if (idx >= M) continue;
    float val;
    if (c < DH) {
      val = 0.f;
#pragma unroll
      for (int w = 0; w < NW; ++w) val += pw[(w * 16 + i) * DH + c];
    } else {
      float mm = -INFINITY;
#pragma unroll
      for (int w = 0; w < NW; ++w) mm = fmaxf(mm, ml[(w * 16 + i) * 2]);
      if (c == DH) val = mm;
      else {
        val = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) {
          const float mw = ml[(w * 16 + i) * 2];
          val += (mw == -INFINITY ? 0.f : exp2f(mw - mm)) * ml[(w * 16 + i) * 2 + 1];
        }
      }
    }
    if (!single) gpart[(size_t)i * (DH + 2) + c] = val;      // columns: output, maximum, sum
    else if (c < DH) pw[NW * 16 * DH + NW * 32 + i * DH + c] = val;
    else if (c == DH + 1) ml[NW * 32 + 16 * DH + i] = val;
  }
  if (single) {                                              // one group: normalise and store the result
    __syncthreads();
    const float* res = pw + NW * 16 * DH + NW * 32;          // [16][DH] sums, then [16] normalisers
    for (int e = threadIdx.x; e < 16 * DH; e += CF::THREADS) {
      const int i = e / DH, c = e - i * DH;
      const int idx = mt * 16 + i;
      if (idx >= M) continue;
      const int r = group == 1 ? idx : idx / group, gh = idx - r * group;
      const size_t orow = a.out_row_stride > 0 ? (size_t)r * a.out_row_stride + b : (size_t)(b * m_rows + r);
      attn::store_out(a.out, (orow * 2 * dm.H + hk * group + gh) * DH + c, res[e] / res[16 * DH + i], dm.H * DH);
    }
    return;
  }

  // ---- merge of the groups, in group order
  const int rows_here = min(16, M - mt * 16);
  constexpr int gstride = 16 * (DH + 2);            // floats per state; the ring holds RING / STATE of them
  // ticket: the CTA that arrives last for this (sequence, kv-head, query tile) merges.  The
  // barrier orders the CTA's stores before thread 0's release; the last CTA's acquire, followed by
  // the barrier, orders every group's stores before its loads.
  __syncthreads();
  if (threadIdx.x == 0) {
    int t;
    asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;" : "=r"(t) : "l"(a.ticket + pt) : "memory");
    s_last = (t == n_groups - 1) ? 1 : 0;
  }
  __syncthreads();
  if (!s_last) return;
  // Bring the groups' states into shared memory first: one round of wide, independent loads (the
  // ring is idle).  Merging straight from global memory would serialise a load per group.
  const float4* src4 = reinterpret_cast<const float4*>(a.part + pt * a.max_groups * gstride);
  float4* dst4 = reinterpret_cast<float4*>(sm);
  const int n4 = n_groups * (int)(gstride / 4);
  for (int i0 = 0; i0 < n4; i0 += CF::THREADS * 10) {    // 10 loads per thread: 9 groups of heads of 64 in one trip
    float4 v[10];
#pragma unroll
    for (int k = 0; k < 10; ++k) {
      const int i = i0 + k * CF::THREADS + threadIdx.x;
      if (i < n4) v[k] = __ldcg(src4 + i);
    }
#pragma unroll
    for (int k = 0; k < 10; ++k) {
      const int i = i0 + k * CF::THREADS + threadIdx.x;
      if (i < n4) dst4[i] = v[k];
    }
  }
  __syncthreads();
  const float* base = reinterpret_cast<const float*>(sm);
  // per row: common maximum, each group's weight (in group order) and the normaliser
  float* wgt = reinterpret_cast<float*>(sm) + (size_t)n_groups * gstride;      // [16][n_groups + 1]
  // (one warp per row, one lane per group: there are at most 24 groups; the normaliser is summed
  // by shuffles in group order)
  for (int i = warp; i < rows_here; i += NW + 1) {
    const float* pr = base + (size_t)i * (DH + 2);
    const float mc = lane < n_groups ? pr[lane * gstride + DH] : -INFINITY;
    const float lc = lane < n_groups ? pr[lane * gstride + DH + 1] : 0.f;
    const float mm = warp_max(mc);
    const float sc = mc == -INFINITY ? 0.f : exp2f(mc - mm);
    if (lane < n_groups) wgt[i * (n_groups + 1) + lane] = sc;
    float lsum = 0.f;
    for (int ck = 0; ck < n_groups; ++ck)
      lsum = fmaf(__shfl_sync(0xffffffffu, sc, ck), __shfl_sync(0xffffffffu, lc, ck), lsum);
    if (lane == 0) wgt[i * (n_groups + 1) + n_groups] = lsum;
  }
  __syncthreads();
  for (int e = threadIdx.x; e < rows_here * (DH / 2); e += CF::THREADS) {     // two neighbouring columns per thread
    const int i = e / (DH / 2), c = 2 * (e - i * (DH / 2));
    const float* pr = base + (size_t)i * (DH + 2) + c;
    const float* wr = wgt + i * (n_groups + 1);
    float acc0 = 0.f, acc1 = 0.f;
#pragma unroll 4
    for (int ck = 0; ck < n_groups; ++ck) {                                     // group order
      const float2 v = *reinterpret_cast<const float2*>(pr + ck * gstride);
      acc0 += wr[ck] * v.x;
      acc1 += wr[ck] * v.y;
    }
    const int idx = mt * 16 + i;
    const int r = group == 1 ? idx : idx / group, gh = idx - r * group;
    const size_t orow = a.out_row_stride > 0 ? (size_t)r * a.out_row_stride + b : (size_t)(b * m_rows + r);
    const size_t at = (orow * 2 * dm.H + hk * group + gh) * DH + c;
    const float o0 = acc0 / wr[n_groups], o1 = acc1 / wr[n_groups];
    const __nv_bfloat162 hi = __floats2bfloat162_rn(o0, o1);
    *reinterpret_cast<__nv_bfloat162*>(a.out + at) = hi;
    *reinterpret_cast<__nv_bfloat162*>(a.out + at + dm.H * DH) =
        __floats2bfloat162_rn(o0 - __bfloat162float(hi.x), o1 - __bfloat162float(hi.y));
  }
  if (threadIdx.x == 0) a.ticket[pt] = 0;
}
