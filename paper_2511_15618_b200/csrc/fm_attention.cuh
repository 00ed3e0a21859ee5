// Few-row causal attention over one level's KV cache (Sec. 3.3: the candidates of a pass are
// masked causally among themselves; conditioning enters as prefix keys visible to every row).
#pragma once
#include "fm_common.cuh"

// One CTA per (row, head).  Keys visible to the row at level position p: prefix slots [0,P) and
// positions max(0, p-W+1) .. p at slot P + pos % cap.  Each warp takes key blocks of 32 in a
// fixed round-robin; lane j scores key j of the block, then the block's probabilities are
// broadcast while each lane accumulates its own dh/32 output dims.  The four warps' partial
// (max, sum, acc) are merged in warp order, so a row's result does not depend on how many other
// rows the launch holds.
template <int DH>
__global__ void __launch_bounds__(128) attn_rows_kernel(Dims dm, SeqState st, int batch, int level,
                                                         const float* __restrict__ q /*[rows,H*dh]*/,
                                                         const bf16* __restrict__ Kc, const bf16* __restrict__ Vc,
                                                         bf16* __restrict__ out /*[rows,H*dh]*/) {
  constexpr int PER = DH / 32;                     // output dims per lane
  const int row = blockIdx.x, h = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int b, p;
  const bool valid = fm_row_map(dm, st, batch, level, row, b, p);
  bf16* orow = out + (size_t)row * dm.H * DH + h * DH;
  if (!valid) {
    for (int i = threadIdx.x; i < DH; i += blockDim.x) orow[i] = __float2bfloat16(0.f);
    return;
  }
  __shared__ float qs[DH];
  __shared__ float part_m[4], part_l[4], part_acc[4][DH];
  const float scale = rsqrtf((float)DH);
  for (int i = threadIdx.x; i < DH; i += blockDim.x) qs[i] = q[(size_t)row * dm.H * DH + h * DH + i] * scale;
  __syncthreads();

  const int hk = (h * dm.Hkv) / dm.H;
  const int slots = dm.P + dm.cap[level], cap = dm.cap[level], W = dm.window[level];
  const bf16* Kb = Kc + ((size_t)b * dm.Hkv + hk) * slots * DH;
  const bf16* Vb = Vc + ((size_t)b * dm.Hkv + hk) * slots * DH;
  const int lo = W > 0 ? max(0, p - W + 1) : 0;
  const int nkeys = dm.P + (p - lo + 1);

  float m = -INFINITY, l = 0.f, acc[PER];
#pragma unroll
  for (int i = 0; i < PER; ++i) acc[i] = 0.f;

  for (int k0 = warp * 32; k0 < nkeys; k0 += 128) {
    const int t = k0 + lane;
    int slot = 0;
    float s = -INFINITY;
    if (t < nkeys) {
      slot = t < dm.P ? t : dm.P + ((lo + t - dm.P) % cap);
      const uint4* kr = reinterpret_cast<const uint4*>(Kb + (size_t)slot * DH);
      float dot = 0.f;
#pragma unroll
      for (int c = 0; c < DH / 8; ++c) {
        const uint4 u = kr[c];
        const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 f = __bfloat1622float2(h2[e]);
          dot = fmaf(qs[c * 8 + 2 * e], f.x, dot);
          dot = fmaf(qs[c * 8 + 2 * e + 1], f.y, dot);
        }
      }
      s = dot;
    }
    const float bm = warp_max(s);
    const float mn = fmaxf(m, bm);
    const float corr = __expf(m - mn);               // 0 when m = -inf
    const float pj = t < nkeys ? __expf(s - mn) : 0.f;
    l = l * corr + warp_sum(pj);
#pragma unroll
    for (int i = 0; i < PER; ++i) acc[i] *= corr;
    m = mn;
    const int cnt = min(32, nkeys - k0);
    for (int jj = 0; jj < cnt; ++jj) {
      const float pp = __shfl_sync(0xffffffffu, pj, jj);
      const int sl = __shfl_sync(0xffffffffu, slot, jj);
      const bf16* vr = Vb + (size_t)sl * DH + lane * PER;
#pragma unroll
      for (int i = 0; i < PER; ++i) acc[i] = fmaf(pp, __bfloat162float(vr[i]), acc[i]);
    }
  }
  if (lane == 0) { part_m[warp] = m; part_l[warp] = l; }
#pragma unroll
  for (int i = 0; i < PER; ++i) part_acc[warp][lane * PER + i] = acc[i];
  __syncthreads();
  float M = part_m[0];
  for (int w = 1; w < 4; ++w) M = fmaxf(M, part_m[w]);
  float Lsum = 0.f;
  for (int w = 0; w < 4; ++w) Lsum += part_l[w] * __expf(part_m[w] - M);
  for (int i = threadIdx.x; i < DH; i += blockDim.x) {
    float a = 0.f;
    for (int w = 0; w < 4; ++w) a += part_acc[w][i] * __expf(part_m[w] - M);
    orow[i] = __float2bfloat16(a / Lsum);
  }
}
