// Skinny weight-streaming GEMM: out[r, m] = sum_k A[r, k] * W[m, k]  (bf16 operands, fp32 sums).
#pragma once
#include "fm_common.cuh"

enum GemmMode { GEMM_STORE_F32 = 0, GEMM_ADD_F32 = 1, GEMM_GELU_BF16 = 2, GEMM_STORE_BF16 = 3 };

struct GemmArgs {
  const bf16* W;      // [M(pad), K] row-major
  const bf16* A;      // [R, K] row-major
  void* out;          // [R, ldo] fp32 or bf16
  int M, K, R, ldo;
  long long strideW, strideA, strideO;   // per blockIdx.z (elements)
  const int* n_active;                   // skip all work when *n_active == 0 (may be null)
};

__device__ inline float gelu_erf(float x) { return 0.5f * x * (1.f + erff(x * 0.70710678118654752f)); }

template <int MODE>
__device__ inline void gemm_store(void* out, size_t idx, float v) {
  if (MODE == GEMM_STORE_F32) reinterpret_cast<float*>(out)[idx] = v;
  else if (MODE == GEMM_ADD_F32) reinterpret_cast<float*>(out)[idx] += v;
  else if (MODE == GEMM_GELU_BF16) reinterpret_cast<bf16*>(out)[idx] = __float2bfloat16(gelu_erf(v));
  else reinterpret_cast<bf16*>(out)[idx] = __float2bfloat16(v);
}

// CUDA-core version: one warp per output feature, a tile of 16 rows, lanes stride over K in
// 16-byte pieces; the warp sum has a fixed shuffle order, so results do not depend on R.
template <int MODE>
__global__ void __launch_bounds__(128) gemm_simt_kernel(GemmArgs g) {
  if (g.n_active != nullptr && *g.n_active == 0) return;
  constexpr int TR = 16;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m = blockIdx.x * 4 + warp;
  const int r0 = blockIdx.y * TR;
  if (m >= g.M) return;
  const bf16* W = g.W + blockIdx.z * g.strideW + (size_t)m * g.K;
  const bf16* A = g.A + blockIdx.z * g.strideA;
  float acc[TR];
#pragma unroll
  for (int r = 0; r < TR; ++r) acc[r] = 0.f;
  const int nr = min(TR, g.R - r0);
  for (int k = lane * 8; k < g.K; k += 256) {
    const uint4 wu = *reinterpret_cast<const uint4*>(W + k);
    const __nv_bfloat162* w2 = reinterpret_cast<const __nv_bfloat162*>(&wu);
    float wf[8];
#pragma unroll
    for (int e = 0; e < 4; ++e) { const float2 f = __bfloat1622float2(w2[e]); wf[2 * e] = f.x; wf[2 * e + 1] = f.y; }
#pragma unroll
    for (int r = 0; r < TR; ++r) {
      if (r < nr) {
        const uint4 au = *reinterpret_cast<const uint4*>(A + (size_t)(r0 + r) * g.K + k);
        const __nv_bfloat162* a2 = reinterpret_cast<const __nv_bfloat162*>(&au);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 f = __bfloat1622float2(a2[e]);
          acc[r] = fmaf(wf[2 * e], f.x, acc[r]);
          acc[r] = fmaf(wf[2 * e + 1], f.y, acc[r]);
        }
      }
    }
  }
#pragma unroll
  for (int r = 0; r < TR; ++r) {
    const float v = warp_sum(acc[r]);
    if (lane == 0 && r < nr) gemm_store<MODE>(g.out, blockIdx.z * g.strideO + (size_t)(r0 + r) * g.ldo + m, v);
  }
}
