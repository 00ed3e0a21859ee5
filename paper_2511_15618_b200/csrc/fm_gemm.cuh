// Row-wise consumers of the split-K partial tiles written by the tensor-core GEMM:
// part[z][row][m], z < nsplit, summed in split order (a fixed order).
#pragma once
#include "fm_common.cuh"

struct PartView {
  const float* part;      // null: nothing pending
  int nsplit;
  long long split_stride; // elements between splits
  int ldm;                // elements between rows
};

// loads are issued eight at a time (independent), the additions stay in split order
__device__ inline float part_sum(const PartView& pv, int row, int m) {
  const float* p = pv.part + (size_t)row * pv.ldm + m;
  float v = 0.f;
  int z = 0;
  for (; z + 8 <= pv.nsplit; z += 8) {
    float t[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) t[u] = __ldcg(p + (size_t)(z + u) * pv.split_stride);
#pragma unroll
    for (int u = 0; u < 8; ++u) v += t[u];
  }
  float t[8];
#pragma unroll
  for (int u = 0; u < 8; ++u) t[u] = (z + u < pv.nsplit) ? __ldcg(p + (size_t)(z + u) * pv.split_stride) : 0.f;
#pragma unroll
  for (int u = 0; u < 8; ++u) if (z + u < pv.nsplit) v += t[u];
  return v;
}

__device__ inline float gelu_erf(float x) { return 0.5f * x * (1.f + erff(x * 0.70710678118654752f)); }

enum FoldMode { FOLD_F32 = 0, FOLD_BF16 = 1, FOLD_GELU_BF16 = 2 };

// out[row][m] = f(sum of partials); grid (rows, ceil(M / 256)), block 256
template <int MODE>
__global__ void fold_kernel(PartView pv, void* __restrict__ out, int ldo, int M) {
  const int row = blockIdx.x;
  for (int m = blockIdx.y * blockDim.x + threadIdx.x; m < M; m += gridDim.y * blockDim.x) {
    const float v = part_sum(pv, row, m);
    if (MODE == FOLD_F32) reinterpret_cast<float*>(out)[(size_t)row * ldo + m] = v;
    else if (MODE == FOLD_BF16) reinterpret_cast<bf16*>(out)[(size_t)row * ldo + m] = __float2bfloat16(v);
    else reinterpret_cast<bf16*>(out)[(size_t)row * ldo + m] = __float2bfloat16(gelu_erf(v));
  }
}
