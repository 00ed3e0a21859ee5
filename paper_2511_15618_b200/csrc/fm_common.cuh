// Shared definitions of the device code: dimensions, per-sequence state, row maps.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

typedef __nv_bfloat16 bf16;

// Ring sizes (entries per sequence) of the hourglass carry state, indexed by level-local
// position modulo the size.  A verify pass touches coordinate positions L-2 .. L+D, vertices
// ceil(L/3)-2 .. floor((L+D)/3) and faces ceil(L/9)-1 .. floor((L+D)/9); with D <= 27 these
// spans are at most 30, 12 and 5 entries.
constexpr int FM_RING_C = 32;
constexpr int FM_RING_V = 16;
constexpr int FM_RING_F = 8;
constexpr int FM_HIST = 32;             // the correction stage looks back at most two faces (18 tokens)

struct Dims {
  int d, H, Hkv, dh, dff;
  int n_bins, V, Vpad, P;
  int D, R1, mv, mf;          // drafts, rows per sequence at the three levels
  int window[3];
  int cap[3];                 // cache slots per level behind the prefix
  int max_batch, max_tokens;
  int allow_eos;
  float eps, theta;
  int Ef, NH;                 // face heads, total draft heads (nc + nv + Ef)
  int nc, nv;                 // coordinate heads (2, or D when only the coordinate level drafts), vertex heads (2 or 0)
  int full, avg, hf;          // full SP / HF blocks, averaged merge of the levels, width of the HF feed-forward
  int has_label;              // a label head was given
};

// Per-sequence decoding state, all int32 arrays of max_batch entries in device memory.
struct SeqState {
  int* L;          // inputs consumed (coordinate KV length behind the prefix)
  int* nrow;       // rows the next / current forward pass feeds (0 = inactive)
  int* main_tok;   // pending main token t_{L-1}
  int* done;
  int* t_end;      // index one past the last mesh token to emit
  int* plen;       // prompt length in tokens
  int* cand;       // [max_batch, R1] inputs of the current pass
  int* o;          // [max_batch, R1] masked argmax per row
  float* margin;   // [max_batch, R1]
  int* status;     // device status word
  int* n_active;   // sequences with nrow > 0 in the current pass
  int* step;       // passes executed by fm_generate (schedule index)
  int* hist;       // [max_batch, FM_HIST] accepted mesh tokens, token t_i at entry i mod FM_HIST
};

__host__ __device__ inline int fm_ratio(int level) { return level == 0 ? 1 : (level == 1 ? 3 : 9); }
__host__ __device__ inline int fm_ring(int level) { return level == 0 ? FM_RING_C : (level == 1 ? FM_RING_V : FM_RING_F); }
__host__ __device__ inline int fm_rows_per_seq(const Dims& dm, int level) {
  return level == 0 ? dm.R1 : (level == 1 ? dm.mv : dm.mf);
}

// Row `row` of a level's activation matrix -> (sequence b, level-local position p).
// Level rows of a pass are the multiples of ratio in [L, L+nrow-1]: p = ceil(L/ratio) + k.
__device__ inline bool fm_row_map(const Dims& dm, const SeqState& st, int batch, int level, int row, int& b, int& p) {
  const int m = fm_rows_per_seq(dm, level);
  b = row / m;
  const int k = row - b * m;
  p = 0;
  if (b >= batch) return false;
  const int n = st.nrow[b];
  if (n <= 0) return false;
  const int Lb = st.L[b];
  const int ratio = fm_ratio(level);
  p = (Lb + ratio - 1) / ratio + k;
  return ratio * p <= Lb + n - 1;
}

__device__ inline float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ inline float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
