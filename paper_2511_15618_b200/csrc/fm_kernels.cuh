// Element-wise, row-wise and bookkeeping kernels of the decode step.
#pragma once
#include "fm_common.cuh"
#include "fm_ptx.cuh"

// ------------------------------------------------------------------------------------------
// block reductions (blockDim.x multiple of 32, <= 1024)
// ------------------------------------------------------------------------------------------
__device__ inline float block_sum(float v, float* sh) {
  v = warp_sum(v);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = blockDim.x >> 5;
  __syncthreads();
  if (l == 0) sh[w] = v;
  __syncthreads();
  float t = 0.f;
  for (int i = 0; i < nw; ++i) t += sh[i];          // fixed order: same result in every thread
  return t;
}

__device__ inline float block_max(float v, float* sh) {
  v = warp_max(v);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = blockDim.x >> 5;
  __syncthreads();
  if (l == 0) sh[w] = v;
  __syncthreads();
  float t = -INFINITY;
  for (int i = 0; i < nw; ++i) t = fmaxf(t, sh[i]);
  return t;
}

// ------------------------------------------------------------------------------------------
// A GEMM operand value as two bfloat16 terms: hi = bf16(v) at p[0], lo = bf16(v - hi) at p[lo_off].
__device__ inline void store_hi_lo(bf16* p, float v, int lo_off) {
  const bf16 hi = __float2bfloat16(v);
  p[0] = hi;
  p[lo_off] = __float2bfloat16(__fsub_rn(v, __bfloat162float(hi)));   // never fused with a product behind v
}

// Hand a freshly written residual row to the first layer of a stack: the GEMM operand row
// x * g as [hi | lo] terms, row length 2d (the RMSNorm scale 1/rms is applied by the GEMM's
// epilogue) and the row's sum of squares in slot 0 of `ssq` (the consumer is told that one slot is
// filled).
// ------------------------------------------------------------------------------------------
__device__ inline void stack_entry_row(const float* xr, int row, int d, const float* __restrict__ g,
                                       bf16* __restrict__ a_out, float* __restrict__ ssq) {
  __shared__ float sh[32];
  float ss = 0.f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    const float v = xr[i];
    ss += v * v;
    store_hi_lo(a_out + (size_t)row * 2 * d + i, __fmul_rn(v, g[i]), d);
  }
  ss = block_sum(ss, sh);
  if (threadIdx.x == 0) ssq[row] = ss;
}

// first level-local position of sequence b in this pass
__device__ inline int fm_first_pos(const SeqState& st, int b, int level) {
  const int r = fm_ratio(level);
  return (st.L[b] + r - 1) / r;
}

// ------------------------------------------------------------------------------------------
// a1. candidate embedding: x[row] = E[cand[b][j]]  (zeros for rows that are not fed)
// ------------------------------------------------------------------------------------------
__global__ void embed_kernel(Dims dm, SeqState st, int batch, const bf16* __restrict__ E, float* __restrict__ x,
                             const float* __restrict__ g, bf16* __restrict__ a_out, float* __restrict__ ssq,
                             int rows, const float* __restrict__ hc_ring, const float* __restrict__ hv_ring,
                             bf16* __restrict__ cat_v, bf16* __restrict__ cat_f, int rows_v, int rows_f) {
  if ((int)blockIdx.x >= rows) {
    // Blocks behind the coordinate rows prepare the operand rows of the two shorten GEMMs (used when
    // the gather is fused into the producing GEMM's epilogue): part k of parent row u pools position
    // 3u - 2 + k of the level below; what lies before this pass comes from the carry ring (zeros
    // below position 0 and for rows that are not fed), the rest is written by the epilogue of the
    // last layer below.
    int j = (int)blockIdx.x - rows;
    const int level_out = j < 3 * rows_v ? 1 : 2;
    if (level_out == 2) j -= 3 * rows_v;
    if (cat_v == nullptr || j >= 3 * (level_out == 1 ? rows_v : rows_f)) return;
    const int row = j / 3, part = j - 3 * row, lb = level_out - 1, rs = fm_ring(lb), d = dm.d;
    int b, u;
    const bool valid = fm_row_map(dm, st, batch, level_out, row, b, u);
    const int pos = 3 * u - 2 + part, p0 = valid ? fm_first_pos(st, b, lb) : 0;
    if (valid && pos >= p0) return;                  // a hidden of this pass
    const bool ok = valid && pos >= 0;
    const float* src = (lb == 0 ? hc_ring : hv_ring) + ((size_t)b * rs + ((pos + rs) % rs)) * d;
    bf16* out = (level_out == 1 ? cat_v : cat_f) + (size_t)row * 6 * d + part * d;
    for (int i = threadIdx.x; i < d; i += blockDim.x) store_hi_lo(out + i, ok ? src[i] : 0.f, 3 * d);
    return;
  }
  const int row = blockIdx.x;
  int b, p;
  const bool valid = fm_row_map(dm, st, batch, 0, row, b, p);
  int tok = 0;
  if (valid) {
    tok = st.cand[b * dm.R1 + (row - b * dm.R1)];
    if (tok < 0 || tok >= dm.V) {                    // never index outside the table
      if (threadIdx.x == 0) atomicExch(st.status, -1);
      tok = dm.n_bins + 2;
    }
  }
  for (int i = threadIdx.x; i < dm.d; i += blockDim.x)
    x[(size_t)row * dm.d + i] = valid ? __bfloat162float(E[(size_t)tok * dm.d + i]) : 0.f;
  __syncthreads();
  stack_entry_row(x + (size_t)row * dm.d, row, dm.d, g, a_out, ssq);
}

// RMSNorm of read-only fp32 rows (conditioning vectors, draft features) -> bf16 operand rows
__global__ void rmsnorm_kernel(const float* __restrict__ x, const float* __restrict__ g, bf16* __restrict__ out,
                               int d, float eps) {
  ptx::grid_dep_launch();
  ptx::grid_dep_wait();
  __shared__ float sh[32];
  const float* xr = x + (size_t)blockIdx.x * d;
  float ss = 0.f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) { const float v = xr[i]; ss += v * v; }
  ss = block_sum(ss, sh);
  const float inv = rsqrtf(ss / (float)d + eps);
  for (int i = threadIdx.x; i < d; i += blockDim.x)
    out[(size_t)blockIdx.x * d + i] = __float2bfloat16(xr[i] * inv * g[i]);
}

// ------------------------------------------------------------------------------------------
// RoPE table: (cos, sin) of pos * theta^(-2i/dh) for every level-local position, evaluated in
// double precision when the context is created (the rotation itself is in the QKV epilogue).
// ------------------------------------------------------------------------------------------
__global__ void rope_table_kernel(float2* __restrict__ tab, const double* __restrict__ inv_freq, int n_pos, int half) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (size_t)n_pos * half) return;
  const int pos = (int)(i / half), k = (int)(i - (size_t)pos * half);
  double s, c;
  sincos((double)pos * inv_freq[k], &s, &c);
  tab[i] = make_float2((float)c, (float)s);
}

// prefix keys/values of one layer: kv fp32 [rows, 2*Hkv*dh] (rows = chunk of b*P+j) -> slots [0,P)
__global__ void prefix_store_kernel(Dims dm, int level, int row0, const float* __restrict__ kv,
                                    bf16* __restrict__ Kc, bf16* __restrict__ Vc) {
  const int r = row0 + blockIdx.x;
  const int b = r / dm.P, j = r - b * dm.P;
  const int slots = dm.P + dm.cap[level];
  const int n = dm.Hkv * dm.dh;
  const float* src = kv + (size_t)blockIdx.x * 2 * n;
  for (int t = threadIdx.x; t < n; t += blockDim.x) {
    const int hk = t / dm.dh, i = t - hk * dm.dh;
    const size_t o = (((size_t)b * dm.Hkv + hk) * slots + j) * dm.dh + i;
    Kc[o] = __float2bfloat16(src[t]);
    Vc[o] = __float2bfloat16(src[n + t]);
  }
}

// ------------------------------------------------------------------------------------------
// hourglass carry rings
// ------------------------------------------------------------------------------------------

// a3/a5 shorten, gather half, fused with the ring store of the level below.  Blocks [0, rows_out):
// row v of level `level_out` <- [h_{3v-2}; h_{3v-1}; h_{3v}] (zeros for negative positions and for
// rows that are not fed) as [hi | lo] terms, row length 6d; a hidden of this pass is read from
// x_below, an older one from the carry ring.  Blocks [rows_out, rows_out + rows_below): this pass's
// hiddens of the level below go into its ring for later passes.
__global__ void shorten_gather_kernel(Dims dm, SeqState st, int batch, int level_out, const float* __restrict__ x_below,
                                      float* __restrict__ ring, bf16* __restrict__ out, int rows_out) {
  ptx::grid_dep_launch();
  ptx::grid_dep_wait();
  const int lb = level_out - 1, rs = fm_ring(lb), d = dm.d;
  if ((int)blockIdx.x >= rows_out) {
    if (blockIdx.y != 0) return;
    const int row = blockIdx.x - rows_out;
    int b, p;
    if (!fm_row_map(dm, st, batch, lb, row, b, p)) return;
    float* dst = ring + ((size_t)b * rs + (p % rs)) * d;
    const float* src = x_below + (size_t)row * d;
    for (int i = threadIdx.x; i < d; i += blockDim.x) dst[i] = src[i];
    return;
  }
  const int row = blockIdx.x;
  int b, v;
  const bool valid = fm_row_map(dm, st, batch, level_out, row, b, v);
  const int p0 = valid ? fm_first_pos(st, b, lb) : 0, m_below = fm_rows_per_seq(dm, lb);
  {
    const int part = blockIdx.y;                     // grid.y = 3: one of the three concatenated hiddens
    const int pos = 3 * v - 2 + part;
    const bool ok = valid && pos >= 0;
    const float* src = (ok && pos >= p0) ? x_below + ((size_t)b * m_below + (pos - p0)) * d
                                         : ring + ((size_t)b * rs + ((pos + rs) % rs)) * d;
    for (int i = threadIdx.x; i < d; i += blockDim.x)
      store_hi_lo(out + (size_t)row * 6 * d + part * d + i, ok ? src[i] : 0.f, 3 * d);
  }
}

// a7/a9 upsample, residual half, fused with the ring store of the upsampled triples.  Blocks
// [0, rows): x[row] = h[b][p] + tri[b][p/3][(p%3)*d ...], where h is the pre-shorten hidden of the
// position (kept in the carry ring by the shorten step of this pass) and the triple comes from
// `tri_new` if its parent row belongs to this pass, else from the ring; the row is then handed to
// the first layer of the stack above (operand row and sum of squares).  Blocks [rows, rows +
// rows_up): this pass's triples go into the ring.
__global__ void upsample_add_kernel(Dims dm, SeqState st, int batch, int level, const float* __restrict__ h_ring,
                                    const float* __restrict__ tri_new, float* __restrict__ tri_ring, float* __restrict__ x,
                                    const float* __restrict__ g, bf16* __restrict__ a_out, float* __restrict__ ssq, int rows) {
  ptx::grid_dep_launch();
  ptx::grid_dep_wait();
  const int rs = fm_ring(level), rsu = fm_ring(level + 1), d = dm.d;
  if ((int)blockIdx.x >= rows) {
    const int row = blockIdx.x - rows;
    int b, p;
    if (!fm_row_map(dm, st, batch, level + 1, row, b, p)) return;
    float* dst = tri_ring + ((size_t)b * rsu + (p % rsu)) * 3 * d;
    const float* src = tri_new + (size_t)row * 3 * d;
    for (int i = threadIdx.x; i < 3 * d; i += blockDim.x) dst[i] = src[i];
    return;
  }
  const int row = blockIdx.x;
  int b, p;
  const bool valid = fm_row_map(dm, st, batch, level, row, b, p);
  const float* h = h_ring + ((size_t)b * rs + (p % rs)) * d;
  const int up = p / 3, p0u = valid ? fm_first_pos(st, b, level + 1) : 0;
  const float* t = (valid && up >= p0u) ? tri_new + ((size_t)b * fm_rows_per_seq(dm, level + 1) + (up - p0u)) * 3 * d + (p % 3) * d
                                        : tri_ring + ((size_t)b * rsu + (up % rsu)) * 3 * d + (p % 3) * d;
  for (int i = threadIdx.x; i < d; i += blockDim.x) x[(size_t)row * d + i] = valid ? h[i] + t[i] : 0.f;
  __syncthreads();
  stack_entry_row(x + (size_t)row * d, row, d, g, a_out, ssq);
}

// ------------------------------------------------------------------------------------------
// a11. masked top-2 of the logits rows: ids >= n_bins forbidden, except EOS where a face
// starts (target index % 9 == 0) when allowed; ties go to the lowest id.
// ------------------------------------------------------------------------------------------
struct Top2 { float v1; int i1; float v2; };
__device__ inline void top2_push(Top2& t, float v, int i) {
  if (v > t.v1 || (v == t.v1 && i < t.i1)) { t.v2 = t.v1; t.v1 = v; t.i1 = i; }
  else if (v > t.v2) t.v2 = v;
}
__device__ inline void top2_merge(Top2& a, const Top2& b) {
  if (b.i1 < 0) return;
  if (a.i1 < 0) { a = b; return; }
  if (b.v1 > a.v1 || (b.v1 == a.v1 && b.i1 < a.i1)) { const float lose = a.v1; a.v1 = b.v1; a.i1 = b.i1; a.v2 = fmaxf(fmaxf(a.v2, b.v2), lose); }
  else a.v2 = fmaxf(fmaxf(a.v2, b.v2), b.v1);
}
__device__ inline Top2 block_top2(const float* __restrict__ z, const Dims& dm, int target_index) {
  Top2 t{-INFINITY, -1, -INFINITY};
  const bool eos_ok = dm.allow_eos && (target_index % 9 == 0);
  const int n = dm.n_bins + (eos_ok ? 2 : 0);
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    if (i == dm.n_bins) continue;                    // BOS
    top2_push(t, z[i], i);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    Top2 u;
    u.v1 = __shfl_xor_sync(0xffffffffu, t.v1, o);
    u.i1 = __shfl_xor_sync(0xffffffffu, t.i1, o);
    u.v2 = __shfl_xor_sync(0xffffffffu, t.v2, o);
    top2_merge(t, u);
  }
  __shared__ Top2 sh[32];
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = blockDim.x >> 5;
  __syncthreads();
  if (l == 0) sh[w] = t;
  __syncthreads();
  Top2 r = sh[0];
  for (int i = 1; i < nw; ++i) top2_merge(r, sh[i]);
  return r;
}

__global__ void verify_top2_kernel(Dims dm, SeqState st, int batch, const float* __restrict__ logits,
                                   float* __restrict__ logits_out) {
  ptx::grid_dep_launch();
  ptx::grid_dep_wait();
  const int row = blockIdx.x;
  int b, p;
  const bool valid = fm_row_map(dm, st, batch, 0, row, b, p);
  const int j = row % dm.R1;
  const int bb = row / dm.R1;
  if (bb >= batch) return;
  if (logits_out != nullptr)
    for (int i = threadIdx.x; i < dm.V; i += blockDim.x)
      logits_out[(size_t)row * dm.V + i] = valid ? logits[(size_t)row * dm.Vpad + i] : 0.f;
  if (!valid) {
    if (threadIdx.x == 0) { st.o[bb * dm.R1 + j] = -1; st.margin[bb * dm.R1 + j] = 0.f; }
    return;
  }
  const Top2 t = block_top2(logits + (size_t)row * dm.Vpad, dm, p);
  if (threadIdx.x == 0) { st.o[b * dm.R1 + j] = t.i1; st.margin[b * dm.R1 + j] = t.v1 - t.v2; }
}

// ------------------------------------------------------------------------------------------
// a12. acceptance + rollback: one warp per sequence.
// ------------------------------------------------------------------------------------------
struct GenOut {            // where fm_generate collects tokens (device-resident parameter block)
  int* out_tok; int out_stride; int* out_len;
  const int* truth; int truth_stride; const int* keep; int n_sched;
  int plain;
  long long* stats;        // [0] steps, [1] emitted, [2..] accept histogram
  volatile int* host_done; // mapped pinned flag: number of unfinished sequences
};

__device__ inline void accept_one(const Dims& dm, const SeqState& st, int b, int lane, const int* __restrict__ force_len,
                                  const int* __restrict__ force_tok, int* __restrict__ n_acc, int* __restrict__ emitted,
                                  int* __restrict__ kv_len, const GenOut* __restrict__ gen) {
  const int R1 = dm.R1, eos = dm.n_bins + 1;
  const int rows = st.nrow[b];
  int a = 0;
  int L = st.L[b];
  const int* o = (force_tok != nullptr ? force_tok : st.o) + b * R1;
  const int cand = lane < R1 ? st.cand[b * R1 + lane] : -1;
  if (rows > 0 && !st.done[b]) {
    // lane j holds candidate j; it matches if it is the main token or equals the argmax at row j-1
    const bool match = lane < rows && (lane == 0 || cand == o[lane - 1]);
    const unsigned mm = __ballot_sync(0xffffffffu, match);
    a = __ffs(~mm) - 1;                              // length of the leading run of matches
    if (gen != nullptr && gen->plain) a = 1;
    if (force_len != nullptr) a = force_len[b];
    a = max(1, min(a, rows));
    const unsigned em = __ballot_sync(0xffffffffu, lane < a && cand == eos);
    bool fin = false;
    if (em) { a = __ffs(em); fin = true; }           // an accepted EOS ends the sequence
    if (lane < a) st.hist[b * FM_HIST + ((L - 1 + lane) & (FM_HIST - 1))] = cand;   // accepted token t_{L-1+lane}
    L += a;
    if (L - 1 >= st.t_end[b]) fin = true;
    if (gen != nullptr && gen->out_tok != nullptr && lane < a) {
      const int at = gen->out_len[b] + lane;
      if (at < gen->out_stride) gen->out_tok[(size_t)b * gen->out_stride + at] = cand;
    }
    __syncwarp();
    if (lane == 0) {
      st.L[b] = L;
      st.main_tok[b] = o[a - 1];
      st.done[b] = fin ? 1 : 0;
      st.nrow[b] = fin ? 0 : min(R1, st.t_end[b] - (L - 1));
      if (gen != nullptr) {
        if (gen->out_len != nullptr) gen->out_len[b] += a;
        if (gen->stats != nullptr) {
          atomicAdd((unsigned long long*)&gen->stats[1], (unsigned long long)a);
          atomicAdd((unsigned long long*)&gen->stats[2 + a], 1ull);
        }
      }
    }
  } else if (lane == 0) {
    st.nrow[b] = 0;
  }
  if (n_acc != nullptr && lane == 0) n_acc[b] = a;
  if (emitted != nullptr && lane < R1) emitted[b * R1 + lane] = lane < a ? cand : -1;
  if (kv_len != nullptr && lane == 0) {
    kv_len[b * 3 + 0] = L; kv_len[b * 3 + 1] = (L + 2) / 3; kv_len[b * 3 + 2] = (L + 8) / 9;
  }
}

// rows fed at each level in the next pass (n_active[level]); n_active[3] = unfinished sequences
__device__ inline void count_rows(const Dims& dm, const SeqState& st, int batch) {
  int cnt[3] = {0, 0, 0}, act = 0;
  for (int b = 0; b < batch; ++b) {
    const int n = st.nrow[b], L = st.L[b];
    if (n <= 0) continue;
    act++;
    for (int l = 0; l < 3; ++l) {
      const int r = fm_ratio(l);
      cnt[l] += (L + n - 1) / r - (L + r - 1) / r + 1;
    }
  }
  st.n_active[0] = cnt[0]; st.n_active[1] = cnt[1]; st.n_active[2] = cnt[2]; st.n_active[3] = act;
}

// One block; its warps walk over the sequences.  Afterwards thread 0 counts the rows of the next
// pass and, inside fm_generate (step_end != 0), bumps the pass counter and tells the host how many
// sequences are still running.
__global__ void accept_kernel(Dims dm, SeqState st, int batch, const int* __restrict__ force_len,
                              const int* __restrict__ force_tok, int* __restrict__ n_acc, int* __restrict__ emitted,
                              int* __restrict__ kv_len, const GenOut* __restrict__ gen, int step_end) {
  const int lane = threadIdx.x & 31;
  for (int b = threadIdx.x >> 5; b < batch; b += blockDim.x >> 5) accept_one(dm, st, b, lane, force_len, force_tok, n_acc, emitted, kv_len, gen);
  __syncthreads();
  if (threadIdx.x != 0) return;
  count_rows(dm, st, batch);
  if (step_end) {
    *st.step += 1;
    if (gen->stats != nullptr) gen->stats[0] += 1;
    if (gen->host_done != nullptr) { *gen->host_done = st.n_active[3]; __threadfence_system(); }
  }
}
// ------------------------------------------------------------------------------------------
// prefill helpers
// ------------------------------------------------------------------------------------------
// next chunk of BOS + prompt: cand[b][j] = u_{L+j}, nrow = min(R1, inputs left)
__global__ void prefill_feed_kernel(Dims dm, SeqState st, int batch, const int* __restrict__ prompt,
                                    const int* __restrict__ prompt_off) {
  const int b = blockIdx.x;
  if (b >= batch) return;
  const int L = st.L[b], total = 1 + st.plen[b];
  const int n = max(0, min(dm.R1, total - L));
  for (int j = threadIdx.x; j < dm.R1; j += blockDim.x) {
    const int pos = L + j;
    int tok = dm.n_bins + 2;
    if (j < n) tok = pos == 0 ? dm.n_bins : prompt[prompt_off[b] + pos - 1];
    st.cand[b * dm.R1 + j] = tok;
    if (j < n && pos >= 1) st.hist[b * FM_HIST + ((pos - 1) & (FM_HIST - 1))] = tok;            // input u_pos is mesh token t_{pos-1}
  }
  if (threadIdx.x == 0) st.nrow[b] = n;
}

// all fed rows are accepted; when the prompt is used up the argmax of the last row is the main token
__global__ void prefill_advance_kernel(Dims dm, SeqState st, int batch) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= batch) return;
  const int n = st.nrow[b];
  if (n <= 0) return;
  const int L = st.L[b] + n;
  st.L[b] = L;
  if (L == 1 + st.plen[b]) st.main_tok[b] = st.o[b * dm.R1 + n - 1];
}

// set the rows of the first verify pass (and after fm_set_max_faces)
__global__ void arm_kernel(Dims dm, SeqState st, int batch) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b < batch) {
    const int L = st.L[b];
    const bool fin = st.done[b] || (L - 1 >= st.t_end[b]);
    st.done[b] = fin ? 1 : 0;
    st.nrow[b] = fin ? 0 : min(dm.R1, st.t_end[b] - (L - 1));
  }
}

// ------------------------------------------------------------------------------------------
// a13. draft heads
// ------------------------------------------------------------------------------------------
// Split-node hidden that head h of sequence b reads.  Head index h: [0, nc) coordinate heads,
// [nc, nc + nv) vertex heads, the rest face heads.
__device__ inline const float* head_split_node(const Dims& dm, int h, int b, int n, const float* zc, const float* zv, const float* zf) {
  return h < dm.nc ? zc + ((size_t)b * FM_RING_C + n % FM_RING_C) * dm.d
       : h < dm.nc + dm.nv ? zv + ((size_t)b * FM_RING_V + (n / 3) % FM_RING_V) * dm.d
                           : zf + ((size_t)b * FM_RING_F + (n / 9) % FM_RING_F) * dm.d;
}

// Head inputs.  Row (h, b): a[h][b] = bf16(rms(z) * g_h) with z the stashed split-node hidden of
// the pending position.
__global__ void draft_prep_kernel(Dims dm, SeqState st, int batch, const float* __restrict__ zc, const float* __restrict__ zv,
                                  const float* __restrict__ zf, const float* __restrict__ gains /*[NH,d]*/,
                                  bf16* __restrict__ a /*[NH, max_batch, d]*/) {
  __shared__ float sh[32];
  const int h = blockIdx.y, b = blockIdx.x, d = dm.d;
  if (b >= batch) return;
  const int n = max(0, st.L[b] - 1);
  const float* z = head_split_node(dm, h, b, n, zc, zv, zf);
  float ss = 0.f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) ss += z[i] * z[i];
  ss = block_sum(ss, sh);
  const float inv = rsqrtf(ss / (float)d + dm.eps);
  bf16* dst = a + ((size_t)h * dm.max_batch + b) * d;
  for (int i = threadIdx.x; i < d; i += blockDim.x) dst[i] = __float2bfloat16(z[i] * inv * gains[(size_t)h * d + i]);
}

// y = z + A a  (Eq. 1 reduced to Linear + residual).  Coordinate-head features go straight to the
// feature matrix (rows h*B+b); vertex/face head features become bf16 inputs of the upsample GEMMs.
__global__ void draft_residual_kernel(Dims dm, SeqState st, int batch, const float* __restrict__ zc, const float* __restrict__ zv,
                                      const float* __restrict__ zf, const float* __restrict__ y /*[NH,max_batch,d]*/,
                                      float* __restrict__ feat /*[NF*B, d]*/, bf16* __restrict__ up_in_v /*[2B + 3*Ef*B, d]*/,
                                      bf16* __restrict__ up_in_f /*[Ef*B, d]*/) {
  ptx::grid_dep_launch();
  ptx::grid_dep_wait();
  const int h = blockIdx.y, b = blockIdx.x, d = dm.d;
  if (b >= batch) return;
  const int n = max(0, st.L[b] - 1);
  const float* z = head_split_node(dm, h, b, n, zc, zv, zf);
  const float* yr = y + ((size_t)h * dm.max_batch + b) * d;
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    const float v = z[i] + yr[i];
    if (h < dm.nc) feat[((size_t)h * batch + b) * d + i] = v;
    else if (h < dm.nc + dm.nv) up_in_v[((size_t)(h - dm.nc) * batch + b) * d + i] = __float2bfloat16(v);
    else up_in_f[((size_t)(h - dm.nc - dm.nv) * batch + b) * d + i] = __float2bfloat16(v);
  }
}

// ---- full draft modules (Sec. 3.1 Eq. 1-5): row-wise pieces around the stacked GEMMs and the
// attention launches.  A "set" is one SP head (set = head index h) or one HF-Block (set = offset
// index t); operand and result rows of set t and sequence b sit at row t * max_batch + b.
enum DraftStage { DS_SP = 0, DS_HF_V = 1, DS_HF_C = 2 };

// the fp32 feature that HF-Block t of sequence b refines
//   DS_HF_V: vertex rv = t % 3 of face head e = 1 + t / 3, in the face level's upsampled triples [Ef*B, 3d]
//   DS_HF_C: t < 3 nv: coordinate r = t % 3 of vertex head e = 1 + t / 3; else slot s of face head e,
//            both in the coordinate-level feature matrix (rows as in draft_feature_row)
__device__ inline float* hf_feature(const Dims& dm, int stage, int t, int b, int B, float* xv_pre, float* feat) {
  if (stage == DS_HF_V) return xv_pre + ((size_t)(t / 3) * B + b) * 3 * dm.d + (size_t)(t % 3) * dm.d;
  const int tv = 3 * dm.nv;
  if (t < tv) return feat + ((size_t)dm.nc * B + 3 * ((size_t)(t / 3) * B + b) + t % 3) * dm.d;
  const int tt = t - tv, e0 = tt / 9, s = tt % 9;
  return feat + ((size_t)dm.nc * B + 3 * ((size_t)dm.nv * B + 3 * ((size_t)e0 * B + b) + s / 3) + s % 3) * dm.d;
}
// level-local position of the query of set t (SP: the split node's own position)
__device__ inline int draft_query_pos(const Dims& dm, int stage, int level, int t, int n) {
  if (stage == DS_SP) return level == 0 ? n : (level == 1 ? n / 3 : n / 9);
  if (stage == DS_HF_V) return 3 * (n / 9) + t;
  const int tv = 3 * dm.nv;
  if (t < tv) return 3 * (n / 3 + 1 + t / 3) + t % 3;
  return 9 * (n / 9) + (t - tv);
}

// a[t][b] = bf16(rms(x) * g_t) for the HF-Blocks' inputs
__global__ void hf_prep_kernel(Dims dm, SeqState st, int batch, int stage, float* xv_pre, float* feat,
                               const float* __restrict__ gains /*[T, d]*/, bf16* __restrict__ a /*[T*max_batch, d]*/) {
  ptx::grid_dep_launch();
  ptx::grid_dep_wait();
  __shared__ float sh[32];
  const int b = blockIdx.x, t = blockIdx.y, d = dm.d;
  if (b >= batch) return;
  const float* x = hf_feature(dm, stage, t, b, batch, xv_pre, feat);
  float ss = 0.f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) ss += x[i] * x[i];
  ss = block_sum(ss, sh);
  const float inv = rsqrtf(ss / (float)d + dm.eps);
  bf16* dst = a + ((size_t)t * dm.max_batch + b) * d;
  for (int i = threadIdx.x; i < d; i += blockDim.x) dst[i] = __float2bfloat16(x[i] * inv * gains[(size_t)t * d + i]);
}

// queries of the draft modules: rotate to the query's level position, scale, round; rows
// [t0, t0 + T) of the projection's output become rows (b * T + (t - t0)) of the attention's q
__global__ void draft_q_kernel(Dims dm, SeqState st, int batch, int stage, int level, int t0, int T,
                               const float* __restrict__ qf /*[sets*max_batch, H*dh]*/, const float2* __restrict__ rope_tab,
                               float qscale, bf16* __restrict__ q /*[B*T, H*dh]*/) {
  ptx::grid_dep_launch();
  ptx::grid_dep_wait();
  const int b = blockIdx.x, t = blockIdx.y;        // t counts from t0
  if (b >= batch) return;
  const int n = max(0, st.L[b] - 1), half = dm.dh >> 1, hd = dm.H * dm.dh;
  const int pos = draft_query_pos(dm, stage, level, t0 + t, n);
  const float* src = qf + ((size_t)(t0 + t) * dm.max_batch + b) * hd;
  bf16* dst = q + ((size_t)b * T + t) * hd;
  for (int i = threadIdx.x; i < dm.H * half; i += blockDim.x) {
    const int head = i / half, k = i - head * half;
    float2 cs = make_float2(1.f, 0.f);
    if (dm.theta != 0.f) cs = rope_tab[(size_t)pos * half + k];
    const float x1 = src[head * dm.dh + k], x2 = src[head * dm.dh + half + k];
    dst[head * dm.dh + k] = __float2bfloat16((x1 * cs.x - x2 * cs.y) * qscale);
    dst[head * dm.dh + half + k] = __float2bfloat16((x2 * cs.x + x1 * cs.y) * qscale);
  }
}

// SP-Block, between its attention and its linear layer: y = z + Wo o, a[h][b] = bf16(rms(y) * g_h)
__global__ void sp_mid_kernel(Dims dm, SeqState st, int batch, const float* __restrict__ zc, const float* __restrict__ zv,
                              const float* __restrict__ zf, const float* __restrict__ u /*[NH*max_batch, d]*/,
                              const float* __restrict__ gains, bf16* __restrict__ a) {
  ptx::grid_dep_launch();
  ptx::grid_dep_wait();
  __shared__ float sh[32];
  const int h = blockIdx.y, b = blockIdx.x, d = dm.d;
  if (b >= batch) return;
  const int n = max(0, st.L[b] - 1);
  const float* z = head_split_node(dm, h, b, n, zc, zv, zf);
  const float* ur = u + ((size_t)h * dm.max_batch + b) * d;
  float ss = 0.f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) { const float y = z[i] + ur[i]; ss += y * y; }
  ss = block_sum(ss, sh);
  const float inv = rsqrtf(ss / (float)d + dm.eps);
  bf16* dst = a + ((size_t)h * dm.max_batch + b) * d;
  for (int i = threadIdx.x; i < d; i += blockDim.x) dst[i] = __float2bfloat16((z[i] + ur[i]) * inv * gains[(size_t)h * d + i]);
}

// HF-Block, last step: x += FFN output; the vertex-level blocks also hand the refined vertex
// feature to the next upsample GEMM (bf16 operand row)
__global__ void hf_finish_kernel(Dims dm, SeqState st, int batch, int stage, float* xv_pre, float* feat,
                                 const float* __restrict__ y /*[T*max_batch, d]*/, bf16* __restrict__ up_in_v) {
  ptx::grid_dep_launch();
  ptx::grid_dep_wait();
  const int b = blockIdx.x, t = blockIdx.y, d = dm.d;
  if (b >= batch) return;
  float* x = hf_feature(dm, stage, t, b, batch, xv_pre, feat);
  const float* yr = y + ((size_t)t * dm.max_batch + b) * d;
  bf16* up = stage == DS_HF_V ? up_in_v + ((size_t)dm.nv * batch + 3 * ((size_t)(t / 3) * batch + b) + t % 3) * d : nullptr;
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    const float v = x[i] + yr[i];
    x[i] = v;
    if (up != nullptr) up[i] = __float2bfloat16(v);
  }
}

// Source of draft offset j (single source per offset; supplement, "Optimizations"): offsets 1,2
// -> coordinate heads (rule B); targets in the next two vertices v*+1, v*+2 -> vertex head
// floor(p/3) - v*, wherever the face boundary lies, except where the latest vertex row was also a
// face row (v* % 3 == 0): there the face level keeps the rest of its own face (rule A), face head
// 1; targets beyond two vertices -> face head floor(p/9) - f* + 1 (head e drafts face f* + e - 1).
// With only the coordinate level drafting, coordinate head j serves offset j.
// level 0: head = j; level 1: head = e (1, 2), slot = p % 3; level 2: head = e, slot = p % 9.
__device__ inline void draft_source(const Dims& dm, int n, int j, int& level, int& head, int& slot) {
  const int p = n + j;
  if (j <= 2 || dm.nv == 0) { level = 0; head = j; slot = 0; return; }
  const int ev = p / 3 - n / 3;
  if (ev <= 2 && !((n / 3) % 3 == 0 && p / 9 == n / 9)) { level = 1; head = ev; slot = p % 3; return; }
  level = 2; head = p / 9 - n / 9 + 1; slot = p % 9;
}
// row of the coordinate-level feature matrix [NF*B, d] that holds the feature of (level, head, slot)
__device__ inline int draft_feature_row(const Dims& dm, int level, int head, int slot, int b, int B) {
  if (level == 0) return (head - 1) * B + b;
  if (level == 1) return dm.nc * B + 3 * ((head - 1) * B + b) + slot;
  return dm.nc * B + 3 * (dm.nv * B + 3 * ((head - 1) * B + b) + slot / 3) + slot % 3;
}
// row of the point-level feature matrix [(nv + 3 Ef)*B, d] (the upsample GEMM's operand rows) behind it
__device__ inline int draft_point_row(const Dims& dm, int level, int head, int slot, int b, int B) {
  if (level == 1) return (head - 1) * B + b;
  return dm.nv * B + 3 * ((head - 1) * B + b) + slot / 3;
}

// masked argmax of the chosen feature's logits -> cand[b][j]; cand[b][0] = pending main token
// With a teacher (fm_generate's benchmark stand-in for trained heads, sitting where the Correct stage
// edits drafts) the drafts 1..keep are then replaced by the known continuation and draft keep+1 by a
// different coordinate id.
__global__ void draft_pick_kernel(Dims dm, SeqState st, int batch, const float* __restrict__ logits /*[NF*B, Vpad]*/,
                                  float* __restrict__ logits_out, float* __restrict__ margin_out,
                                  const GenOut* __restrict__ gen, const bf16* __restrict__ point_feat /*[(nv+3Ef)*B, d]*/,
                                  const float* __restrict__ label_g, const float* __restrict__ label_W,
                                  int* __restrict__ labels /*[B, R1]*/, float* __restrict__ label_margin,
                                  float* __restrict__ avg_rows /*[B*R1, Vpad] scratch of the averaged merge*/) {
  ptx::grid_dep_launch();
  ptx::grid_dep_wait();
  const int b = blockIdx.x, j = blockIdx.y;        // j = 0..D
  if (b >= batch) return;
  const bool fin = st.done[b] != 0 || st.nrow[b] <= 0;
  const int n = st.L[b] - 1;
  // ---- label of the point that starts at slot j (Sec. 3.2): a vertex whose three tokens are drafts
  if (labels != nullptr) {
    const bool starts = !fin && j >= 1 && j + 2 <= dm.D && (n + j) % 3 == 0 && dm.nv > 0;
    if (!starts) {
      if (threadIdx.x == 0) { labels[b * dm.R1 + j] = -1; label_margin[b * dm.R1 + j] = 0.f; }
    } else {
      __shared__ float shl[32];
      int level, head, slot;
      draft_source(dm, n, j + 2, level, head, slot);        // the head that drafts the point's last coordinate
      const bf16* f = point_feat + (size_t)draft_point_row(dm, level, head, slot, b, batch) * dm.d;
      float ss = 0.f, z0 = 0.f, z1 = 0.f, z2 = 0.f;
      for (int i = threadIdx.x; i < dm.d; i += blockDim.x) {
        const float v = __bfloat162float(f[i]), vg = v * label_g[i];
        ss += v * v;
        z0 += label_W[i] * vg; z1 += label_W[dm.d + i] * vg; z2 += label_W[2 * dm.d + i] * vg;
      }
      ss = block_sum(ss, shl); z0 = block_sum(z0, shl); z1 = block_sum(z1, shl); z2 = block_sum(z2, shl);
      if (threadIdx.x == 0) {
        const float inv = rsqrtf(ss / (float)dm.d + dm.eps);
        z0 *= inv; z1 *= inv; z2 *= inv;
        int best = 0; float top = z0;
        if (z1 > top) { best = 1; top = z1; }
        if (z2 > top) { best = 2; top = z2; }
        const float second = best == 0 ? fmaxf(z1, z2) : (best == 1 ? fmaxf(z0, z2) : fmaxf(z0, z1));
        labels[b * dm.R1 + j] = best;
        label_margin[b * dm.R1 + j] = top - second;
      }
      __syncthreads();
    }
  }
  if (j == 0) {
    if (threadIdx.x == 0) st.cand[b * dm.R1] = fin ? dm.n_bins + 2 : st.main_tok[b];
    return;
  }
  if (fin) {
    if (threadIdx.x == 0) { st.cand[b * dm.R1 + j] = dm.n_bins + 2; if (margin_out) margin_out[b * dm.D + j - 1] = 0.f; }
    if (logits_out)
      for (int i = threadIdx.x; i < dm.V; i += blockDim.x) logits_out[((size_t)b * dm.D + j - 1) * dm.V + i] = 0.f;
    return;
  }
  int level, head, slot;
  draft_source(dm, n, j, level, head, slot);
  const float* z = logits + (size_t)draft_feature_row(dm, level, head, slot, b, batch) * dm.Vpad;
  if (dm.avg) {
    // every level that predicts this position (supplement, "Integrating the three levels"): the
    // coordinate head of the offset if there is one, the point level for the next two vertices,
    // the face level for the faces its heads draft; the row becomes log(mean of the softmaxes)
    __shared__ float sha[32];
    const float* zs[3];
    int ns = 0;
    const int p = n + j, ev = p / 3 - n / 3, ef = p / 9 - n / 9 + 1;
    if (j <= dm.nc) zs[ns++] = logits + (size_t)draft_feature_row(dm, 0, j, 0, b, batch) * dm.Vpad;
    if (dm.nv > 0 && ev >= 1 && ev <= 2) zs[ns++] = logits + (size_t)draft_feature_row(dm, 1, ev, p % 3, b, batch) * dm.Vpad;
    if (dm.nv > 0 && ev >= 1 && ef >= 1 && ef <= dm.Ef) zs[ns++] = logits + (size_t)draft_feature_row(dm, 2, ef, p % 9, b, batch) * dm.Vpad;
    float mx[3], inv_sum[3];
    for (int k = 0; k < ns; ++k) {
      float m = -INFINITY;
      for (int i = threadIdx.x; i < dm.V; i += blockDim.x) m = fmaxf(m, zs[k][i]);
      m = block_max(m, sha);
      float e = 0.f;
      for (int i = threadIdx.x; i < dm.V; i += blockDim.x) e += expf(zs[k][i] - m);
      e = block_sum(e, sha);
      mx[k] = m; inv_sum[k] = 1.f / e;
    }
    float* row = avg_rows + (size_t)(b * dm.R1 + j) * dm.Vpad;
    for (int i = threadIdx.x; i < dm.V; i += blockDim.x) {
      float pr = 0.f;
      for (int k = 0; k < ns; ++k) pr += expf(zs[k][i] - mx[k]) * inv_sum[k];
      row[i] = logf(pr / (float)ns);
    }
    __syncthreads();
    z = row;
  }
  if (logits_out)
    for (int i = threadIdx.x; i < dm.V; i += blockDim.x) logits_out[((size_t)b * dm.D + j - 1) * dm.V + i] = z[i];
  const Top2 t = block_top2(z, dm, n + j);
  if (threadIdx.x == 0) {
    int tok = t.i1;
    if (gen != nullptr && gen->truth != nullptr) {
      const int keep = gen->keep != nullptr ? gen->keep[(size_t)(*st.step % gen->n_sched) * batch + b] : dm.D;
      const int idx = n + j;
      if (idx < gen->truth_stride) {
        const int tt = gen->truth[(size_t)b * gen->truth_stride + idx];
        if (tt >= 0 && tt < dm.V) {
          if (j <= keep) tok = tt;
          else if (j == keep + 1) tok = (tt + 1) % dm.n_bins;
        }
      }
    }
    st.cand[b * dm.R1 + j] = tok;
    if (margin_out) margin_out[b * dm.D + j - 1] = t.v1 - t.v2;
  }
}

// Self-check of the bounded waits: one thread waits on a barrier of its own that nothing ever
// completes (no copy is in flight, nobody else knows the barrier), with a short limit; the wait
// must come back false, and the kernel then reports it the way the GEMM and attention kernels do.
__global__ void wait_timeout_probe_kernel(int* status, long long limit_cycles) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);
    ptx::fence_mbar_init();
    if (!ptx::mbar_wait(&bar, 0, limit_cycles)) atomicExch(status, -5);
  }
}

__global__ void copy_i32_kernel(const int* __restrict__ src, int* __restrict__ dst, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = src[i];
}
__global__ void copy_f32_kernel(const float* __restrict__ src, float* __restrict__ dst, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = src[i];
}

// ------------------------------------------------------------------------------------------
// Correction of the drafts (Sec. 3.2), one thread per sequence: a row has at most 16 points.
// Slot s of a row is mesh token L - 1 + s; a point is a vertex (3 slots, mesh token index a
// multiple of 3) made of drafts only, inside the rows the next pass feeds.
// ------------------------------------------------------------------------------------------
constexpr int FM_CORRECT_MAX_POINTS = 16;

__device__ inline bool vertex_less(const int* a, const int* b) {       // (z, y, x) order
  if (a[0] != b[0]) return a[0] < b[0];
  if (a[1] != b[1]) return a[1] < b[1];
  return a[2] < b[2];
}

__global__ void correct_kernel(Dims dm, SeqState st, int batch, int* __restrict__ cand, const int* __restrict__ labels,
                               int use_history) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= batch) return;
  const int n = st.nrow[b];
  if (n <= 0) return;
  int* row = cand + (size_t)b * dm.R1;
  const int* lab = labels + (size_t)b * dm.R1;
  const int first = st.L[b] - 1;                 // mesh token index of slot 0
  int slot[FM_CORRECT_MAX_POINTS], face[FM_CORRECT_MAX_POINTS], kind[FM_CORRECT_MAX_POINTS];
  bool usable[FM_CORRECT_MAX_POINTS];
  int m = 0;
  for (int s = 1; s + 2 < n && m < FM_CORRECT_MAX_POINTS; ++s) {
    const int j = first + s;
    if (j % 3 != 0) continue;
    slot[m] = s;
    face[m] = j / 9;
    kind[m] = lab[s];
    usable[m] = row[s] >= 0 && row[s] < dm.n_bins && row[s + 1] >= 0 && row[s + 1] < dm.n_bins && row[s + 2] >= 0 &&
                row[s + 2] < dm.n_bins;
    ++m;
  }
  // historical points against the accepted vertices: the complete ones of the face that holds the
  // main token and of the face before it (at most five), oldest first; a point that equals none of
  // them becomes the nearest (ties to the earliest)
  if (use_history) {
    int win[5][3], nw = 0;
    const int* h = st.hist + (size_t)b * FM_HIST;
    const int fprev = first / 9 - 1;
    for (int v = fprev > 0 ? 3 * fprev : 0; v < first / 3 && nw < 5; ++v) {
      const int t0 = h[(3 * v) & (FM_HIST - 1)], t1 = h[(3 * v + 1) & (FM_HIST - 1)], t2 = h[(3 * v + 2) & (FM_HIST - 1)];
      if (t0 < 0 || t0 >= dm.n_bins || t1 < 0 || t1 >= dm.n_bins || t2 < 0 || t2 >= dm.n_bins) continue;
      win[nw][0] = t0; win[nw][1] = t1; win[nw][2] = t2; ++nw;
    }
    for (int k = 0; k < m && nw > 0; ++k) {
      if (kind[k] != 0 || !usable[k]) continue;
      const int z = row[slot[k]], y = row[slot[k] + 1], x = row[slot[k] + 2];
      int src = -1;
      long long best = 0;
      for (int q = 0; q < nw; ++q) {
        const long long dz = win[q][0] - z, dy = win[q][1] - y, dx = win[q][2] - x;
        const long long dist = dz * dz + dy * dy + dx * dx;
        if (src < 0 || dist < best) { src = q; best = dist; }
      }
      if (best != 0) { row[slot[k]] = win[src][0]; row[slot[k] + 1] = win[src][1]; row[slot[k] + 2] = win[src][2]; }
    }
  }
  // intra-batch points in sequence order; each sees the corrections before it
  for (int k = 0; k < m; ++k) {
    if (kind[k] != 2 || !usable[k]) continue;
    const int z = row[slot[k]], y = row[slot[k] + 1], x = row[slot[k] + 2];
    bool twin = false;
    for (int q = 0; q < m; ++q)
      if (q != k && usable[q] && row[slot[q]] == z && row[slot[q] + 1] == y && row[slot[q] + 2] == x) twin = true;
    if (twin) continue;
    int src = -1;
    long long best = 0;
    for (int q = 0; q < k; ++q) {
      if (kind[q] != 1 || !usable[q] || face[q] == face[k]) continue;
      const long long dz = row[slot[q]] - z, dy = row[slot[q] + 1] - y, dx = row[slot[q] + 2] - x;
      const long long dist = dz * dz + dy * dy + dx * dx;
      if (src < 0 || dist < best) { src = q; best = dist; }
    }
    if (src >= 0) {
      row[slot[k]] = row[slot[src]];
      row[slot[k] + 1] = row[slot[src] + 1];
      row[slot[k] + 2] = row[slot[src] + 2];
    }
  }
  // z-y-x order inside every face, among the slots its usable points occupy (a face has at most
  // three): exchange sort on the triples
  for (int k0 = 0; k0 < m;) {
    int k1 = k0;
    while (k1 < m && face[k1] == face[k0]) ++k1;
    for (int i = k0; i < k1; ++i) {
      if (!usable[i]) continue;
      for (int j = i + 1; j < k1; ++j) {
        if (!usable[j]) continue;
        int* a = row + slot[i];
        int* c = row + slot[j];
        if (vertex_less(c, a)) {
          for (int t = 0; t < 3; ++t) { const int tmp = a[t]; a[t] = c[t]; c[t] = tmp; }
        }
      }
    }
    k0 = k1;
  }
}
