// C ABI and host orchestration of the speculative decode step (see include/flashmesh.h).
// All arithmetic of the path runs in the kernels of this directory; the host only carves the
// workspace, uploads weights and enqueues launches.
#include "../../include/flashmesh.h"

#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>
#include <new>
#include <utility>
#include <vector>

#include "fm_attention.cuh"
#include "fm_common.cuh"
#include "fm_gemm_tc.cuh"
#include "fm_kernels.cuh"

namespace {

constexpr int STACK_LEVEL[5] = {0, 1, 2, 1, 0};
constexpr int PREFILL_CHUNK = 256;      // conditioning rows projected per launch group
constexpr int FM_ROPE_SLACK = 64;       // the HF-Blocks of the face level query positions up to 4 faces ahead

struct LayerDev {
  bf16 *Wqkv, *Wo, *W1, *W2;
  float *g1, *g2;
  bf16 *K, *V;                          // [max_batch, Hkv, P + cap, dh]
  int tmK, tmV;                         // tensor-map indices
};

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline int round_up(int v, int a) { return (v + a - 1) / a * a; }

}  // namespace

// Attention scratch (group partials, then tickets) for fm_verify_static_scratch: lives in the
// library image, so every GPU that loads the library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_static_attn_scratch[FM_STATIC_SCRATCH_BYTES];

struct fm_ctx {
  fm_config cfg;
  Dims dm;
  cudaStream_t stream;
  char* ws;
  size_t ws_bytes;
  // weights
  bf16* E;
  std::vector<LayerDev> layers[5];
  bf16 *S_cv, *S_vf, *U_fv, *U_vc, *W_out, *headA;
  float *g_out, *head_g;
  double* inv_freq;
  float2* rope_tab;                      // [max level positions][dh/2] (cos, sin)
  // state
  SeqState st;
  // activations
  float *xc, *xv, *xf, *logits, *tmp3d;
  bf16 *qbuf, *a_norm, *a_up, *a_cat, *a_cat2, *a_attn, *a_ff;
  bool fuse_hourglass;                     // shorten gather and upsample add inside the adjacent GEMM epilogues
  float *hc_ring, *hv_ring, *trif_ring, *triv_ring, *zc, *zv, *zf;
  // draft
  bf16 *dh_a, *up_in_v, *up_in_f, *feat_n;
  float *dh_y, *feat, *dlogits;
  float *label_g, *label_W, *label_margin;   // label head of the correction stage and its last results
  int* labels;
  int *step_in, *step_cand, *step_nacc, *step_em, *step_kv;     // device side of fm_step_host
  float* avg_rows;                           // [B*R1, Vpad] rows of the averaged merge
  // full draft modules: SP-Block attention (per head) and HF-Blocks (per offset), stacked per stage
  bf16 *spWq, *spWo; float* sp_ga;
  bf16 *hfWq[2], *hfW1[2], *hfW2[2]; float* hf_g[2];       // [0] vertex-level blocks (3 Ef), [1] coordinate-level blocks (3 nv + 9 Ef)
  int hf_T[2];
  float *d_qf, *d_out, *xv_pre;              // projections' fp32 results [sets*max_batch, .], face level's upsampled triples
  bf16 *d_q, *d_attn, *d_a, *d_h1;           // rotated queries, attention output [hi | lo], block inputs, FFN hidden [hi | lo]
  int draft_sets;                            // rows reserved per stage: max number of sets
  int attn_mt_draft[3];                      // query tiles of the draft modules' attention launches per level
  // attention scratch and TMA descriptors
  float* attn_part;
  int* attn_ticket;
  int attn_chunk, attn_G[3], attn_max_groups[3], attn_mt[3];
  CUtensorMap* tmaps;                    // device array
  std::vector<CUtensorMap> tmaps_host;
  struct TmapKey { const void* base; uint64_t rows, cols; uint32_t box_rows; uint32_t parts; };   // parts = 0: 2-D map
  std::vector<TmapKey> tmap_keys;
  size_t tmaps_cap, tmaps_uploaded;
  // per-tile sums of squares of the residual rows (RMSNorm statistics handed between GEMMs)
  float* ssq;
  int ssq_n, ssq_ld;    // slots the last producer filled, floats between slots
  bool use_pdl;
  bool debug_sync;      // FM_DEBUG_SYNC: wait for and check every launch
  // prefill temporaries
  bf16* pre_a;
  float* pre_o;
  int* prompt_off_dev;
  // generate
  GenOut* gen_dev;
  long long* stats_dev;
  int* host_done;       // pinned, mapped
  int* host_done_dev;
  // optional per-kernel-class timing (fm_profile_begin / fm_profile_end)
  bool prof_on;
  std::vector<cudaEvent_t> prof_ev;     // pairs
  std::vector<int> prof_cls;
  size_t prof_used;
  double prof_ms[3], prof_bytes[3];
  long long prof_n[3];
  int only_class;       // -1, or the kernel class (ProfClass) that alone is launched (fm_profile_class)
  int cur_class;        // class of the launch being enqueued
  double class_bytes;   // weight bytes of the GEMM launches enqueued by fm_profile_class
  int split_target;     // CTAs a GEMM launch aims for (M tiles x K splits)
  int stage_cap;        // tuning knob: upper bound on the GEMM ring depth (0 = none)
  int n_sm;                                  // SMs of the device
  int device;                                // ordinal of the device the context was created on
  size_t attn_ticket_n;                      // entries of attn_ticket
  int split_target_deep;                     // the same for launches whose CTAs stream long K ranges
  int launch_error;     // first error met while enqueueing (capacity, descriptor creation)
  // one decode pass (draft, teacher edit, verify, accept) captured as a CUDA graph
  cudaGraph_t graph;
  cudaGraphExec_t graph_exec;
  int graph_batch;
  int64_t graph_launches;
  bool capturing, graph_unavailable;
  // Stepwise calls repeated with the same pointer arguments are replayed as CUDA graphs.
  struct CallGraph {
    const void* key[4] = {nullptr, nullptr, nullptr, nullptr};
    int batch = -1;
    bool valid = false, failed = false;
    int64_t launches = 0;
    cudaGraphExec_t exec = nullptr;
  } cg_verify, cg_draft;
  bool call_graphs_off;   // plain launches only (diagnostic modes, calls that swap scratch buffers)
  int batch;
  bool gen_fresh;       // no fm_generate call since the last fm_prefill
  std::vector<int> plen_host;
  int phase;            // 0 created, 1 prefilled / accepted, 2 verified
  int64_t launches;
};

namespace {

// ------------------------------------------------------------------------------------------
// configuration checks and workspace layout
// ------------------------------------------------------------------------------------------
int check_config(const fm_config* c) {
  if (c == nullptr) return FM_ERR_INVALID_ARG;
  if (c->d_model <= 0 || c->n_heads <= 0 || c->n_kv_heads <= 0 || c->head_dim <= 0 || c->d_ff <= 0) return FM_ERR_INVALID_ARG;
  if (c->n_heads % c->n_kv_heads != 0) return FM_ERR_INVALID_ARG;
  if (c->n_bins <= 0 || c->n_prefix < 0 || c->max_batch <= 0 || c->max_tokens <= 0) return FM_ERR_INVALID_ARG;
  if (c->draft_len < 0 || c->norm_eps < 0.f) return FM_ERR_INVALID_ARG;
  for (int i = 0; i < 3; ++i) if (c->window[i] < 0) return FM_ERR_INVALID_ARG;
  for (int i = 0; i < 5; ++i) if (c->layers[i] < 1) return FM_ERR_UNSUPPORTED;
  if (c->draft_len > FM_MAX_DRAFT) return FM_ERR_UNSUPPORTED;
  if (c->d_model % 64 != 0 || c->d_ff % 64 != 0 || (c->n_heads * c->head_dim) % 128 != 0) return FM_ERR_UNSUPPORTED;
  if (c->head_dim != 64 && c->head_dim != 128) return FM_ERR_UNSUPPORTED;
  if (c->draft_len >= 7 && (c->draft_len + 8) / 9 + 1 > FM_MAX_FACE_HEADS) return FM_ERR_UNSUPPORTED;
  if (c->draft_heads != FM_HEADS_REDUCED && c->draft_heads != FM_HEADS_FULL) return FM_ERR_INVALID_ARG;
  if (c->draft_levels != FM_LEVELS_THREE && c->draft_levels != FM_LEVELS_COORD) return FM_ERR_INVALID_ARG;
  if (c->hf_ff < 0 || c->hf_ff % 64 != 0) return FM_ERR_UNSUPPORTED;
  if (c->max_tokens < c->draft_len + 2) return FM_ERR_INVALID_ARG;
  return FM_OK;
}

Dims make_dims(const fm_config& c) {
  Dims dm;
  dm.d = c.d_model; dm.H = c.n_heads; dm.Hkv = c.n_kv_heads; dm.dh = c.head_dim; dm.dff = c.d_ff;
  dm.n_bins = c.n_bins; dm.V = c.n_bins + 3; dm.Vpad = round_up(dm.V, 128); dm.P = c.n_prefix;
  dm.D = c.draft_len; dm.R1 = dm.D + 1; dm.mv = (dm.R1 + 2) / 3; dm.mf = (dm.R1 + 8) / 9;
  for (int l = 0; l < 3; ++l) {
    dm.window[l] = c.window[l];
    const int ratio = fm_ratio(l);
    const int linear = (c.max_tokens + ratio - 1) / ratio + 1;
    // a windowed level keeps a ring of window + rows of one pass (+ slack) slots
    const int ring = c.window[l] > 0 ? c.window[l] + fm_rows_per_seq(dm, l) + 8 : linear;
    dm.cap[l] = ring < linear ? ring : linear;
  }
  dm.max_batch = c.max_batch; dm.max_tokens = c.max_tokens; dm.allow_eos = c.allow_eos;
  dm.eps = c.norm_eps; dm.theta = c.rope_theta;
  // face head e drafts face f* + e - 1 (f* holds the pending token); offsets below 7 never leave
  // the next two points, a draft of D tokens reaches face f* + (8 + D) / 9
  const bool coord_only = c.draft_levels == FM_LEVELS_COORD;
  dm.nc = coord_only ? (dm.D > 0 ? dm.D : 1) : 2;
  dm.nv = coord_only ? 0 : 2;
  dm.Ef = coord_only ? 0 : (dm.D >= 7 ? (dm.D + 8) / 9 + 1 : 1);
  dm.NH = dm.nc + dm.nv + dm.Ef;
  dm.full = c.draft_heads == FM_HEADS_FULL ? 1 : 0;
  dm.avg = c.avg_levels != 0 ? 1 : 0;
  dm.hf = c.hf_ff > 0 ? c.hf_ff : c.d_model;
  dm.has_label = 0;                     // set by fm_create when the weights hold a label head
  return dm;
}

// bump allocator; with base == nullptr it only measures
struct Carver {
  char* base; size_t off;
  template <typename T> T* take(size_t n) {
    off = align_up(off, 256);
    T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off += n * sizeof(T);
    return p;
  }
};

void carve(fm_ctx* c, Carver& cv) {
  const Dims& dm = c->dm;
  const size_t d = dm.d, B = dm.max_batch;
  const size_t qkvw = (size_t)(dm.H + 2 * dm.Hkv) * dm.dh, hd = (size_t)dm.H * dm.dh;
  c->E = cv.take<bf16>((size_t)dm.V * d);
  for (int s = 0; s < 5; ++s) {
    c->layers[s].resize(c->cfg.layers[s]);
    const int lvl = STACK_LEVEL[s];
    const size_t kvn = B * dm.Hkv * (size_t)(dm.P + dm.cap[lvl]) * dm.dh;
    for (auto& L : c->layers[s]) {
      L.Wqkv = cv.take<bf16>(align_up(qkvw, 128) * d);
      L.Wo = cv.take<bf16>(align_up(d, 128) * hd);
      L.W1 = cv.take<bf16>(align_up((size_t)dm.dff, 128) * d);
      L.W2 = cv.take<bf16>(align_up(d, 128) * dm.dff);
      L.g1 = cv.take<float>(d);
      L.g2 = cv.take<float>(d);
      L.K = cv.take<bf16>(kvn);
      L.V = cv.take<bf16>(kvn);
    }
  }
  c->S_cv = cv.take<bf16>(align_up(d, 128) * 3 * d);
  c->S_vf = cv.take<bf16>(align_up(d, 128) * 3 * d);
  c->U_fv = cv.take<bf16>(align_up(3 * d, 128) * d);
  c->U_vc = cv.take<bf16>(align_up(3 * d, 128) * d);
  c->W_out = cv.take<bf16>((size_t)dm.Vpad * d);
  c->headA = cv.take<bf16>((size_t)dm.NH * align_up(d, 128) * d);
  c->g_out = cv.take<float>(d);
  c->head_g = cv.take<float>((size_t)dm.NH * d);
  c->inv_freq = cv.take<double>(dm.dh / 2);
  c->rope_tab = cv.take<float2>((size_t)(dm.max_tokens + 1 + FM_ROPE_SLACK) * (dm.dh / 2));
  // state
  c->st.L = cv.take<int>(B); c->st.nrow = cv.take<int>(B); c->st.main_tok = cv.take<int>(B);
  c->st.done = cv.take<int>(B); c->st.t_end = cv.take<int>(B); c->st.plen = cv.take<int>(B);
  c->st.cand = cv.take<int>(B * dm.R1); c->st.o = cv.take<int>(B * dm.R1);
  c->st.margin = cv.take<float>(B * dm.R1);
  c->st.status = cv.take<int>(1); c->st.n_active = cv.take<int>(4); c->st.step = cv.take<int>(1);
  // activations (row counts padded to 16 so that later tiles never run off the end)
  const size_t Rc = align_up(B * dm.R1, 16), Rv = align_up(B * dm.mv, 16), Rf = align_up(B * dm.mf, 16);
  c->xc = cv.take<float>(Rc * d); c->xv = cv.take<float>(Rv * d); c->xf = cv.take<float>(Rf * d);
  c->qbuf = cv.take<bf16>(Rc * hd);
  c->ssq_ld = (int)Rc;
  c->ssq = cv.take<float>((size_t)((d + 127) / 128) * tc::MAX_SPLIT * Rc);
  c->logits = cv.take<float>(Rc * dm.Vpad); c->tmp3d = cv.take<float>(Rv * 3 * d);
  // GEMM operand rows of the backbone hold two bfloat16 terms per value: [hi | lo]
  c->a_norm = cv.take<bf16>(Rc * 2 * d); c->a_up = cv.take<bf16>(Rc * 2 * d); c->a_cat = cv.take<bf16>(Rv * 6 * d); c->a_cat2 = cv.take<bf16>(Rf * 6 * d);
  c->a_attn = cv.take<bf16>(Rc * 2 * hd); c->a_ff = cv.take<bf16>(Rc * 2 * dm.dff);
  c->hc_ring = cv.take<float>(B * FM_RING_C * d); c->hv_ring = cv.take<float>(B * FM_RING_V * d);
  c->trif_ring = cv.take<float>(B * FM_RING_F * 3 * d); c->triv_ring = cv.take<float>(B * FM_RING_V * 3 * d);
  c->zc = cv.take<float>(B * FM_RING_C * d); c->zv = cv.take<float>(B * FM_RING_V * d);
  c->zf = cv.take<float>(B * FM_RING_F * d);
  // draft
  const size_t NF = (size_t)dm.nc + 3 * dm.nv + 9 * (size_t)dm.Ef;
  c->dh_a = cv.take<bf16>(((size_t)dm.NH * B + 16) * d); c->dh_y = cv.take<float>((size_t)dm.NH * B * d);
  c->up_in_v = cv.take<bf16>(align_up((dm.nv + 3 * (size_t)dm.Ef) * B + 1, 16) * d);
  c->up_in_f = cv.take<bf16>(align_up((size_t)dm.Ef * B + 1, 16) * d);
  c->feat = cv.take<float>(align_up(NF * B, 16) * d); c->feat_n = cv.take<bf16>(align_up(NF * B, 16) * d);
  c->dlogits = cv.take<float>(align_up(NF * B, 16) * dm.Vpad);
  c->label_g = cv.take<float>(d); c->label_W = cv.take<float>(3 * d);
  c->labels = cv.take<int>(B * dm.R1); c->label_margin = cv.take<float>(B * dm.R1);
  c->st.hist = cv.take<int>(B * FM_HIST);
  c->step_in = cv.take<int>(B * dm.R1); c->step_cand = cv.take<int>(B * dm.R1); c->step_nacc = cv.take<int>(B);
  c->step_em = cv.take<int>(B * dm.R1); c->step_kv = cv.take<int>(B * 3);
  c->avg_rows = dm.avg ? cv.take<float>(B * dm.R1 * (size_t)dm.Vpad) : nullptr;
  c->hf_T[0] = 3 * dm.Ef; c->hf_T[1] = 3 * dm.nv + 9 * dm.Ef;
  c->draft_sets = dm.NH > c->hf_T[1] ? dm.NH : c->hf_T[1];
  if (dm.full) {
    const size_t hdp = align_up(hd, 128), dp = align_up(d, 128), hfp = align_up((size_t)dm.hf, 128), S = c->draft_sets;
    c->spWq = cv.take<bf16>((size_t)dm.NH * hdp * d); c->spWo = cv.take<bf16>((size_t)dm.NH * dp * hd);
    c->sp_ga = cv.take<float>((size_t)dm.NH * d);
    for (int k = 0; k < 2; ++k) {
      const size_t T = c->hf_T[k] > 0 ? c->hf_T[k] : 1;
      c->hfWq[k] = cv.take<bf16>(T * hdp * d); c->hfW1[k] = cv.take<bf16>(T * hfp * hd); c->hfW2[k] = cv.take<bf16>(T * dp * dm.hf);
      c->hf_g[k] = cv.take<float>(T * d);
    }
    const size_t rows = S * B + 16;
    c->d_qf = cv.take<float>(rows * hd); c->d_out = cv.take<float>(rows * d);
    c->xv_pre = cv.take<float>(((size_t)dm.Ef * B + 16) * 3 * d);
    c->d_q = cv.take<bf16>(rows * hd); c->d_attn = cv.take<bf16>(rows * 2 * hd); c->d_a = cv.take<bf16>(rows * d);
    c->d_h1 = cv.take<bf16>(rows * 2 * dm.hf);
  }
  // attention: chunk size, chunks per group (fixed per level so that the reduction order of a row
  // never depends on the cache length), group partials (max over levels), tickets
  c->attn_chunk = dm.dh == 64 ? 128 : 64;
  size_t part_max = 0, ticket_max = 0;
  for (int l = 0; l < 3; ++l) {
    const int max_chunks = (dm.P + dm.cap[l] + c->attn_chunk - 1) / c->attn_chunk;
    c->attn_mt[l] = (fm_rows_per_seq(dm, l) * (dm.H / dm.Hkv) + 15) / 16;
    // query rows of the draft modules at this level: SP heads and HF offsets, whichever launch has more
    const int dq = !dm.full ? 0 : (l == 0 ? (dm.nc > 3 * dm.nv + 9 * dm.Ef ? dm.nc : 3 * dm.nv + 9 * dm.Ef) : (l == 1 ? (dm.nv > 3 * dm.Ef ? dm.nv : 3 * dm.Ef) : dm.Ef));
    c->attn_mt_draft[l] = (dq * (dm.H / dm.Hkv) + 15) / 16;
    const int mt_max = c->attn_mt[l] > c->attn_mt_draft[l] ? c->attn_mt[l] : c->attn_mt_draft[l];
    // Chunks per group: the number of groups (1 .. what the merge can stage: 24, fewer for wide
    // heads) that minimises waves x (chunks per CTA + a CTA's fixed cost), with the cache full.
    // The fixed cost (pipeline start, merge of the warps, and with several groups the partials,
    // the ticket and the last CTA's merge) was measured at batch 16 as about 5 chunk times:
    // 87 / 70 / 63 / 61 us per launch with at most 8 / 16 / 32 / 64 chunks per group.
    const int g_cap = dm.dh == 64 ? AttnCfg<64, 128, 8>::MAX_GROUPS : AttnCfg<128, 64, 4>::MAX_GROUPS;
    const size_t tiles_l = (size_t)dm.Hkv * B * c->attn_mt[l];      // the verify pass decides the grouping
    int G = max_chunks;
    double best = 0.0;
    for (int ng = 1; ng <= g_cap && ng <= max_chunks; ++ng) {
      const int Gc = (max_chunks + ng - 1) / ng, groups = (max_chunks + Gc - 1) / Gc;
      const size_t waves = (tiles_l * groups + 147) / 148;
      const double cost = (double)waves * (Gc + (groups == 1 ? 3 : 6));
      if (ng == 1 || cost < best) { best = cost; G = Gc; }
    }
    const char* gm = getenv("FM_ATTN_G");                 // tuning knob: chunks per group, all levels
    if (gm != nullptr && atoi(gm) > 0) {
      const int G_min = (max_chunks + g_cap - 1) / g_cap;
      G = atoi(gm) < G_min ? G_min : atoi(gm);
    }
    c->attn_G[l] = G;
    c->attn_max_groups[l] = (max_chunks + G - 1) / G;
    const size_t need = B * dm.Hkv * (size_t)mt_max * c->attn_max_groups[l] * 16 * (dm.dh + 2);
    part_max = need > part_max ? need : part_max;
    const size_t tk = B * dm.Hkv * (size_t)mt_max;
    ticket_max = tk > ticket_max ? tk : ticket_max;
  }
  c->attn_part = cv.take<float>(part_max);
  c->attn_ticket = cv.take<int>(ticket_max);
  c->attn_ticket_n = ticket_max;
  int n_layers = 0;
  for (int s = 0; s < 5; ++s) n_layers += c->cfg.layers[s];
  c->tmaps_cap = (size_t)6 * n_layers + 128;
  c->tmaps = cv.take<CUtensorMap>(c->tmaps_cap);
  // prefill temporaries
  c->pre_a = cv.take<bf16>((size_t)PREFILL_CHUNK * d);
  c->pre_o = cv.take<float>((size_t)PREFILL_CHUNK * 2 * dm.Hkv * dm.dh);
  c->prompt_off_dev = cv.take<int>(B + 1);
  c->gen_dev = cv.take<GenOut>(1);
  c->stats_dev = cv.take<long long>(FM_MAX_DRAFT + 4);
  cv.off = align_up(cv.off, 256);
}

#define CUDA_OK(expr) do { if ((expr) != cudaSuccess) return FM_ERR_CUDA; } while (0)

// fp32 host matrix [rows, cols] -> bf16 device rows (nearest-even), staged through `tmp`
int upload_bf16(bf16* dst, const float* src, size_t n, std::vector<uint16_t>& tmp) {
  if (src == nullptr) return FM_ERR_INVALID_ARG;
  tmp.resize(n);
  for (size_t i = 0; i < n; ++i) {
    uint32_t u;
    memcpy(&u, src + i, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) { tmp[i] = 0x7fc0; continue; }     // NaN
    u += 0x7fffu + ((u >> 16) & 1u);
    tmp[i] = (uint16_t)(u >> 16);
  }
  CUDA_OK(cudaMemcpy(dst, tmp.data(), n * 2, cudaMemcpyHostToDevice));
  return FM_OK;
}
// fp32 host matrix [M, K] -> device weight slabs for the tensor-core GEMM: M padded to tiles of
// 128 rows (zeros), K cut into slabs of 64; slab (t, k) is stored as the 16 KB image the MMA reads
// from shared memory (row r at r*128 bytes, its 16-byte chunk c at position c ^ (r & 7): the
// 128-byte swizzle), slabs of one tile one after the other.
int upload_packed(bf16* dst, const float* src, size_t M, size_t K, std::vector<uint16_t>& tmp) {
  if (src == nullptr) return FM_ERR_INVALID_ARG;
  const size_t tiles = (M + 127) / 128, slabs = K / 64;
  tmp.assign(tiles * 128 * K, 0);
  for (size_t m = 0; m < M; ++m) {
    const size_t t = m / 128, r = m % 128;
    for (size_t k = 0; k < K; ++k) {
      uint32_t u;
      memcpy(&u, src + m * K + k, 4);
      uint16_t h;
      if ((u & 0x7fffffffu) > 0x7f800000u) h = 0x7fc0;                        // NaN
      else { u += 0x7fffu + ((u >> 16) & 1u); h = (uint16_t)(u >> 16); }
      const size_t kb = k / 64, c = (k % 64) / 8, e = k % 8;
      tmp[((t * slabs + kb) * 128 + r) * 64 + ((c ^ (r & 7)) * 8) + e] = h;
    }
  }
  CUDA_OK(cudaMemcpy(dst, tmp.data(), tmp.size() * 2, cudaMemcpyHostToDevice));
  return FM_OK;
}
int upload_f32(float* dst, const float* src, size_t n) {
  if (src == nullptr) return FM_ERR_INVALID_ARG;
  CUDA_OK(cudaMemcpy(dst, src, n * 4, cudaMemcpyHostToDevice));
  return FM_OK;
}

// ------------------------------------------------------------------------------------------
// launch helpers
// ------------------------------------------------------------------------------------------
#define LAUNCH(ctx, kern, grid, block, smem, ...)                        \
  do {                                                                   \
    if ((ctx)->only_class >= 0 && (ctx)->cur_class != (ctx)->only_class) break; \
    if ((ctx)->launch_error != FM_OK) break;                             \
    kern<<<grid, block, smem, (ctx)->stream>>>(__VA_ARGS__);             \
    (ctx)->launches++;                                                   \
    if ((ctx)->debug_sync) debug_sync_check(ctx, #kern);                 \
  } while (0)

enum ProfClass { PROF_GEMM = 0, PROF_ATTN = 1, PROF_OTHER = 2 };

// Diagnostic mode (environment FM_DEBUG_SYNC): wait for every launch and name the first one that
// ends with an error; nothing is launched after it.  Not used while a graph is being captured.
void debug_sync_check(fm_ctx* c, const char* what) {
  if (c->capturing || c->launch_error != FM_OK) return;
  cudaError_t err = cudaStreamSynchronize(c->stream);
  if (err == cudaSuccess) err = cudaGetLastError();
  if (err != cudaSuccess) {
    fprintf(stderr, "flashmesh: launch %ld (%s, class %d) ended with: %s\n", c->launches, what, c->cur_class,
            cudaGetErrorString(err));
    c->launch_error = FM_ERR_CUDA;
  }
}

void prof_drain(fm_ctx* c) {
  if (c->prof_used == 0) return;
  cudaStreamSynchronize(c->stream);
  for (size_t i = 0; i < c->prof_used; ++i) {
    float ms = 0.f;
    cudaEventElapsedTime(&ms, c->prof_ev[2 * i], c->prof_ev[2 * i + 1]);
    c->prof_ms[c->prof_cls[i]] += ms;
  }
  c->prof_used = 0;
}
// bracket the launches issued between prof_open and prof_close with an event pair
inline long prof_open(fm_ctx* c, int cls, double bytes) {
  if (!c->prof_on) return -1;
  if (c->prof_used == c->prof_cls.size()) prof_drain(c);
  const size_t i = c->prof_used++;
  c->prof_cls[i] = cls;
  c->prof_bytes[cls] += bytes;
  c->prof_n[cls] += 1;
  cudaEventRecord(c->prof_ev[2 * i], c->stream);
  return (long)i;
}
inline void prof_close(fm_ctx* c, long i) {
  if (i >= 0) cudaEventRecord(c->prof_ev[2 * i + 1], c->stream);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// 2-D bf16 tensor [rows, cols] row-major, box [box_rows, 64 columns] (128 bytes), 128-byte swizzle.
// Returns the index of the new map in ctx->tmaps_host, or -1.
int add_tmap_bf16(fm_ctx* c, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (fn == nullptr) return -1;
  CUtensorMap m;
  const cuuint64_t gdim[2] = {cols, rows};
  const cuuint64_t gstride[1] = {cols * 2};
  const cuuint32_t box[2] = {64, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  if (fn(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return -1;
  c->tmaps_host.push_back(m);
  return (int)c->tmaps_host.size() - 1;
}

// GEMM operand rows [rows, parts * K] bf16 seen as a 3-D tensor (K, rows, parts): box 64 columns x
// box_rows rows x parts, 128-byte swizzle, so that one copy brings the hi and the lo tile of a K slab,
// one tile after the other.
int add_tmap_operand(fm_ctx* c, const void* base, uint64_t rows, uint64_t K, uint32_t parts, uint32_t box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (fn == nullptr) return -1;
  CUtensorMap m;
  const cuuint64_t gdim[3] = {K, rows, parts};
  const cuuint64_t gstride[2] = {parts * K * 2, K * 2};
  const cuuint32_t box[3] = {64, box_rows, parts};
  const cuuint32_t estr[3] = {1, 1, 1};
  if (fn(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), gdim, gstride, box, estr,
         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return -1;
  c->tmaps_host.push_back(m);
  return (int)c->tmaps_host.size() - 1;
}

// index of the tensor map for a bf16 matrix / box, created on first use (all call sites are
// visited by the first pass, before any timing or capture)
int tmap_for(fm_ctx* c, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows, uint32_t parts) {
  for (size_t i = 0; i < c->tmap_keys.size(); ++i) {
    const auto& k = c->tmap_keys[i];
    if (k.base == base && k.rows == rows && k.cols == cols && k.box_rows == box_rows && k.parts == parts) return (int)i;
  }
  if (c->tmaps_host.size() >= c->tmaps_cap || c->capturing) return -1;   // descriptors are made before capture
  const int idx = add_tmap_operand(c, base, rows, cols, parts, box_rows);
  if (idx < 0) return -1;
  c->tmap_keys.push_back({base, rows, cols, box_rows, parts});
  cudaMemcpyAsync(c->tmaps + idx, &c->tmaps_host[idx], sizeof(CUtensorMap), cudaMemcpyHostToDevice, c->stream);
  cudaStreamSynchronize(c->stream);
  return idx;
}

// Launch with the programmatic-dependent-launch attribute: the kernel may start while its
// predecessor is still running and must execute griddepcontrol.wait before it touches anything a
// predecessor produces (and before it exits).  Kernels launched through LAUNCH are full barriers.
// `cluster` with more than one CTA makes thread-block clusters of that shape.
template <typename... KArgs, typename... CArgs>
void launch_pdl(fm_ctx* c, dim3 cluster, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, CArgs&&... args) {
  if (c->only_class >= 0 && c->cur_class != c->only_class) return;
  if (c->launch_error != FM_OK) return;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = c->stream;
  cudaLaunchAttribute at[2];
  int n = 0;
  if (c->use_pdl) {
    at[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  if (cluster.x * cluster.y * cluster.z > 1) {
    at[n].id = cudaLaunchAttributeClusterDimension;
    at[n].val.clusterDim.x = cluster.x;
    at[n].val.clusterDim.y = cluster.y;
    at[n].val.clusterDim.z = cluster.z;
    ++n;
  }
  cfg.attrs = at;
  cfg.numAttrs = n;
  const cudaError_t err = cudaLaunchKernelEx(&cfg, kern, std::forward<CArgs>(args)...);
  if (err != cudaSuccess) {
    if (getenv("FM_DEBUG") != nullptr)
      fprintf(stderr, "flashmesh: launch failed: %s (grid %u %u %u, block %u, smem %zu, cluster %u %u %u)\n", cudaGetErrorString(err),
              grid.x, grid.y, grid.z, block.x, smem, cluster.x, cluster.y, cluster.z);
    if (c->launch_error == FM_OK) c->launch_error = FM_ERR_CUDA;
  }
  c->launches++;
  if (c->debug_sync) {
    char what[96];
    snprintf(what, sizeof what, "grid %u %u %u block %u smem %zu cluster %u", grid.x, grid.y, grid.z, block.x, smem, cluster.y);
    debug_sync_check(c, what);
  }
}

tc::Epi epi_plain(void* out, int ldo) {
  tc::Epi e{};
  e.out = out;
  e.ldo = ldo;
  return e;
}

// y[n][m] = W[w_row0 + m, :] . A[a_row0 + n, :], n < R, m < M, finished by the epilogue `mode`
// (see fm_gemm_tc.cuh).  W: packed weight slabs of a matrix with K columns (w_row0 a multiple of
// 128), A: [a_rows_alloc, a_parts * K] bf16 (rows padded to 16; a_parts = 2: [hi | lo] terms).  The
// K split (= cluster size) depends on the shapes only.
void gemm(fm_ctx* c, const bf16* W, size_t w_rows_alloc, int w_row0, const bf16* A, size_t a_rows_alloc, int a_row0,
          int M, int K, int R, const int* n_active, int mode, tc::Epi e, int a_parts = 1, int stacked = 1, int z_rows = 0,
          int z_w_rows = 0) {
  if (R <= 0) return;
  (void)w_rows_alloc;
  if (w_row0 % tc::BM != 0) { c->launch_error = FM_ERR_UNSUPPORTED; return; }
  const int tiles = (M + tc::BM - 1) / tc::BM, slabs = K / tc::BK;
  // Few rows: one N tile, K split over a cluster so that enough SMs stream weights.  Many rows:
  // N tiles of 32 rows as well (each weight slab then comes from HBM once and from L2 for the other
  // N tiles), which keeps the K split, and with it the cluster reduction, small.
  const int Rpad = round_up(R, 16);
  const int N = Rpad <= 32 ? Rpad : 32;
  const int n_tiles = stacked > 1 ? stacked : (Rpad + N - 1) / N;   // stacked problems share a launch through grid.z
  // K split: up to about one CTA per SM; while a CTA would still stream more than 8 slabs (or the
  // launch has several N tiles) up to two CTAs per SM, whose rings are then kept small enough to share it.
  const bool tiled = n_tiles > 1 && stacked == 1;
  int split = 1;
  while (split * 2 <= tc::MAX_SPLIT && split * 2 <= slabs) {
    const bool deep = tiled || slabs / split > 8;
    if (tiles * n_tiles * split * 2 > (deep ? c->split_target_deep : c->split_target)) break;
    split *= 2;
  }
  const int tA = tmap_for(c, A, a_rows_alloc, (uint64_t)K, N, (uint32_t)a_parts);
  if (tA < 0) { c->launch_error = FM_ERR_CUDA; return; }
  // only the residual and the QKV epilogue have side rows, and only when a thread gets more than two items
  const bool side = (mode == tc::EPI_RESID || mode == tc::EPI_QKV) && tc::side_bytes(N, split) > 0;
  const int side_b = side ? tc::side_bytes(N, split) : 0;
  int stages = tc::pick_stages(N, (slabs + split - 1) / split, a_parts, side_b);
  if (c->stage_cap > 0 && stages > c->stage_cap) stages = c->stage_cap;
  if (tiles * n_tiles * split > c->n_sm) {                 // two CTAs per SM: each at most 112 KB
    const int fit = (112 * 1024 - tc::smem_bytes(N, 0, a_parts, side_b)) / tc::stage_bytes(N, a_parts);
    stages = stages > fit ? (fit < 2 ? 2 : fit) : stages;
  }
  const long pi = prof_open(c, PROF_GEMM, 2.0 * M * K);            // algorithmic bytes: the weight matrix once
  tc::Args g{W, c->tmaps + tA, M, K, N, R, split, stages, a_parts, w_row0 / tc::BM, a_row0, stacked > 1 ? z_rows : 0,
             stacked > 1 ? z_w_rows / tc::BM : 0, n_active, c->st.status};
  e.row0 = 0;
  const int smem = tc::smem_bytes(N, stages, a_parts, side_b);
  const dim3 grid(tiles, split, n_tiles), cl(1, split, 1);
  c->cur_class = PROF_GEMM;
  if (c->only_class == PROF_GEMM) c->class_bytes += 2.0 * M * K * (stacked > 1 ? stacked : 1);
  switch (mode) {
    case tc::EPI_F32: launch_pdl(c, cl, tc::gemm_tc_kernel<tc::EPI_F32, false>, grid, 128, smem, g, e); break;
    case tc::EPI_BF16: launch_pdl(c, cl, tc::gemm_tc_kernel<tc::EPI_BF16, false>, grid, 128, smem, g, e); break;
    case tc::EPI_GELU: launch_pdl(c, cl, tc::gemm_tc_kernel<tc::EPI_GELU, false>, grid, 128, smem, g, e); break;
    case tc::EPI_RESID_CAT: launch_pdl(c, cl, tc::gemm_tc_kernel<tc::EPI_RESID_CAT, false>, grid, 128, smem, g, e); break;
    case tc::EPI_UP: launch_pdl(c, cl, tc::gemm_tc_kernel<tc::EPI_UP, false>, grid, 128, smem, g, e); break;
    case tc::EPI_RESID:
      if (side) launch_pdl(c, cl, tc::gemm_tc_kernel<tc::EPI_RESID, true>, grid, 128, smem, g, e);
      else launch_pdl(c, cl, tc::gemm_tc_kernel<tc::EPI_RESID, false>, grid, 128, smem, g, e);
      break;
    default:
      if (side) launch_pdl(c, cl, tc::gemm_tc_kernel<tc::EPI_QKV, true>, grid, 128, smem, g, e);
      else launch_pdl(c, cl, tc::gemm_tc_kernel<tc::EPI_QKV, false>, grid, 128, smem, g, e);
      break;
  }
  c->cur_class = PROF_OTHER;
  prof_close(c, pi);
  if ((mode == tc::EPI_RESID || mode == tc::EPI_RESID_CAT) && e.ssq_out != nullptr) c->ssq_n = tiles * split * (split == 1 ? 2 : 1);     // slots the next consumer adds
  if (mode == tc::EPI_UP && e.ssq_out != nullptr) c->ssq_n = (c->dm.d / tc::BM) * split * (split == 1 ? 2 : 1);   // tiles within d
}

// rows fed at each level in this pass (n_active[level]); n_active[3] = unfinished sequences
__global__ void row_count_kernel(Dims dm, SeqState st, int batch) {
  if (threadIdx.x == 0 && blockIdx.x == 0) count_rows(dm, st, batch);
}

// threads of a kernel that walks over one row of d values: one element per thread up to 512
inline int row_threads(int d) { return d >= 512 ? 512 : (d >= 256 ? 256 : 128); }
inline int accept_threads(int batch) { return batch >= 32 ? 1024 : 32 * (batch < 1 ? 1 : batch); }

void attention(fm_ctx* c, int level, const LayerDev& L) {
  const Dims& dm = c->dm;
  const int groups = c->attn_max_groups[level];
  AttnArgs a{dm, c->st, c->batch, level, c->qbuf, c->tmaps + L.tmK, c->tmaps + L.tmV, c->attn_part, c->attn_ticket,
             c->a_attn, c->attn_G[level], groups, c->attn_mt[level]};
  const dim3 grid(groups, dm.Hkv * c->attn_mt[level], c->batch);
  const long pi = prof_open(c, PROF_ATTN, 0.0);
  c->cur_class = PROF_ATTN;
  if (dm.dh == 64) launch_pdl(c, dim3(1, 1, 1), attn_stream_kernel<64, 128, 8>, grid, AttnCfg<64, 128, 8>::THREADS, AttnCfg<64, 128, 8>::BYTES, a);
  else launch_pdl(c, dim3(1, 1, 1), attn_stream_kernel<128, 64, 4>, grid, AttnCfg<128, 64, 4>::THREADS, AttnCfg<128, 64, 4>::BYTES, a);
  c->cur_class = PROF_OTHER;
  prof_close(c, pi);
}

inline size_t pad128(size_t v) { return align_up(v, 128); }

// One stack of pre-norm blocks on the rows of its level (a2/a4/a6/a8/a10): five launches per
// layer.  On entry c->a_norm (or `a_entry`) holds bf16(x * g1 of the first layer) and c->ssq the rows' sums of
// squares; on exit, if `want_a`, c->a_norm holds bf16(x * next_gain) (gain 1 when null) and c->ssq
// the sums of squares of the stack's output rows.
void run_stack(fm_ctx* c, int s, float* x, float* stash_ring, const float* next_gain, bool want_a, const tc::Epi* cat = nullptr,
               const bf16* a_entry = nullptr) {
  const Dims& dm = c->dm;
  const int level = STACK_LEVEL[s];
  const int rows = c->batch * fm_rows_per_seq(dm, level);
  const int qkvw = (dm.H + 2 * dm.Hkv) * dm.dh, hd = dm.H * dm.dh, d = dm.d;
  const size_t Rc_alloc = align_up((size_t)dm.max_batch * dm.R1, 16);
  const int* na = c->st.n_active + level;
  const int nl = (int)c->layers[s].size();
  for (int l = 0; l < nl; ++l) {
    const LayerDev& L = c->layers[s][l];
    tc::Epi eq{};
    if (stash_ring != nullptr && l == nl - 1) {          // split-node hiddens: the input of the stack's last layer
      eq.stash_x = x; eq.stash_ring = stash_ring; eq.stash_d = d; eq.stash_rs = fm_ring(level);
    }
    eq.ssq_in = c->ssq; eq.ssq_n = c->ssq_n; eq.ld_ssq = c->ssq_ld; eq.inv_d_in = 1.f / d; eq.eps = dm.eps;
    eq.dm = dm; eq.st = c->st; eq.batch = c->batch; eq.level = level; eq.rope_tab = c->rope_tab;
    eq.q_out = c->qbuf; eq.Kc = L.K; eq.Vc = L.V;
    eq.qscale = (float)(1.4426950408889634 / sqrt((double)dm.dh));   // 1/sqrt(dh) * log2(e)
    gemm(c, L.Wqkv, pad128(qkvw), 0, l == 0 && a_entry != nullptr ? a_entry : c->a_norm, Rc_alloc, 0, qkvw, d, rows, na, tc::EPI_QKV, eq, 2);
    attention(c, level, L);
    tc::Epi eo{};
    eo.x = x; eo.ldx = d; eo.add = 1; eo.gain = L.g2; eo.a_out = c->a_norm; eo.lda = 2 * d; eo.lo_off = d;
    eo.ssq_out = c->ssq; eo.ld_ssq_out = c->ssq_ld;
    gemm(c, L.Wo, pad128(d), 0, c->a_attn, Rc_alloc, 0, d, hd, rows, na, tc::EPI_RESID, eo, 2);
    tc::Epi e1 = epi_plain(c->a_ff, 2 * dm.dff);
    e1.lo_off = dm.dff;
    e1.ssq_in = c->ssq; e1.ssq_n = c->ssq_n; e1.ld_ssq = c->ssq_ld; e1.inv_d_in = 1.f / d; e1.eps = dm.eps;
    gemm(c, L.W1, pad128(dm.dff), 0, c->a_norm, Rc_alloc, 0, dm.dff, d, rows, na, tc::EPI_GELU, e1, 2);
    tc::Epi e2 = eo;
    const bool last = l == nl - 1;
    e2.gain = last ? next_gain : c->layers[s][l + 1].g1;
    if (last && !want_a) { e2.a_out = nullptr; e2.ssq_out = nullptr; }
    if (last && cat != nullptr) {                           // the stack below a shortening: hiddens leave through the epilogue
      e2.dm = dm; e2.st = c->st; e2.batch = c->batch; e2.level = level; e2.d_model = d;
      e2.cat_out = cat->cat_out; e2.cat_ring = cat->cat_ring; e2.cat_tri = cat->cat_tri;
      gemm(c, L.W2, pad128(d), 0, c->a_ff, Rc_alloc, 0, d, dm.dff, rows, na, tc::EPI_RESID_CAT, e2, 2);
      continue;
    }
    gemm(c, L.W2, pad128(d), 0, c->a_ff, Rc_alloc, 0, d, dm.dff, rows, na, tc::EPI_RESID, e2, 2);
  }
}

// the verify forward pass over st.cand / st.nrow (a1..a11)
void forward(fm_ctx* c, float* logits_out) {
  const Dims& dm = c->dm;
  const int B = c->batch, d = dm.d;
  const int Rc = B * dm.R1, Rv = B * dm.mv, Rf = B * dm.mf;
  const size_t Rc_alloc = align_up((size_t)dm.max_batch * dm.R1, 16), Rv_alloc = align_up((size_t)dm.max_batch * dm.mv, 16);
  const int* na = c->st.n_active;
  // The launch that opens a pass is a full barrier: the per-pass state (rows, lengths, row counts
  // -- every call that changes them ends with a row count -- and candidates) is final before any
  // later kernel's prologue can run.
  const size_t Rf_alloc = align_up((size_t)dm.max_batch * dm.mf, 16);
  tc::Epi es{};
  es.ldx = d; es.add = 0; es.a_out = c->a_norm; es.lda = 2 * d; es.lo_off = d;
  es.ssq_out = c->ssq; es.ld_ssq_out = c->ssq_ld;
  if (c->fuse_hourglass) {
    // Shorten and upsample inside the adjacent GEMMs.  Down: the epilogue of a down-stack's last layer
    // scatters the new hiddens into the shorten GEMM's concatenated operand rows and the carry ring
    // (the parts that precede the pass were laid down by the opening launch) and gives rows whose
    // parent belongs to an earlier pass that parent's stored slot.  Up: the upsampling GEMM's
    // epilogue adds slot r of parent u to child row 3u + r, whose residual row still holds the
    // pre-shorten hidden, and hands the child rows to the stack above.
    LAUNCH(c, embed_kernel, Rc + 3 * (Rv + Rf), row_threads(d), 0, dm, c->st, B, c->E, c->xc, c->layers[0][0].g1, c->a_norm, c->ssq, Rc,
           (const float*)c->hc_ring, (const float*)c->hv_ring, c->a_cat, c->a_cat2, Rv, Rf);
    c->ssq_n = 1;
    tc::Epi cat{};
    cat.cat_out = c->a_cat; cat.cat_ring = c->hc_ring; cat.cat_tri = c->triv_ring;
    run_stack(c, 0, c->xc, nullptr, nullptr, false, &cat);
    es.x = c->xv; es.gain = c->layers[1][0].g1;
    gemm(c, c->S_cv, pad128(d), 0, c->a_cat, Rv_alloc, 0, d, 3 * d, Rv, na + 1, tc::EPI_RESID, es, 2);
    cat.cat_out = c->a_cat2; cat.cat_ring = c->hv_ring; cat.cat_tri = c->trif_ring;
    run_stack(c, 1, c->xv, nullptr, nullptr, false, &cat);
    es.x = c->xf; es.gain = c->layers[2][0].g1;
    gemm(c, c->S_vf, pad128(d), 0, c->a_cat2, Rf_alloc, 0, d, 3 * d, Rf, na + 2, tc::EPI_RESID, es, 2);
    run_stack(c, 2, c->xf, c->zf, nullptr, true);                  // leaves bf16(xf) in a_norm
    tc::Epi eu{};
    eu.dm = dm; eu.st = c->st; eu.batch = B; eu.d_model = d;
    // (the child rows' operand goes to a buffer of its own: the launch is still reading its parent
    // rows from a_norm while the first epilogues write)
    eu.ldx = d; eu.a_out = c->a_up; eu.lda = 2 * d; eu.lo_off = d; eu.ssq_out = c->ssq; eu.ld_ssq_out = c->ssq_ld;
    eu.level = 2; eu.x = c->xv; eu.gain = c->layers[3][0].g1; eu.tri_ring = c->trif_ring;
    // (skipped only when the CHILD level has no rows: children whose parent is older than the pass
    // still need their operand rows and sums of squares)
    gemm(c, c->U_fv, pad128(3 * d), 0, c->a_norm, Rc_alloc, 0, 3 * d, d, Rf, na + 1, tc::EPI_UP, eu, 2);
    run_stack(c, 3, c->xv, c->zv, nullptr, true, nullptr, c->a_up);   // leaves bf16(xv) in a_norm
    eu.level = 1; eu.x = c->xc; eu.gain = c->layers[4][0].g1; eu.tri_ring = c->triv_ring;
    gemm(c, c->U_vc, pad128(3 * d), 0, c->a_norm, Rc_alloc, 0, 3 * d, d, Rv, na, tc::EPI_UP, eu, 2);
  } else {
    LAUNCH(c, embed_kernel, Rc, row_threads(d), 0, dm, c->st, B, c->E, c->xc, c->layers[0][0].g1, c->a_norm, c->ssq, Rc,
           (const float*)nullptr, (const float*)nullptr, (bf16*)nullptr, (bf16*)nullptr, 0, 0);
    c->ssq_n = 1;
    run_stack(c, 0, c->xc, nullptr, nullptr, false);
    launch_pdl(c, dim3(1, 1, 1), shorten_gather_kernel, dim3(Rv + Rc, 3), row_threads(d), 0, dm, c->st, B, 1, (const float*)c->xc, c->hc_ring, c->a_cat, Rv);
    es.x = c->xv; es.gain = c->layers[1][0].g1;
    gemm(c, c->S_cv, pad128(d), 0, c->a_cat, Rv_alloc, 0, d, 3 * d, Rv, na + 1, tc::EPI_RESID, es, 2);
    run_stack(c, 1, c->xv, nullptr, nullptr, false);
    launch_pdl(c, dim3(1, 1, 1), shorten_gather_kernel, dim3(Rf + Rv, 3), row_threads(d), 0, dm, c->st, B, 2, (const float*)c->xv, c->hv_ring, c->a_cat, Rf);
    es.x = c->xf; es.gain = c->layers[2][0].g1;
    gemm(c, c->S_vf, pad128(d), 0, c->a_cat, Rv_alloc, 0, d, 3 * d, Rf, na + 2, tc::EPI_RESID, es, 2);
    run_stack(c, 2, c->xf, c->zf, nullptr, true);                  // leaves bf16(xf) in a_norm
    gemm(c, c->U_fv, pad128(3 * d), 0, c->a_norm, Rc_alloc, 0, 3 * d, d, Rf, na + 2, tc::EPI_F32, epi_plain(c->tmp3d, 3 * d), 2);
    launch_pdl(c, dim3(1, 1, 1), upsample_add_kernel, Rv + Rf, row_threads(d), 0, dm, c->st, B, 1, (const float*)c->hv_ring, (const float*)c->tmp3d,
               c->trif_ring, c->xv, (const float*)c->layers[3][0].g1, c->a_norm, c->ssq, Rv);
    c->ssq_n = 1;
    run_stack(c, 3, c->xv, c->zv, nullptr, true);                  // leaves bf16(xv) in a_norm
    gemm(c, c->U_vc, pad128(3 * d), 0, c->a_norm, Rc_alloc, 0, 3 * d, d, Rv, na + 1, tc::EPI_F32, epi_plain(c->tmp3d, 3 * d), 2);
    launch_pdl(c, dim3(1, 1, 1), upsample_add_kernel, Rc + Rv, row_threads(d), 0, dm, c->st, B, 0, (const float*)c->hc_ring, (const float*)c->tmp3d,
               c->triv_ring, c->xc, (const float*)c->layers[4][0].g1, c->a_norm, c->ssq, Rc);
    c->ssq_n = 1;
  }
  run_stack(c, 4, c->xc, c->zc, c->g_out, true, nullptr, c->fuse_hourglass ? c->a_up : nullptr);   // leaves bf16(xc * g_out) and its sums of squares
  tc::Epi el = epi_plain(c->logits, dm.Vpad);
  el.ssq_in = c->ssq; el.ssq_n = c->ssq_n; el.ld_ssq = c->ssq_ld; el.inv_d_in = 1.f / d; el.eps = dm.eps;
  gemm(c, c->W_out, dm.Vpad, 0, c->a_norm, Rc_alloc, 0, dm.V, d, Rc, na, tc::EPI_F32, el, 2);
  launch_pdl(c, dim3(1, 1, 1), verify_top2_kernel, Rc, 256, 0, dm, c->st, B, (const float*)c->logits, logits_out);
}

// T problems of the same shape in one launch (grid.z): set t multiplies weight matrix t of the stacked
// buffer W (Mpad rows each) with operand rows [t*max_batch, t*max_batch + batch) and writes the same
// rows of the output.  More than 32 sequences: one launch per set.
void gemm_sets(fm_ctx* c, const bf16* W, int Mpad, int M, int K, const bf16* A, int a_parts, int T, int mode, tc::Epi e) {
  const Dims& dm = c->dm;
  const int B = c->batch, MB = dm.max_batch;
  const size_t a_rows = (size_t)c->draft_sets * MB + 16;
  const int* na = c->st.n_active + 3;
  const size_t esz = (mode == tc::EPI_F32) ? 4 : 2;
  if (T <= 0) return;
  if (B <= 32) {
    gemm(c, W, (size_t)T * Mpad, 0, A, a_rows, 0, M, K, B, na, mode, e, a_parts, T, MB, Mpad);
    return;
  }
  for (int t = 0; t < T; ++t) {
    tc::Epi et = e;
    et.out = static_cast<char*>(e.out) + (size_t)t * MB * e.ldo * esz;
    gemm(c, W, (size_t)T * Mpad, t * Mpad, A, a_rows, t * MB, M, K, B, na, mode, et, a_parts);
  }
}

// attention of nq draft queries per sequence over the cache of the last layer of stack s; the
// result of query r of sequence b goes to row r * max_batch + b of `out`
void attention_draft(fm_ctx* c, int s, int nq, const bf16* q, bf16* out) {
  const Dims& dm = c->dm;
  const int level = STACK_LEVEL[s];
  const LayerDev& L = c->layers[s].back();
  const int groups = c->attn_max_groups[level];
  const int MT = (nq * (dm.H / dm.Hkv) + 15) / 16;
  if (MT > c->attn_mt_draft[level] && MT > c->attn_mt[level]) { c->launch_error = FM_ERR_CAPACITY; return; }
  AttnArgs a{dm, c->st, c->batch, level, q, c->tmaps + L.tmK, c->tmaps + L.tmV, c->attn_part, c->attn_ticket,
             out, c->attn_G[level], groups, MT, nq, dm.max_batch};
  const dim3 grid(groups, dm.Hkv * MT, c->batch);
  c->cur_class = PROF_ATTN;
  if (dm.dh == 64) launch_pdl(c, dim3(1, 1, 1), attn_stream_kernel<64, 128, 8>, grid, AttnCfg<64, 128, 8>::THREADS, AttnCfg<64, 128, 8>::BYTES, a);
  else launch_pdl(c, dim3(1, 1, 1), attn_stream_kernel<128, 64, 4>, grid, AttnCfg<128, 64, 4>::THREADS, AttnCfg<128, 64, 4>::BYTES, a);
  c->cur_class = PROF_OTHER;
}

// One stage of HF-Blocks (Eq. 3-5) on the fp32 features hf_feature() names: T offsets, each with its
// own W_q, FFN and gain; k = 0: vertex level (cache of the vertex-up stack), 1: coordinate level.
void hf_stage(fm_ctx* c, int k) {
  const Dims& dm = c->dm;
  const int B = c->batch, d = dm.d, hd = dm.H * dm.dh, T = c->hf_T[k];
  if (T <= 0) return;
  const int stage = k == 0 ? DS_HF_V : DS_HF_C, s = k == 0 ? 3 : 4;
  const int hdp = round_up(hd, 128), dp = round_up(d, 128), hfp = round_up(dm.hf, 128);
  const float qscale = (float)(1.4426950408889634 / sqrt((double)dm.dh));
  launch_pdl(c, dim3(1, 1, 1), hf_prep_kernel, dim3(B, T), 256, 0, dm, c->st, B, stage, c->xv_pre, c->feat, (const float*)c->hf_g[k], c->d_a);
  gemm_sets(c, c->hfWq[k], hdp, hd, d, c->d_a, 1, T, tc::EPI_F32, epi_plain(c->d_qf, hd));
  launch_pdl(c, dim3(1, 1, 1), draft_q_kernel, dim3(B, T), 256, 0, dm, c->st, B, stage, STACK_LEVEL[s], 0, T, (const float*)c->d_qf,
             (const float2*)c->rope_tab, qscale, c->d_q);
  attention_draft(c, s, T, c->d_q, c->d_attn);
  tc::Epi e1 = epi_plain(c->d_h1, 2 * dm.hf);
  e1.lo_off = dm.hf;
  gemm_sets(c, c->hfW1[k], hfp, dm.hf, hd, c->d_attn, 2, T, tc::EPI_GELU, e1);
  gemm_sets(c, c->hfW2[k], dp, d, dm.hf, c->d_h1, 2, T, tc::EPI_F32, epi_plain(c->d_out, d));
  launch_pdl(c, dim3(1, 1, 1), hf_finish_kernel, dim3(B, T), 256, 0, dm, c->st, B, stage, c->xv_pre, c->feat, (const float*)c->d_out, c->up_in_v);
}

// a13: draft modules on the stashed split-node hiddens.  Reduced heads: SP = h + A rms(h), the
// upsample matrices alone.  Full: the SP-Blocks' attention before the linear layer and an HF-Block
// after every upsample (Sec. 3.1, Eq. 1-5; supplement "Three-Level Speculative Decoding").
void draft(fm_ctx* c, float* logits_out, float* margin_out, const GenOut* gen) {
  const Dims& dm = c->dm;
  const int B = c->batch, d = dm.d;
  if (dm.D > 0) {
    const int dpad = round_up(d, 128), hd = dm.H * dm.dh;
    const int NF = dm.nc + 3 * dm.nv + 9 * dm.Ef, NP = dm.nv + 3 * dm.Ef;
    const int* na = c->st.n_active + 3;
    const size_t MB = dm.max_batch;
    if (dm.full) {
      // SP-Block attention: a = rms(z, ga); q = Wq a at the split node's position; o over the cache of
      // the level's last layer; u = Wo o; then the head's input is rms(z + u, g) instead of rms(z, g)
      const float qscale = (float)(1.4426950408889634 / sqrt((double)dm.dh));
      LAUNCH(c, draft_prep_kernel, dim3(B, dm.NH), 256, 0, dm, c->st, B, c->zc, c->zv, c->zf, c->sp_ga, c->d_a);
      gemm_sets(c, c->spWq, round_up(hd, 128), hd, d, c->d_a, 1, dm.NH, tc::EPI_F32, epi_plain(c->d_qf, hd));
      const int cnt[3] = {dm.nc, dm.nv, dm.Ef}, stack_of[3] = {4, 3, 2};
      int h0 = 0;
      for (int l = 0; l < 3; ++l) {
        if (cnt[l] > 0) {
          bf16* ql = c->d_q + (size_t)h0 * MB * hd;           // this level's queries, rows (b * cnt + r)
          launch_pdl(c, dim3(1, 1, 1), draft_q_kernel, dim3(B, cnt[l]), 256, 0, dm, c->st, B, (int)DS_SP, l, h0, cnt[l], (const float*)c->d_qf,
                     (const float2*)c->rope_tab, qscale, ql);
          attention_draft(c, stack_of[l], cnt[l], ql, c->d_attn + (size_t)h0 * MB * 2 * hd);
        }
        h0 += cnt[l];
      }
      gemm_sets(c, c->spWo, dpad, d, hd, c->d_attn, 2, dm.NH, tc::EPI_F32, epi_plain(c->d_out, d));
      launch_pdl(c, dim3(1, 1, 1), sp_mid_kernel, dim3(B, dm.NH), 256, 0, dm, c->st, B, (const float*)c->zc, (const float*)c->zv,
                 (const float*)c->zf, (const float*)c->d_out, (const float*)c->head_g, c->dh_a);
    } else {
      LAUNCH(c, draft_prep_kernel, dim3(B, dm.NH), 256, 0, dm, c->st, B, c->zc, c->zv, c->zf, c->head_g, c->dh_a);
    }
    if (B <= 32) {                                               // the NH head matrices as one launch
      gemm(c, c->headA, (size_t)dm.NH * dpad, 0, c->dh_a, (size_t)dm.NH * MB + 16, 0, d, d, B, na, tc::EPI_F32, epi_plain(c->dh_y, d), 1,
           dm.NH, (int)MB, dpad);
    } else {
      for (int h = 0; h < dm.NH; ++h)
        gemm(c, c->headA, (size_t)dm.NH * dpad, h * dpad, c->dh_a, (size_t)dm.NH * MB + 16, h * (int)MB, d, d, B, na, tc::EPI_F32,
             epi_plain(c->dh_y + (size_t)h * MB * d, d));
    }
    launch_pdl(c, dim3(1, 1, 1), draft_residual_kernel, dim3(B, dm.NH), 128, 0, dm, c->st, B, (const float*)c->zc, (const float*)c->zv,
               (const float*)c->zf, (const float*)c->dh_y, c->feat, c->up_in_v, c->up_in_f);
    if (dm.Ef > 0) {
      if (dm.full) {                                             // face -> 3 vertices, each refined at the vertex level
        gemm(c, c->U_fv, pad128(3 * d), 0, c->up_in_f, align_up((size_t)dm.Ef * MB + 1, 16), 0, 3 * d, d, dm.Ef * B, na, tc::EPI_F32,
             epi_plain(c->xv_pre, 3 * d));
        hf_stage(c, 0);
      } else {
        gemm(c, c->U_fv, pad128(3 * d), 0, c->up_in_f, align_up((size_t)dm.Ef * MB + 1, 16), 0, 3 * d, d, dm.Ef * B, na, tc::EPI_BF16,
             epi_plain(c->up_in_v + (size_t)dm.nv * B * d, 3 * d));
      }
    }
    if (NP > 0) {
      gemm(c, c->U_vc, pad128(3 * d), 0, c->up_in_v, align_up((size_t)NP * MB + 1, 16), 0, 3 * d, d, NP * B, na,
           tc::EPI_F32, epi_plain(c->feat + (size_t)dm.nc * B * d, 3 * d));
      if (dm.full) hf_stage(c, 1);                               // every upsampled coordinate feature refined at the coordinate level
    }
    launch_pdl(c, dim3(1, 1, 1), rmsnorm_kernel, NF * B, 256, 0, (const float*)c->feat, (const float*)c->g_out, c->feat_n, d, dm.eps);
    gemm(c, c->W_out, dm.Vpad, 0, c->feat_n, align_up((size_t)NF * MB, 16), 0, dm.V, d, NF * B, na, tc::EPI_F32,
         epi_plain(c->dlogits, dm.Vpad));
  }
  const bool lab = dm.has_label != 0 && dm.D > 0;
  launch_pdl(c, dim3(1, 1, 1), draft_pick_kernel, dim3(B, dm.R1), 256, 0, dm, c->st, B, (const float*)c->dlogits, logits_out, margin_out, gen,
             (const bf16*)c->up_in_v, (const float*)c->label_g, (const float*)c->label_W, lab ? c->labels : (int*)nullptr, c->label_margin,
             c->avg_rows);
}

__global__ void verify_load_kernel(Dims dm, SeqState st, int batch, const int* __restrict__ cand) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= batch * dm.R1) return;
  const int b = i / dm.R1, j = i - b * dm.R1;
  const int t = cand[i];
  if (j == 0 && st.nrow[b] > 0 && t != st.main_tok[b]) atomicExch(st.status, FM_ERR_INVALID_ARG);
  st.cand[i] = t;
}

// candidates of a host-driven pass: the host's entry where it gave one (>= 0), else the draft modules'
__global__ void step_merge_kernel(Dims dm, SeqState st, int batch, const int* __restrict__ host_cand, int* __restrict__ out) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= batch * dm.R1) return;
  const int h = host_cand != nullptr ? host_cand[i] : -1;
  out[i] = (h >= 0 && i % dm.R1 != 0) ? h : st.cand[i];          // slot 0 is always the pending main token
}

__global__ void init_state_kernel(Dims dm, SeqState st, int batch, const int* __restrict__ prompt_off) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= dm.max_batch) return;
  st.L[b] = 0; st.nrow[b] = 0; st.main_tok[b] = dm.n_bins + 2; st.done[b] = b < batch ? 0 : 1;
  st.plen[b] = b < batch ? prompt_off[b + 1] - prompt_off[b] : 0;
  st.t_end[b] = dm.max_tokens - dm.D - 2;
  if (b == 0) { *st.step = 0; }
}

__global__ void set_limits_kernel(Dims dm, SeqState st, int batch, const int* __restrict__ max_faces) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= batch) return;
  const int cap = dm.max_tokens - dm.D - 2;
  const long long want = (long long)st.plen[b] + 9ll * max_faces[b];
  st.t_end[b] = want < cap ? (int)want : cap;
}

// one decode pass of fm_generate
void step_body(fm_ctx* c) {
  const Dims& dm = c->dm;
  draft(c, nullptr, nullptr, (const GenOut*)c->gen_dev);
  forward(c, nullptr);
  LAUNCH(c, accept_kernel, 1, accept_threads(c->batch), 0, dm, c->st, c->batch, (const int*)nullptr, (const int*)nullptr,
         (int*)nullptr, (int*)nullptr, (int*)nullptr, (const GenOut*)c->gen_dev, 1);
}

void drop_graph(fm_ctx* c) {
  if (c->graph_exec != nullptr) cudaGraphExecDestroy(c->graph_exec);
  if (c->graph != nullptr) cudaGraphDestroy(c->graph);
  c->graph_exec = nullptr;
  c->graph = nullptr;
}

void drop_call_graph(fm_ctx::CallGraph& g) {
  if (g.exec != nullptr) cudaGraphExecDestroy(g.exec);
  g.exec = nullptr;
  g.valid = false;
  g.batch = -1;
}

// Runs `body` (which only enqueues work on the context's stream).  The first time a set of caller
// pointers is seen the kernels are launched one by one (this also creates every descriptor the
// path needs); when the same pointers come again the launches are captured into a graph, and
// from then on the graph is replayed: a pass is 180 launches, and a host that drives the loop
// call by call would otherwise pay for each of them.  All state the kernels read lives in device
// memory, so the same graph serves every pass.
template <typename F>
void run_cached(fm_ctx* c, fm_ctx::CallGraph& g, const void* k0, const void* k1, const void* k2, const void* k3, F&& body) {
  const bool off = c->call_graphs_off || c->graph_unavailable || c->debug_sync || c->prof_on || g.failed;
  const bool same = g.valid && g.batch == c->batch && g.key[0] == k0 && g.key[1] == k1 && g.key[2] == k2 && g.key[3] == k3;
  if (off) { body(); return; }
  if (same && g.exec != nullptr) {
    if (cudaGraphLaunch(g.exec, c->stream) != cudaSuccess) { cudaGetLastError(); c->launch_error = FM_ERR_CUDA; }
    c->launches += g.launches;
    return;
  }
  if (!same) {
    drop_call_graph(g);
    g.key[0] = k0; g.key[1] = k1; g.key[2] = k2; g.key[3] = k3;
    g.batch = c->batch;
    g.valid = true;
    body();
    return;
  }
  // same pointers as last time and no graph yet: capture
  if (cudaStreamBeginCapture(c->stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
    cudaGetLastError();
    g.failed = true;
    body();
    return;
  }
  const int64_t l0 = c->launches;
  c->capturing = true;
  body();
  c->capturing = false;
  g.launches = c->launches - l0;
  c->launches = l0;
  cudaGraph_t gr = nullptr;
  if (cudaStreamEndCapture(c->stream, &gr) != cudaSuccess || gr == nullptr || c->launch_error != FM_OK ||
      cudaGraphInstantiate(&g.exec, gr, 0) != cudaSuccess) {
    cudaGetLastError();
    if (gr != nullptr) cudaGraphDestroy(gr);
    g.exec = nullptr;
    g.failed = true;
    c->launch_error = FM_OK;
    body();                                          // nothing ran during the failed capture
    return;
  }
  cudaGraphDestroy(gr);
  if (cudaGraphLaunch(g.exec, c->stream) != cudaSuccess) { cudaGetLastError(); c->launch_error = FM_ERR_CUDA; }
  c->launches += g.launches;
}

// Capture the pass once per batch size.  All state the kernels read lives in device memory, so the
// same graph serves every pass.  Streams that cannot be captured (the legacy default stream) fall
// back to plain launches of the same kernels.
void ensure_graph(fm_ctx* c) {
  if (c->graph_unavailable || (c->graph_exec != nullptr && c->graph_batch == c->batch)) return;
  drop_graph(c);
  draft(c, nullptr, nullptr, nullptr);             // makes the draft path's TMA descriptors exist
  cudaStreamSynchronize(c->stream);
  if (cudaStreamBeginCapture(c->stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
    cudaGetLastError();
    c->graph_unavailable = true;
    return;
  }
  const int64_t l0 = c->launches;
  c->capturing = true;
  step_body(c);
  c->capturing = false;
  c->graph_launches = c->launches - l0;
  c->launches = l0;
  cudaGraph_t g = nullptr;
  if (cudaStreamEndCapture(c->stream, &g) != cudaSuccess || g == nullptr || c->launch_error != FM_OK) {
    cudaGetLastError();
    if (g != nullptr) cudaGraphDestroy(g);
    c->graph_unavailable = true;
    c->launch_error = FM_OK;
    return;
  }
  c->graph = g;
  if (cudaGraphInstantiate(&c->graph_exec, g, 0) != cudaSuccess) {
    cudaGetLastError();
    drop_graph(c);
    c->graph_unavailable = true;
    return;
  }
  c->graph_batch = c->batch;
}

}  // namespace

// ------------------------------------------------------------------------------------------
// C ABI
// ------------------------------------------------------------------------------------------
extern "C" {

const char* fm_strerror(int code) {
  switch (code) {
    case FM_OK: return "ok";
    case FM_ERR_INVALID_ARG: return "invalid argument";
    case FM_ERR_BAD_STATE: return "call out of order";
    case FM_ERR_CAPACITY: return "capacity exceeded";
    case FM_ERR_CUDA: return "CUDA runtime error";
    case FM_ERR_TIMEOUT: return "device-side wait timed out";
    case FM_ERR_UNSUPPORTED: return "unsupported shape";
    default: return "unknown error";
  }
}

size_t fm_workspace_bytes(const fm_config* cfg) {
  if (check_config(cfg) != FM_OK) return 0;
  fm_ctx tmp{};
  tmp.cfg = *cfg;
  tmp.dm = make_dims(*cfg);
  Carver cv{nullptr, 0};
  carve(&tmp, cv);
  return cv.off;
}

int fm_create(const fm_config* cfg, const fm_weights* w, void* dev_workspace, size_t workspace_bytes, void* cuda_stream,
              fm_ctx** out) {
  if (out == nullptr) return FM_ERR_INVALID_ARG;
  *out = nullptr;
  int rc = check_config(cfg);
  if (rc != FM_OK) return rc;
  if (w == nullptr || dev_workspace == nullptr) return FM_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(dev_workspace) & 255u) != 0) return FM_ERR_INVALID_ARG;
  const size_t need = fm_workspace_bytes(cfg);
  if (workspace_bytes < need) return FM_ERR_CAPACITY;
  for (int s = 0; s < 5; ++s) if (w->stack[s] == nullptr) return FM_ERR_INVALID_ARG;

  fm_ctx* c = new (std::nothrow) fm_ctx{};
  if (c == nullptr) return FM_ERR_INVALID_ARG;
  c->cfg = *cfg;
  c->dm = make_dims(*cfg);
  c->stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  c->ws = static_cast<char*>(dev_workspace);
  c->ws_bytes = need;
  Carver cv{c->ws, 0};
  carve(c, cv);
  const Dims& dm = c->dm;
  const size_t d = dm.d, qkvw = (size_t)(dm.H + 2 * dm.Hkv) * dm.dh, hd = (size_t)dm.H * dm.dh;

#define TRY(expr) do { rc = (expr); if (rc != FM_OK) { delete c; return rc; } } while (0)
#define TRYCUDA(expr) do { if ((expr) != cudaSuccess) { delete c; return FM_ERR_CUDA; } } while (0)
  // everything that is not explicitly uploaded (row padding, caches, rings, state) starts at zero
  TRYCUDA(cudaMemset(c->ws, 0, need));
  std::vector<uint16_t> tmp;
  TRY(upload_bf16(c->E, w->E, (size_t)dm.V * d, tmp));
  for (int s = 0; s < 5; ++s)
    for (size_t l = 0; l < c->layers[s].size(); ++l) {
      const fm_layer_weights& hw = w->stack[s][l];
      LayerDev& L = c->layers[s][l];
      TRY(upload_packed(L.Wqkv, hw.Wqkv, qkvw, d, tmp));
      TRY(upload_packed(L.Wo, hw.Wo, d, hd, tmp));
      TRY(upload_packed(L.W1, hw.W1, (size_t)dm.dff, d, tmp));
      TRY(upload_packed(L.W2, hw.W2, d, (size_t)dm.dff, tmp));
      TRY(upload_f32(L.g1, hw.g1, d));
      TRY(upload_f32(L.g2, hw.g2, d));
    }
  TRY(upload_packed(c->S_cv, w->S_cv, d, 3 * d, tmp));
  TRY(upload_packed(c->S_vf, w->S_vf, d, 3 * d, tmp));
  TRY(upload_packed(c->U_fv, w->U_fv, 3 * d, d, tmp));
  TRY(upload_packed(c->U_vc, w->U_vc, 3 * d, d, tmp));
  TRY(upload_packed(c->W_out, w->W_out, (size_t)dm.V, d, tmp));
  TRY(upload_f32(c->g_out, w->g_out, d));
  const size_t dpad = align_up(d, 128);
  for (int h = 0; h < dm.NH && dm.D > 0; ++h) {
    const fm_sp_weights* group = h < dm.nc ? w->heads_c : h < dm.nc + dm.nv ? w->heads_v : w->heads_f;
    if (group == nullptr) { delete c; return FM_ERR_INVALID_ARG; }
    const fm_sp_weights& sp = group[h < dm.nc ? h : h < dm.nc + dm.nv ? h - dm.nc : h - dm.nc - dm.nv];
    TRY(upload_packed(c->headA + (size_t)h * dpad * d, sp.A, d, d, tmp));
    TRY(upload_f32(c->head_g + (size_t)h * d, sp.g, d));
  }
  if (dm.full && dm.D > 0) {
    const size_t hdp = align_up(hd, 128), hfp = align_up((size_t)dm.hf, 128);
    for (int h = 0; h < dm.NH; ++h) {
      const fm_sp_weights* group = h < dm.nc ? w->heads_c : h < dm.nc + dm.nv ? w->heads_v : w->heads_f;
      const fm_sp_weights& sp = group[h < dm.nc ? h : h < dm.nc + dm.nv ? h - dm.nc : h - dm.nc - dm.nv];
      TRY(upload_packed(c->spWq + (size_t)h * hdp * d, sp.Wq, hd, d, tmp));
      TRY(upload_packed(c->spWo + (size_t)h * dpad * hd, sp.Wo, d, hd, tmp));
      TRY(upload_f32(c->sp_ga + (size_t)h * d, sp.ga, d));
    }
    for (int k = 0; k < 2; ++k)
      for (int t = 0; t < c->hf_T[k]; ++t) {
        const fm_hf_weights* arr = k == 0 ? w->hf_fv : (t < 3 * dm.nv ? w->hf_vc : w->hf_fc);
        if (arr == nullptr) { delete c; return FM_ERR_INVALID_ARG; }
        const fm_hf_weights& hb = arr[k == 0 ? t : (t < 3 * dm.nv ? t : t - 3 * dm.nv)];
        TRY(upload_packed(c->hfWq[k] + (size_t)t * hdp * d, hb.Wq, hd, d, tmp));
        TRY(upload_packed(c->hfW1[k] + (size_t)t * hfp * hd, hb.W1, (size_t)dm.hf, hd, tmp));
        TRY(upload_packed(c->hfW2[k] + (size_t)t * dpad * dm.hf, hb.W2, d, (size_t)dm.hf, tmp));
        TRY(upload_f32(c->hf_g[k] + (size_t)t * d, hb.g, d));
      }
  }
  if (w->label_g != nullptr && w->label_W != nullptr && dm.nv > 0) {
    TRY(upload_f32(c->label_g, w->label_g, d));
    TRY(upload_f32(c->label_W, w->label_W, 3 * d));
    c->dm.has_label = 1;
  }
  // TMA descriptors of the KV caches: each cache is a 2-D [max_batch*Hkv*slots, dh] bf16 matrix
  for (int s = 0; s < 5; ++s)
    for (auto& L : c->layers[s]) {
      const uint64_t rows = (uint64_t)dm.max_batch * dm.Hkv * (dm.P + dm.cap[STACK_LEVEL[s]]);
      const uint32_t box = (uint32_t)c->attn_chunk;
      L.tmK = add_tmap_bf16(c, L.K, rows, dm.dh, box);
      c->tmap_keys.push_back({L.K, rows, (uint64_t)dm.dh, box, 0u});
      L.tmV = add_tmap_bf16(c, L.V, rows, dm.dh, box);
      c->tmap_keys.push_back({L.V, rows, (uint64_t)dm.dh, box, 0u});
      if (L.tmK < 0 || L.tmV < 0) { delete c; return FM_ERR_CUDA; }
    }
  TRYCUDA(cudaMemcpy(c->tmaps, c->tmaps_host.data(), c->tmaps_host.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice));
  TRYCUDA(cudaFuncSetAttribute(tc::gemm_tc_kernel<tc::EPI_F32, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::max_smem_bytes()));
  TRYCUDA(cudaFuncSetAttribute(tc::gemm_tc_kernel<tc::EPI_BF16, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::max_smem_bytes()));
  TRYCUDA(cudaFuncSetAttribute(tc::gemm_tc_kernel<tc::EPI_GELU, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::max_smem_bytes()));
  TRYCUDA(cudaFuncSetAttribute(tc::gemm_tc_kernel<tc::EPI_RESID, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::max_smem_bytes()));
  TRYCUDA(cudaFuncSetAttribute(tc::gemm_tc_kernel<tc::EPI_QKV, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::max_smem_bytes()));
  TRYCUDA(cudaFuncSetAttribute(tc::gemm_tc_kernel<tc::EPI_RESID, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::max_smem_bytes()));
  TRYCUDA(cudaFuncSetAttribute(tc::gemm_tc_kernel<tc::EPI_RESID_CAT, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::max_smem_bytes()));
  TRYCUDA(cudaFuncSetAttribute(tc::gemm_tc_kernel<tc::EPI_UP, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::max_smem_bytes()));
  TRYCUDA(cudaFuncSetAttribute(tc::gemm_tc_kernel<tc::EPI_QKV, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::max_smem_bytes()));
  TRYCUDA(cudaFuncSetAttribute(attn_stream_kernel<64, 128, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnCfg<64, 128, 8>::BYTES));
  TRYCUDA(cudaFuncSetAttribute(attn_stream_kernel<128, 64, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnCfg<128, 64, 4>::BYTES));
  std::vector<double> freq(dm.dh / 2);
  for (int i = 0; i < dm.dh / 2; ++i)
    freq[i] = dm.theta != 0.f ? pow((double)dm.theta, -2.0 * (double)i / (double)dm.dh) : 0.0;
  TRYCUDA(cudaMemcpy(c->inv_freq, freq.data(), freq.size() * sizeof(double), cudaMemcpyHostToDevice));
  {
    const size_t n = (size_t)(dm.max_tokens + 1 + FM_ROPE_SLACK) * (dm.dh / 2);
    rope_table_kernel<<<(unsigned)((n + 255) / 256), 256, 0, c->stream>>>(c->rope_tab, c->inv_freq, dm.max_tokens + 1 + FM_ROPE_SLACK, dm.dh / 2);
    TRYCUDA(cudaGetLastError());
  }
  TRYCUDA(cudaHostAlloc(reinterpret_cast<void**>(&c->host_done), 64, cudaHostAllocMapped));
  *c->host_done = 0;
  TRYCUDA(cudaHostGetDevicePointer(reinterpret_cast<void**>(&c->host_done_dev), c->host_done, 0));
  TRYCUDA(cudaDeviceSynchronize());
#undef TRY
#undef TRYCUDA
  c->batch = 0;
  c->phase = 0;
  c->launches = 0;
  c->only_class = -1;
  c->cur_class = PROF_OTHER;
  {
    const char* v = getenv("FM_NO_PDL");
    c->use_pdl = !(v != nullptr && v[0] == '1');
    const char* ds = getenv("FM_DEBUG_SYNC");
    c->debug_sync = ds != nullptr && ds[0] == '1';
    const char* ncg = getenv("FM_NO_CALL_GRAPH");
    c->call_graphs_off = ncg != nullptr && ncg[0] == '1';
    const char* t = getenv("FM_SPLIT_TARGET");
    c->split_target = t != nullptr && atoi(t) > 0 ? atoi(t) : 160;
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    c->n_sm = sms > 0 ? sms : 148;
    c->device = dev;
    const char* tt = getenv("FM_SPLIT_TARGET_DEEP");
    c->split_target_deep = tt != nullptr && atoi(tt) > 0 ? atoi(tt) : 296;
    const char* nf = getenv("FM_NO_FUSE");
    // (the upsampling epilogue lists at most 128 carried rows per slot: one per sequence)
    c->fuse_hourglass = c->dm.d % tc::BM == 0 && c->dm.max_batch <= 128 && !(nf != nullptr && nf[0] == '1');
    const char* sc = getenv("FM_STAGE_CAP");
    c->stage_cap = sc != nullptr ? atoi(sc) : 4;        // measured: deeper rings cost more than they prefetch
  }
  *out = c;
  return FM_OK;
}

int fm_profile_begin(fm_ctx* c) {
  if (c == nullptr) return FM_ERR_INVALID_ARG;
  if (c->prof_ev.empty()) {
    const size_t pairs = 4096;
    c->prof_ev.resize(2 * pairs);
    c->prof_cls.assign(pairs, 0);
    for (auto& e : c->prof_ev) CUDA_OK(cudaEventCreate(&e));
  }
  c->prof_used = 0;
  for (int i = 0; i < 3; ++i) { c->prof_ms[i] = 0; c->prof_bytes[i] = 0; c->prof_n[i] = 0; }
  c->prof_on = true;
  return FM_OK;
}

int fm_profile_end(fm_ctx* c, fm_profile* out) {
  if (c == nullptr || out == nullptr) return FM_ERR_INVALID_ARG;
  prof_drain(c);
  c->prof_on = false;
  out->gemm_ms = c->prof_ms[PROF_GEMM]; out->gemm_bytes = c->prof_bytes[PROF_GEMM]; out->gemm_launches = c->prof_n[PROF_GEMM];
  out->attn_ms = c->prof_ms[PROF_ATTN]; out->attn_launches = c->prof_n[PROF_ATTN];
  return FM_OK;
}

int fm_profile_class(fm_ctx* c, int32_t cls, int32_t reps, fm_profile* out) {
  if (c == nullptr || out == nullptr || reps < 1 || (cls != PROF_GEMM && cls != PROF_ATTN)) return FM_ERR_INVALID_ARG;
  if (c->phase < 1) return FM_ERR_BAD_STATE;
  memset(out, 0, sizeof(*out));
  CUDA_OK(cudaStreamSynchronize(c->stream));
  if (cudaStreamBeginCapture(c->stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) { cudaGetLastError(); return FM_ERR_CUDA; }
  const int64_t l0 = c->launches;
  c->only_class = cls;
  c->class_bytes = 0.0;
  c->capturing = true;
  forward(c, nullptr);
  c->capturing = false;
  c->only_class = -1;
  const int64_t n_launch = c->launches - l0;
  c->launches = l0;
  cudaGraph_t g = nullptr;
  cudaGraphExec_t ge = nullptr;
  if (cudaStreamEndCapture(c->stream, &g) != cudaSuccess || g == nullptr || c->launch_error != FM_OK) {
    cudaGetLastError();
    if (g != nullptr) cudaGraphDestroy(g);
    c->launch_error = FM_OK;
    return FM_ERR_CUDA;
  }
  if (cudaGraphInstantiate(&ge, g, 0) != cudaSuccess) { cudaGetLastError(); cudaGraphDestroy(g); return FM_ERR_CUDA; }
  cudaEvent_t e0, e1;
  cudaEventCreate(&e0);
  cudaEventCreate(&e1);
  for (int i = 0; i < 3; ++i) cudaGraphLaunch(ge, c->stream);
  cudaEventRecord(e0, c->stream);
  for (int i = 0; i < reps; ++i) cudaGraphLaunch(ge, c->stream);
  cudaEventRecord(e1, c->stream);
  const bool ok = cudaEventSynchronize(e1) == cudaSuccess;
  float ms = 0.f;
  cudaEventElapsedTime(&ms, e0, e1);
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  cudaGraphExecDestroy(ge);
  cudaGraphDestroy(g);
  if (!ok) return FM_ERR_CUDA;
  if (cls == PROF_GEMM) { out->gemm_ms = ms / reps; out->gemm_launches = n_launch; out->gemm_bytes = c->class_bytes; }
  else { out->attn_ms = ms / reps; out->attn_launches = n_launch; }
  c->phase = 1;
  return FM_OK;
}

int fm_destroy(fm_ctx* c) {
  if (c == nullptr) return FM_ERR_INVALID_ARG;
  cudaStreamSynchronize(c->stream);
  for (auto& e : c->prof_ev) cudaEventDestroy(e);
  drop_graph(c);
  drop_call_graph(c->cg_verify);
  drop_call_graph(c->cg_draft);
  if (c->host_done != nullptr) cudaFreeHost(c->host_done);
  delete c;
  return FM_OK;
}

int fm_prefill(fm_ctx* c, int32_t batch, const float* cond, const int32_t* prompt, const int32_t* prompt_off) {
  if (c == nullptr || prompt_off == nullptr) return FM_ERR_INVALID_ARG;
  const Dims& dm = c->dm;
  if (batch < 1) return FM_ERR_INVALID_ARG;
  if (batch > dm.max_batch) return FM_ERR_CAPACITY;
  if (dm.P > 0 && cond == nullptr) return FM_ERR_INVALID_ARG;
  int longest = 0;
  for (int b = 0; b < batch; ++b) {
    const int n = prompt_off[b + 1] - prompt_off[b];
    if (n < 0 || n % 9 != 0) return FM_ERR_INVALID_ARG;
    if (1 + n + dm.D + 2 > dm.max_tokens) return FM_ERR_CAPACITY;
    longest = n > longest ? n : longest;
  }
  if (prompt_off[batch] > 0 && prompt == nullptr) return FM_ERR_INVALID_ARG;
  c->batch = batch;
  c->launch_error = FM_OK;                         // a new start clears an earlier enqueue error
  // ... and whatever a kernel that gave up on a bounded wait left behind: the status word, and
  // the tickets of attention tiles whose last CTA never came to reset them
  CUDA_OK(cudaMemsetAsync(c->st.status, 0, sizeof(int), c->stream));
  CUDA_OK(cudaMemsetAsync(c->attn_ticket, 0, c->attn_ticket_n * sizeof(int), c->stream));
  c->plen_host.assign(batch, 0);
  for (int b = 0; b < batch; ++b) c->plen_host[b] = prompt_off[b + 1] - prompt_off[b];
  CUDA_OK(cudaMemcpyAsync(c->prompt_off_dev, prompt_off, (batch + 1) * sizeof(int), cudaMemcpyHostToDevice, c->stream));
  CUDA_OK(cudaStreamSynchronize(c->stream));       // prompt_off is caller memory: finish reading it now
  LAUNCH(c, init_state_kernel, (dm.max_batch + 127) / 128, 128, 0, dm, c->st, batch, c->prompt_off_dev);
  // per-layer prefix keys/values: K_pre = Wk rms(c, g1), V_pre = Wv rms(c, g1), no rotation
  const int rows_total = batch * dm.P, kvw = 2 * dm.Hkv * dm.dh;
  for (int r0 = 0; r0 < rows_total; r0 += PREFILL_CHUNK) {
    const int rows = rows_total - r0 < PREFILL_CHUNK ? rows_total - r0 : PREFILL_CHUNK;
    for (int s = 0; s < 5; ++s)
      for (auto& L : c->layers[s]) {
        LAUNCH(c, rmsnorm_kernel, rows, 256, 0, cond + (size_t)r0 * dm.d, L.g1, c->pre_a, dm.d, dm.eps);
        gemm(c, L.Wqkv, pad128((size_t)(dm.H + 2 * dm.Hkv) * dm.dh), dm.H * dm.dh, c->pre_a, PREFILL_CHUNK, 0, kvw, dm.d, rows,
             nullptr, tc::EPI_F32, epi_plain(c->pre_o, kvw));
        LAUNCH(c, prefix_store_kernel, rows, 128, 0, dm, STACK_LEVEL[s], r0, c->pre_o, L.K, L.V);
      }
  }
  // BOS + prompt through the multi-row forward, D+1 rows per sequence and pass, all rows kept
  const int passes = (1 + longest + dm.R1 - 1) / dm.R1;
  for (int i = 0; i < passes; ++i) {
    LAUNCH(c, prefill_feed_kernel, batch, 32, 0, dm, c->st, batch, prompt, c->prompt_off_dev);
    LAUNCH(c, row_count_kernel, 1, 32, 0, dm, c->st, batch);
    forward(c, nullptr);
    LAUNCH(c, prefill_advance_kernel, (batch + 127) / 128, 128, 0, dm, c->st, batch);
  }
  LAUNCH(c, arm_kernel, (batch + 127) / 128, 128, 0, dm, c->st, batch);
  LAUNCH(c, row_count_kernel, 1, 32, 0, dm, c->st, batch);
  CUDA_OK(cudaGetLastError());
  if (c->launch_error != FM_OK) return c->launch_error;
  c->phase = 1;
  c->gen_fresh = true;
  return FM_OK;
}

int fm_set_max_faces(fm_ctx* c, const int32_t* max_faces) {
  if (c == nullptr || max_faces == nullptr) return FM_ERR_INVALID_ARG;
  if (c->phase < 1) return FM_ERR_BAD_STATE;
  for (int b = 0; b < c->batch; ++b) if (max_faces[b] < 0) return FM_ERR_INVALID_ARG;
  int* tmp = reinterpret_cast<int*>(c->pre_o);       // scratch that no pass is using now
  CUDA_OK(cudaMemcpyAsync(tmp, max_faces, c->batch * sizeof(int), cudaMemcpyHostToDevice, c->stream));
  LAUNCH(c, set_limits_kernel, (c->batch + 127) / 128, 128, 0, c->dm, c->st, c->batch, tmp);
  LAUNCH(c, arm_kernel, (c->batch + 127) / 128, 128, 0, c->dm, c->st, c->batch);
  LAUNCH(c, row_count_kernel, 1, 32, 0, c->dm, c->st, c->batch);
  CUDA_OK(cudaStreamSynchronize(c->stream));       // max_faces is caller memory
  return FM_OK;
}

int fm_draft(fm_ctx* c, int32_t* cand, float* draft_logits, float* draft_margin) {
  if (c == nullptr) return FM_ERR_INVALID_ARG;
  if (c->phase < 1) return FM_ERR_BAD_STATE;
  run_cached(c, c->cg_draft, cand, draft_logits, draft_margin, nullptr, [&] {
    draft(c, draft_logits, draft_margin, nullptr);
    const int n = c->batch * c->dm.R1;
    if (cand != nullptr) LAUNCH(c, copy_i32_kernel, (n + 127) / 128, 128, 0, c->st.cand, cand, n);
  });
  CUDA_OK(cudaGetLastError());
  if (c->launch_error != FM_OK) return c->launch_error;
  return FM_OK;
}

int fm_correct_ex(fm_ctx* c, int32_t* cand, const int32_t* labels, int32_t use_history) {
  if (c == nullptr || cand == nullptr) return FM_ERR_INVALID_ARG;
  if (c->phase < 1) return FM_ERR_BAD_STATE;
  if (c->dm.R1 > 3 * FM_CORRECT_MAX_POINTS) return FM_ERR_UNSUPPORTED;
  if (labels == nullptr) {
    if (!c->dm.has_label || c->dm.D == 0) return FM_ERR_UNSUPPORTED;
    labels = c->labels;
  }
  LAUNCH(c, correct_kernel, (c->batch + 63) / 64, 64, 0, c->dm, c->st, c->batch, cand, labels, use_history != 0 ? 1 : 0);
  CUDA_OK(cudaGetLastError());
  if (c->launch_error != FM_OK) return c->launch_error;
  return FM_OK;
}

int fm_correct(fm_ctx* c, int32_t* cand, const int32_t* labels) {
  if (labels == nullptr) return FM_ERR_INVALID_ARG;
  return fm_correct_ex(c, cand, labels, 0);
}

int fm_draft_labels(fm_ctx* c, int32_t* labels, float* margin) {
  if (c == nullptr || labels == nullptr) return FM_ERR_INVALID_ARG;
  if (c->phase < 1) return FM_ERR_BAD_STATE;
  if (!c->dm.has_label || c->dm.D == 0) return FM_ERR_UNSUPPORTED;
  const int n = c->batch * c->dm.R1;
  LAUNCH(c, copy_i32_kernel, (n + 127) / 128, 128, 0, c->labels, labels, n);
  if (margin != nullptr) LAUNCH(c, copy_f32_kernel, (n + 127) / 128, 128, 0, c->label_margin, margin, n);
  CUDA_OK(cudaGetLastError());
  return FM_OK;
}

int fm_verify(fm_ctx* c, const int32_t* cand, int32_t* argmax, float* logits, float* margin) {
  if (c == nullptr || cand == nullptr) return FM_ERR_INVALID_ARG;
  if (c->phase < 1) return FM_ERR_BAD_STATE;
  run_cached(c, c->cg_verify, cand, argmax, logits, margin, [&] {
    const int n = c->batch * c->dm.R1;
    LAUNCH(c, verify_load_kernel, (n + 127) / 128, 128, 0, c->dm, c->st, c->batch, cand);
    forward(c, logits);
    if (argmax != nullptr) LAUNCH(c, copy_i32_kernel, (n + 127) / 128, 128, 0, c->st.o, argmax, n);
    if (margin != nullptr) LAUNCH(c, copy_f32_kernel, (n + 127) / 128, 128, 0, c->st.margin, margin, n);
  });
  CUDA_OK(cudaGetLastError());
  if (c->launch_error != FM_OK) return c->launch_error;
  c->phase = 2;
  return FM_OK;
}

int fm_verify_static_scratch(fm_ctx* c, const int32_t* cand, int32_t* argmax, float* logits, float* margin) {
  if (c == nullptr || cand == nullptr) return FM_ERR_INVALID_ARG;
  if (c->phase < 1) return FM_ERR_BAD_STATE;
  // what the attention kernel needs: the largest level's group partials, then one ticket per
  // (sequence, kv-head, query tile)
  const Dims& dm = c->dm;
  size_t part_floats = 0, tickets = 0;
  for (int l = 0; l < 3; ++l) {
    const size_t per = (size_t)dm.max_batch * dm.Hkv * c->attn_mt[l];
    const size_t need = per * c->attn_max_groups[l] * 16 * (dm.dh + 2);
    part_floats = need > part_floats ? need : part_floats;
    tickets = per > tickets ? per : tickets;
  }
  const size_t ticket_off = align_up(part_floats * sizeof(float), 256);
  if (ticket_off + tickets * sizeof(int) > (size_t)FM_STATIC_SCRATCH_BYTES) return FM_ERR_CAPACITY;
  // Device address of the static array, looked up once per device with that device current (the
  // array's name is only a host-side handle; a kernel must be given this address).  Every GPU
  // holds its own copy of the array, so the address must be the one of the context's device:
  // the call is refused when another device is current.
  static void* dev_addr[64] = {nullptr};
  static std::mutex dev_addr_lock;
  int dev = -1;
  CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return FM_ERR_UNSUPPORTED;
  if (dev != c->device) return FM_ERR_BAD_STATE;
  {
    std::lock_guard<std::mutex> hold(dev_addr_lock);
    if (dev_addr[dev] == nullptr) {
      void* p = nullptr;
      if (cudaGetSymbolAddress(&p, g_static_attn_scratch) != cudaSuccess || p == nullptr) return FM_ERR_CUDA;
      dev_addr[dev] = p;
    }
  }
  unsigned char* base = static_cast<unsigned char*>(dev_addr[dev]);
  // tickets must start at zero; the array keeps whatever the last call (of any context) left
  CUDA_OK(cudaMemsetAsync(base + ticket_off, 0, tickets * sizeof(int), c->stream));
  float* saved_part = c->attn_part;
  int* saved_ticket = c->attn_ticket;
  c->attn_part = reinterpret_cast<float*>(base);
  c->attn_ticket = reinterpret_cast<int*>(base + ticket_off);
  const bool was_off = c->call_graphs_off;
  c->call_graphs_off = true;                       // the scratch pointers differ from the cached graph's
  const int rc = fm_verify(c, cand, argmax, logits, margin);
  c->call_graphs_off = was_off;
  c->attn_part = saved_part;
  c->attn_ticket = saved_ticket;
  return rc;
}

int fm_step_host(fm_ctx* c, const int32_t* cand, int32_t* n_acc, int32_t* emitted, int32_t* kv_len) {
  if (c == nullptr || n_acc == nullptr) return FM_ERR_INVALID_ARG;
  if (c->phase < 1) return FM_ERR_BAD_STATE;
  const Dims& dm = c->dm;
  const int n = c->batch * dm.R1;
  int rc = fm_draft(c, nullptr, nullptr, nullptr);
  if (rc != FM_OK) return rc;
  if (cand != nullptr) CUDA_OK(cudaMemcpyAsync(c->step_in, cand, n * sizeof(int), cudaMemcpyHostToDevice, c->stream));
  LAUNCH(c, step_merge_kernel, (n + 127) / 128, 128, 0, dm, c->st, c->batch, cand != nullptr ? (const int*)c->step_in : (const int*)nullptr, c->step_cand);
  rc = fm_verify(c, c->step_cand, nullptr, nullptr, nullptr);
  if (rc != FM_OK) return rc;
  rc = fm_accept(c, nullptr, nullptr, c->step_nacc, c->step_em, c->step_kv);
  if (rc != FM_OK) return rc;
  CUDA_OK(cudaMemcpyAsync(n_acc, c->step_nacc, c->batch * sizeof(int), cudaMemcpyDeviceToHost, c->stream));
  if (emitted != nullptr) CUDA_OK(cudaMemcpyAsync(emitted, c->step_em, n * sizeof(int), cudaMemcpyDeviceToHost, c->stream));
  if (kv_len != nullptr) CUDA_OK(cudaMemcpyAsync(kv_len, c->step_kv, c->batch * 3 * sizeof(int), cudaMemcpyDeviceToHost, c->stream));
  CUDA_OK(cudaStreamSynchronize(c->stream));
  return FM_OK;
}

int fm_accept(fm_ctx* c, const int32_t* force_len, const int32_t* force_tok, int32_t* n_acc, int32_t* emitted,
              int32_t* kv_len) {
  if (c == nullptr) return FM_ERR_INVALID_ARG;
  if (c->phase != 2) return FM_ERR_BAD_STATE;
  LAUNCH(c, accept_kernel, 1, accept_threads(c->batch), 0, c->dm, c->st, c->batch, force_len, force_tok, n_acc, emitted, kv_len,
         (const GenOut*)nullptr, 0);
  CUDA_OK(cudaGetLastError());
  if (c->launch_error != FM_OK) return c->launch_error;
  c->phase = 1;
  return FM_OK;
}

int fm_generate(fm_ctx* c, int32_t max_faces, int32_t* out_tok, int32_t out_stride, int32_t* out_len,
                const fm_teacher* teacher, int32_t plain, int64_t max_steps, fm_stats* stats) {
  if (c == nullptr || max_faces < -1) return FM_ERR_INVALID_ARG;
  if (c->phase < 1) return FM_ERR_BAD_STATE;
  const Dims& dm = c->dm;
  const bool keep_limits = max_faces == -1;          // per-sequence limits of fm_set_max_faces stay
  if (keep_limits) max_faces = (dm.max_tokens + 8) / 9;
  if (out_tok != nullptr && (out_len == nullptr || (!keep_limits && out_stride < 9 * max_faces))) return FM_ERR_CAPACITY;
  if (teacher != nullptr && (teacher->truth == nullptr || teacher->truth_stride <= 0 ||
                             (teacher->keep != nullptr && teacher->n_sched <= 0))) return FM_ERR_INVALID_ARG;
  int rc = FM_OK;
  if (!keep_limits) {
    for (int b = 0; b < c->batch; ++b)
      if ((long long)c->plen_host[b] + 9ll * max_faces + dm.D + 2 > dm.max_tokens) return FM_ERR_CAPACITY;
    std::vector<int> lim(c->batch, max_faces);
    rc = fm_set_max_faces(c, lim.data());
    if (rc != FM_OK) return rc;
  }
  GenOut g{};
  g.out_tok = out_tok; g.out_stride = out_stride; g.out_len = out_len;
  if (teacher != nullptr) { g.truth = teacher->truth; g.truth_stride = teacher->truth_stride; g.keep = teacher->keep; g.n_sched = teacher->n_sched; }
  g.plain = plain;
  g.stats = c->stats_dev;
  g.host_done = c->host_done_dev;
  CUDA_OK(cudaMemcpyAsync(c->gen_dev, &g, sizeof(g), cudaMemcpyHostToDevice, c->stream));
  CUDA_OK(cudaMemsetAsync(c->stats_dev, 0, (FM_MAX_DRAFT + 4) * sizeof(long long), c->stream));
  if (out_len != nullptr && c->gen_fresh) CUDA_OK(cudaMemsetAsync(out_len, 0, c->batch * sizeof(int), c->stream));
  c->gen_fresh = false;
  CUDA_OK(cudaStreamSynchronize(c->stream));       // `g` lives on this stack frame
  if (!c->prof_on) ensure_graph(c);
  const bool use_graph = !c->prof_on && c->graph_exec != nullptr;
  cudaEvent_t e0, e1;
  CUDA_OK(cudaEventCreate(&e0));
  CUDA_OK(cudaEventCreate(&e1));
  CUDA_OK(cudaEventRecord(e0, c->stream));
  *c->host_done = c->batch;
  // upper bound on passes: every pass emits at least one token per unfinished sequence
  const long long bound = max_steps > 0 ? max_steps : 9ll * max_faces + 8;
  long long steps = 0;
  bool finished = false;
  while (!finished && steps < bound) {
    const long long poll = max_steps > 0 ? bound : 8;
    for (long long i = 0; i < poll; ++i) {
      if (use_graph) {
        CUDA_OK(cudaGraphLaunch(c->graph_exec, c->stream));
        c->launches += c->graph_launches;
      } else {
        step_body(c);
      }
      ++steps;
    }
    CUDA_OK(cudaStreamSynchronize(c->stream));
    finished = *c->host_done == 0 || max_steps > 0;
  }
  CUDA_OK(cudaEventRecord(e1, c->stream));
  CUDA_OK(cudaEventSynchronize(e1));
  float ms = 0.f;
  cudaEventElapsedTime(&ms, e0, e1);
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  if (stats != nullptr) {
    long long h[FM_MAX_DRAFT + 4];
    CUDA_OK(cudaMemcpy(h, c->stats_dev, sizeof(h), cudaMemcpyDeviceToHost));
    memset(stats, 0, sizeof(*stats));
    stats->steps = h[0];
    stats->emitted = h[1];
    for (int a = 0; a < FM_MAX_DRAFT + 2; ++a) stats->accept_hist[a] = h[2 + a];
    stats->ms = ms;
  }
  c->phase = 1;
  return finished ? FM_OK : FM_ERR_TIMEOUT;
}

double fm_verify_bytes(const fm_ctx* c, int32_t batch, const int32_t* kv_len) {
  if (c == nullptr || kv_len == nullptr || batch < 1) return 0.0;
  const Dims& dm = c->dm;
  const double d = dm.d;
  const double layer_w = 2.0 * ((double)(dm.H + 2 * dm.Hkv) * dm.dh * d + d * dm.H * dm.dh + 2.0 * d * dm.dff);
  bool has[3] = {false, false, false};
  double kv[3] = {0, 0, 0};
  for (int b = 0; b < batch; ++b) {
    const int L = kv_len[b * 3];
    for (int l = 0; l < 3; ++l) {
      const int r = fm_ratio(l);
      const int p0 = (L + r - 1) / r, p1 = (L + dm.D) / r;
      if (p1 < p0) continue;
      has[l] = true;
      const int lo = dm.window[l] > 0 ? (p0 - dm.window[l] + 1 > 0 ? p0 - dm.window[l] + 1 : 0) : 0;
      kv[l] += (double)(dm.P + p1 - lo + 1) * 2.0 * dm.Hkv * dm.dh * 2.0;     // K and V, bf16
    }
  }
  double bytes = 2.0 * d * dm.V;                                              // output matrix
  for (int s = 0; s < 5; ++s) {
    const int l = STACK_LEVEL[s];
    if (has[l]) bytes += c->cfg.layers[s] * (layer_w + kv[l]);
  }
  if (has[1]) bytes += 2.0 * 2.0 * 3.0 * d * d;                               // S_cv + U_vc
  if (has[2]) bytes += 2.0 * 2.0 * 3.0 * d * d;                               // S_vf + U_fv
  return bytes;
}

int fm_attention_layout(const fm_ctx* c, int32_t level, int32_t* chunk_slots, int32_t* chunks_per_group, int32_t* max_groups) {
  if (c == nullptr || level < 0 || level > 2) return FM_ERR_INVALID_ARG;
  if (chunk_slots != nullptr) *chunk_slots = c->attn_chunk;
  if (chunks_per_group != nullptr) *chunks_per_group = c->attn_G[level];
  if (max_groups != nullptr) *max_groups = c->attn_max_groups[level];
  return FM_OK;
}

int64_t fm_launch_count(const fm_ctx* c) { return c ? c->launches : 0; }

int fm_selftest_wait_timeout(fm_ctx* c, int64_t limit_cycles) {
  if (c == nullptr || limit_cycles < 1 || limit_cycles > 100000000ll) return FM_ERR_INVALID_ARG;
  LAUNCH(c, wait_timeout_probe_kernel, 1, 32, 0, c->st.status, (long long)limit_cycles);
  CUDA_OK(cudaGetLastError());
  return FM_OK;
}

int fm_device_status(fm_ctx* c) {
  if (c == nullptr) return FM_ERR_INVALID_ARG;
  int s = 0;
  if (cudaMemcpyAsync(&s, c->st.status, sizeof(int), cudaMemcpyDeviceToHost, c->stream) != cudaSuccess) return FM_ERR_CUDA;
  if (cudaStreamSynchronize(c->stream) != cudaSuccess) return FM_ERR_CUDA;
  return s;
}

}  // extern "C"
