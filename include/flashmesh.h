/*
 * flashmesh.h -- C ABI of the speculative decode step of an hourglass mesh transformer
 * (FlashMesh, arXiv 2511.15618), hand-written CUDA for sm_100a, one GPU.
 *
 * The paper states the problem as: given a condition c and the accepted prefix, every
 * forward pass of the backbone yields one main token and the draft modules yield D draft
 * tokens (Sec. 3.1); the drafts may be edited before they are fed back (Sec. 3.2); one
 * forward pass with causal masking verifies main + drafts (Sec. 3.3); the main token and
 * the drafts up to the first mismatch are accepted and decoding continues from the
 * backbone's output at the last accepted token (Sec. 3.3).  The calls below are those
 * stages.  The model is the hourglass of the supplement ("Hourglass Transformer": three
 * coordinates form a vertex, three vertices a face; shortening and upsampling layers with
 * residuals between levels) with a KV cache at each level.
 *
 * Where the paper is silent the model is read as follows: pre-norm RMSNorm blocks, FFN =
 * W2 gelu_erf(W1 x) without biases, rotate-half rotary embedding on the level-local index,
 * conditioning as per-layer prefix keys/values (every layer projects rms(c) with its own K/V
 * matrices; un-rotated, visible to every query, sharing the softmax with the causal keys),
 * shortening = linear on the concatenation of hiddens 3v-2, 3v-1, 3v (zeros below 0), upsampling
 * = linear d -> 3d whose slot r is added to the pre-shorten hidden of position 3v+r,
 * longest-matching-prefix acceptance, masked argmax with ties to the lowest id.
 *
 * Conventions
 *   - Every call returns FM_OK (0) or a negative FM_ERR_* code; nothing throws.  On an error
 *     return no decoding state has been changed, except after FM_ERR_CUDA or FM_ERR_TIMEOUT:
 *     then nothing more is enqueued and the sequences must be started again with fm_prefill
 *     (or the context destroyed).
 *   - Pointers are marked HOST or DEV.  DEV pointers are caller-owned device memory that must
 *     stay valid until the work enqueued by the call has finished on the context's stream.
 *   - fm_draft and fm_verify launch their kernels one by one the first time they see a set of
 *     pointer arguments, capture them into a CUDA graph when the same pointers come again, and
 *     replay that graph afterwards: a host that drives the loop call by call should pass the same
 *     buffers every pass.  (A stream that cannot be captured keeps the plain launches.)
 *   - All calls except fm_create / fm_destroy / fm_generate only enqueue work on the
 *     context's stream and return; fm_generate polls a completion flag and returns when every
 *     sequence has finished.
 *   - The library allocates no device memory: the caller hands a workspace of
 *     fm_workspace_bytes() bytes to fm_create, which carves weights (bfloat16), KV caches and
 *     scratch out of it.  (fm_create allocates a few hundred bytes of pinned host memory.)
 *   - Indexing: inputs u_0 = BOS, u_i = t_{i-1}; the row at position i predicts mesh token
 *     t_i.  L = inputs consumed so far; the pending main token is t_{L-1}.  A verify pass
 *     feeds positions L..L+D; accepting a tokens moves L to L+a.
 *   - Lossless by construction (Sec. 3.3): within one context the logits of a position do not
 *     depend on the row of the pass it is fed in, on the other rows or sequences of the pass,
 *     nor on the accept lengths of the passes before it, to the last bit (reduction orders are
 *     fixed by slot and column index; every value that can be produced at two places of the code
 *     is rounded explicitly), so the tokens a speculative run emits are those of one-token-per-
 *     pass decoding with the same context, whatever the drafts were.  Two contexts (another
 *     batch size, draft count or capacity) may group reductions differently.
 *   - Token ids: [0, n_bins) coordinate bins, BOS = n_bins, EOS = n_bins+1, PAD = n_bins+2.
 *     Emitted ids are always coordinate bins, or EOS at a face boundary when allow_eos != 0;
 *     ties in an argmax go to the lowest id.
 */
#ifndef FLASHMESH_H
#define FLASHMESH_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define FM_OK                0
#define FM_ERR_INVALID_ARG  -1   /* null pointer, size out of range, inconsistent config      */
#define FM_ERR_BAD_STATE    -2   /* call out of order (e.g. fm_verify before fm_prefill)       */
#define FM_ERR_CAPACITY     -3   /* batch > max_batch, prompt or run longer than max_tokens    */
#define FM_ERR_CUDA         -4   /* a CUDA runtime call failed                                 */
#define FM_ERR_TIMEOUT      -5   /* a bounded device-side wait gave up (see fm_device_status)  */
#define FM_ERR_UNSUPPORTED  -6   /* shape outside what the kernels were built for              */

#define FM_MAX_FACE_HEADS 4
#define FM_MAX_DRAFT      27

typedef struct fm_ctx fm_ctx;    /* opaque; owns nothing but pinned host flags */

/* Model and capacity description (the hourglass of the supplement, read as stated above). */
typedef struct fm_config {
  int32_t d_model, n_heads, n_kv_heads, head_dim, d_ff;
  int32_t layers[5];          /* coord_down, vertex_down, face, vertex_up, coord_up          */
  int32_t n_bins;             /* vocabulary = n_bins + 3                                     */
  int32_t n_prefix;           /* P conditioning vectors, held as prefix keys/values          */
  int32_t window[3];          /* attention window per level (coordinate, vertex, face); 0 = full */
  int32_t draft_len;          /* D, 0..FM_MAX_DRAFT                                          */
  int32_t max_batch;
  int32_t max_tokens;         /* capacity per sequence in coordinate positions (inputs)      */
  float   rope_theta;         /* 0 = no positional encoding                                  */
  float   norm_eps;
  int32_t allow_eos;          /* 0: EOS is masked everywhere (fixed-length runs)             */
  /* draft modules (Sec. 3.1; supplement "Three-Level Speculative Decoding") */
  int32_t draft_heads;        /* FM_HEADS_REDUCED: SP = h + A rms(h), HF = the upsample matrices alone;
                                 FM_HEADS_FULL: SP-Blocks with attention (Eq. 1), an HF-Block after
                                 every upsample (Eq. 2-5)                                     */
  int32_t draft_levels;       /* FM_LEVELS_THREE: 2 coordinate heads + point level + face level;
                                 FM_LEVELS_COORD: D coordinate heads, no point / face level (the
                                 supplement's ablation on multi-level decoding)               */
  int32_t hf_ff;              /* hidden width of the HF-Blocks' feed-forward networks (0 = d_model;
                                 a multiple of 64)                                            */
  int32_t avg_levels;         /* 1: where several levels predict a position their softmax
                                 distributions are averaged (supplement, "Integrating the three
                                 levels"); 0: one source per position ("Optimizations")       */
} fm_config;
#define FM_HEADS_REDUCED 0
#define FM_HEADS_FULL    1
#define FM_LEVELS_THREE  0
#define FM_LEVELS_COORD  1

/* HOST pointers to float32 matrices, row-major [out, in]; values are rounded to bfloat16
 * (nearest-even) when fm_create copies them.  Gains stay float32. */
typedef struct fm_layer_weights {
  const float* g1;            /* [d]                          RMSNorm gain before attention   */
  const float* Wqkv;          /* [(H + 2*Hkv)*dh, d]          rows: Q heads, K heads, V heads */
  const float* Wo;            /* [d, H*dh]                                                    */
  const float* g2;            /* [d]                          RMSNorm gain before the FFN     */
  const float* W1;            /* [d_ff, d]                                                    */
  const float* W2;            /* [d, d_ff]                                                    */
} fm_layer_weights;

/* One SP-Block head (Eq. 1).  Reduced: y = h + A rms(h, g).  Full: the attention of the block reads
 * the cache of the backbone's last layer at the head's level (keys / values of the split-node hiddens;
 * conditioning as the prefix entries of the same softmax) with the head's own query and output
 * matrices: u = h + Wo Attn(Wq rms(h, ga)), y = h + A rms(u, g).  ga / Wq / Wo are read only with
 * FM_HEADS_FULL. */
typedef struct fm_sp_weights {
  const float* g;  const float* A;        /* [d], [d, d]                                       */
  const float* ga; const float* Wq; const float* Wo;   /* [d], [H*dh, d], [d, H*dh]            */
} fm_sp_weights;

/* One HF-Block (Eq. 3-5) for one offset: x + W2 gelu(W1 Attn(Wq rms(x, g), K, V)) with K, V the cache
 * of the backbone's last layer at the block's level, entries up to the last accepted position. */
typedef struct fm_hf_weights {
  const float* g; const float* Wq; const float* W1; const float* W2;   /* [d], [H*dh, d], [hf, H*dh], [d, hf] */
} fm_hf_weights;

typedef struct fm_weights {
  const float* E;                         /* [V, d] token embedding                          */
  const fm_layer_weights* stack[5];       /* stack[s][l], l < layers[s]                      */
  const float* S_cv;                      /* [d, 3d] shorten coordinate -> vertex            */
  const float* S_vf;                      /* [d, 3d] shorten vertex -> face                  */
  const float* U_fv;                      /* [3d, d] upsample face -> 3 vertices             */
  const float* U_vc;                      /* [3d, d] upsample vertex -> 3 coordinates        */
  const float* g_out;                     /* [d]                                              */
  const float* W_out;                     /* [V, d]                                           */
  /* Draft modules.  heads_c: coordinate heads (2, or D with FM_LEVELS_COORD); heads_v: 2 point-level
   * heads (vertex v*+1, v*+2); heads_f: face-level heads, head e (1-based) drafts the face e-1 after
   * the one that holds the pending token; D < 7 uses 1 head, otherwise (D+8)/9 + 1.  heads_v,
   * heads_f and the HF-Blocks are not read with FM_LEVELS_COORD. */
  const fm_sp_weights* heads_c;
  const fm_sp_weights* heads_v;
  const fm_sp_weights* heads_f;
  /* HF-Blocks (FM_HEADS_FULL only): hf_vc[6] refine the point level's coordinate features (offset
   * 3..8 from the vertex row), hf_fv[3*Ef] the face level's vertex features, hf_fc[9*Ef] the face
   * level's coordinate features. */
  const fm_hf_weights* hf_vc;
  const fm_hf_weights* hf_fv;
  const fm_hf_weights* hf_fc;
  /* label head of the correction stage (Sec. 3.2): gain [d] and matrix [3, d]; may be NULL (then
   * fm_draft produces no labels) */
  const float* label_g;
  const float* label_W;
} fm_weights;

/* Optional device-side draft editor for fm_generate: the place where the paper's Correct
 * stage sits (Sec. 3.2 edits drafts only, never the main token).  Used by the benchmark to
 * pin the true acceptance length: draft j (1..keep) is replaced by the known continuation,
 * draft keep+1 by a deliberately different coordinate id. */
typedef struct fm_teacher {
  const int32_t* truth;       /* DEV [batch, truth_stride]: mesh tokens t_0.. (prompt included) */
  int32_t truth_stride;
  const int32_t* keep;        /* DEV [n_sched, batch]: correct drafts wanted per step, 0..D  */
  int32_t n_sched;            /* the schedule wraps around                                   */
} fm_teacher;

typedef struct fm_stats {
  int64_t steps;                          /* draft+verify+accept passes executed             */
  int64_t emitted;                        /* mesh tokens emitted, all sequences              */
  int64_t accept_hist[FM_MAX_DRAFT + 2];  /* accept_hist[a] = passes that accepted a tokens  */
  float   ms;                             /* device time of the decode loop (CUDA events)    */
} fm_stats;

/* Bytes of device workspace fm_create needs for this configuration (0 if it is invalid). */
size_t fm_workspace_bytes(const fm_config* cfg /*HOST*/);

/* Build a context inside `dev_workspace` (DEV, 256-byte aligned, >= fm_workspace_bytes):
 * copies and rounds the weights, zeroes state.  `cuda_stream` is a cudaStream_t (NULL = the
 * default stream); all later work of this context runs on it.  Synchronous.
 * Errors: INVALID_ARG (null, bad config), CAPACITY (workspace too small), UNSUPPORTED
 * (d_model or d_ff not a multiple of 64, n_heads*head_dim not a multiple of 128, head_dim not
 * 64/128, a stack without layers, D > FM_MAX_DRAFT, hf_ff not a multiple of 64), CUDA. */
int fm_create(const fm_config* cfg /*HOST*/, const fm_weights* w /*HOST*/, void* dev_workspace /*DEV*/,
              size_t workspace_bytes, void* cuda_stream, fm_ctx** out /*HOST*/);
int fm_destroy(fm_ctx* ctx);

/* Start `batch` sequences.  cond: DEV float32 [batch, P, d] conditioning vectors, projected by
 * every layer's own K/V matrices into prefix cache slots.  prompt: DEV int32, the sequences'
 * mesh tokens concatenated; prompt_off: HOST int32 [batch+1] offsets into it (lengths must be
 * multiples of 9).  Runs BOS + prompt through the multi-row forward in chunks of D+1 rows.
 * Afterwards L[b] = 1 + prompt_len[b] and the first main token is pending.
 * Errors: INVALID_ARG, CAPACITY. */
int fm_prefill(fm_ctx* ctx, int32_t batch, const float* cond /*DEV*/, const int32_t* prompt /*DEV*/,
               const int32_t* prompt_off /*HOST*/);

/* Per-sequence limit: sequence b stops once 9*max_faces[b] tokens have been emitted after
 * its prompt (or at EOS).  HOST int32 [batch].  Default: the cache capacity. */
int fm_set_max_faces(fm_ctx* ctx, const int32_t* max_faces /*HOST*/);

/* Predict (Sec. 3.1, supplement "Three-Level Speculative Decoding"): run the draft modules
 * (reduced heads, or the full SP-Blocks and HF-Blocks; fm_config.draft_heads / draft_levels) on
 * the split-node hiddens stashed at the last accepted position; with a label head, also the
 * labels of the drafted points (fm_draft_labels).  cand: DEV int32 out
 * [batch, D+1] = pending main token, then D drafts (PAD for finished sequences).
 * draft_logits: DEV float32 out [batch, D, V] or NULL.  draft_margin: DEV float32 out
 * [batch, D] (top-1 minus top-2 of the masked draft logits) or NULL. */
int fm_draft(fm_ctx* ctx, int32_t* cand /*DEV*/, float* draft_logits /*DEV*/, float* draft_margin /*DEV*/);

/* Correct (Sec. 3.2 "Correction Mechanism"): edit the drafts of a candidate row in place, between
 * fm_draft and fm_verify.  A point is a vertex whose three coordinate tokens (z, y, x) are all
 * drafts of this pass (slot s of sequence b holds mesh token L[b] - 1 + s; slot 0 is the main
 * token and is never touched; vertices that are only partly in the row, or that hold a token that
 * is not a coordinate bin, are left alone).  labels: DEV int32 [batch, D+1]; labels[b][s] is the
 * label of the point that starts at slot s: FM_LABEL_HISTORICAL, FM_LABEL_NEW or FM_LABEL_INTRA
 * (other slots are not read; fm_draft_labels gives the labels of the library's own label head).
 * In sequence order, every FM_LABEL_INTRA point that has no identical point in the row is
 * replaced by the nearest (squared distance between bin indices, ties to the earliest) earlier
 * FM_LABEL_NEW point of another face, if there is one; then the points of every face are sorted
 * ascending by (z, y, x) among the slots they occupy.  Only rows the next pass feeds
 * (the first nrow slots of an unfinished sequence) are considered.
 * cand: DEV int32 in/out [batch, D+1].  Errors: INVALID_ARG (null pointer), BAD_STATE (before
 * fm_prefill), UNSUPPORTED (more than 48 slots per row; cannot happen while FM_MAX_DRAFT is 27). */
#define FM_LABEL_HISTORICAL 0
#define FM_LABEL_NEW 1
#define FM_LABEL_INTRA 2
int fm_correct(fm_ctx* ctx, int32_t* cand /*DEV*/, const int32_t* labels /*DEV*/);

/* Labels of the drafted points (Sec. 3.2: a label head, a linear layer, on every point-level
 * feature), as computed by the last fm_draft: labels[b][s] in {FM_LABEL_HISTORICAL, FM_LABEL_NEW,
 * FM_LABEL_INTRA} where a vertex made of drafts only starts at slot s, -1 elsewhere; the label is
 * the argmax (ties to the lowest) of label_W rms(f, label_g) over the point-level feature f in the
 * pipeline of the head that drafts the point's last coordinate.  margin: top-1 minus top-2, or NULL.
 * DEV out [batch, D+1].  Errors: UNSUPPORTED without a label head or with FM_LEVELS_COORD. */
int fm_draft_labels(fm_ctx* ctx, int32_t* labels /*DEV*/, float* margin /*DEV*/);

/* fm_correct with two options: labels == NULL takes the label head's labels of the last fm_draft;
 * use_history != 0 also enforces the historical label against the accepted tokens: a point labelled
 * FM_LABEL_HISTORICAL that equals no complete accepted vertex of the face that holds the pending
 * token or of the face before it is replaced by the nearest of them (same distance, ties to the
 * earliest); historical points are handled first, in sequence order. */
int fm_correct_ex(fm_ctx* ctx, int32_t* cand /*DEV*/, const int32_t* labels /*DEV or NULL*/, int32_t use_history);

/* Verify (Sec. 3.3): one forward pass over main + D candidates, causal among themselves,
 * through all five level stacks.  cand: DEV int32 in [batch, D+1]; cand[b][0] must be the
 * pending main token.  Rows fed per sequence = min(D+1, tokens left).  argmax: DEV int32 out
 * [batch, D+1] (masked argmax per row, -1 for rows not fed) or NULL; logits: DEV float32 out
 * [batch, D+1, V] or NULL; margin: DEV float32 out [batch, D+1] or NULL.
 * Writes keys/values beyond L (invisible until accepted); does not move L; calling it twice
 * is legal and gives the same result. */
int fm_verify(fm_ctx* ctx, const int32_t* cand /*DEV*/, int32_t* argmax /*DEV*/, float* logits /*DEV*/,
              float* margin /*DEV*/);

/* fm_verify for callers that cannot provide scratch memory of their own (no counterpart in the
 * paper).  Some hosts of this library carve the workspace of fm_create out of an arena that is
 * sized and committed once at start-up -- a serving process with a fixed memory plan, a plug-in that
 * is forbidden to call cudaMalloc because an allocation would synchronise the device under its
 * real-time loop -- and want the attention kernel's split-KV scratch (per-group partial results and
 * the ticket counters of the final merge) kept out of that arena.  This call does what fm_verify
 * does, same arguments, same results, but points the attention kernel at a fixed array of
 * FM_STATIC_SCRATCH_BYTES bytes that is part of the library image: every GPU that loads the library
 * holds that many bytes until the process exits.  It allocates nothing (no cudaMalloc, no
 * cudaFree, no allocating library routine); inputs and outputs are still the caller's.
 *   - Limit: the scratch one pass needs (it grows with max_batch * n_kv_heads and with the cache
 *     capacity) must fit in FM_STATIC_SCRATCH_BYTES, else FM_ERR_CAPACITY is returned and nothing
 *     is enqueued.
 *   - Every GPU has its own copy of the array: the device the context was created on must be the
 *     current device at every call (FM_ERR_BAD_STATE otherwise).  The first call on a device looks
 *     up the array's device address; make that first call before any stream capture is begun.
 *   - All contexts and all calls share the one array.  It keeps the previous call's contents (the
 *     call clears the counters that must start at zero), and two calls whose kernels overlap on
 *     the GPU -- different streams, different contexts -- race on it: serialise them. */
#define FM_STATIC_SCRATCH_BYTES (4 * 1024 * 1024)
int fm_verify_static_scratch(fm_ctx* ctx, const int32_t* cand /*DEV*/, int32_t* argmax /*DEV*/, float* logits /*DEV*/,
                             float* margin /*DEV*/);

/* Accept (Sec. 3.3) and roll back: a = 1 + number of leading drafts that equal the backbone's
 * argmax at the previous row; clipped to the rows fed and at an accepted EOS; L += a; the next
 * main token is the argmax at row a-1.  force_tok: DEV int32 [batch, D+1] or NULL, replaces the
 * stored argmax; force_len: DEV int32 [batch] or NULL, replaces a (values 1..D+1).
 * n_acc: DEV int32 out [batch]; emitted: DEV int32 out [batch, D+1] (accepted ids, then -1);
 * kv_len: DEV int32 out [batch, 3] = (L, ceil(L/3), ceil(L/9)).  Any output may be NULL.
 * Errors: BAD_STATE if no fm_verify preceded it. */
int fm_accept(fm_ctx* ctx, const int32_t* force_len /*DEV*/, const int32_t* force_tok /*DEV*/,
              int32_t* n_acc /*DEV*/, int32_t* emitted /*DEV*/, int32_t* kv_len /*DEV*/);

/* One pass of the loop for a host that sits in it (Sec. 3: predict, edit, verify, accept), with HOST
 * buffers: runs the draft modules; copies `cand` in (HOST int32 [batch, D+1], pinned memory makes
 * the copy asynchronous; an entry >= 0 replaces the draft modules' candidate at that slot, an entry
 * < 0 keeps it, slot 0 always stays the pending main token; NULL keeps all); verifies; accepts;
 * copies n_acc [batch], emitted [batch, D+1] (may be NULL) and kv_len [batch, 3] (may be NULL) back to
 * HOST memory and waits for the stream.  Equivalent to fm_draft, fm_verify, fm_accept with the
 * copies in between, in one call.  Errors as those calls. */
int fm_step_host(fm_ctx* ctx, const int32_t* cand /*HOST*/, int32_t* n_acc /*HOST*/, int32_t* emitted /*HOST*/,
                 int32_t* kv_len /*HOST*/);

/* The whole loop (Sec. 3): draft -> (optional teacher edit) -> verify -> accept, until every
 * sequence has emitted 9*max_faces tokens or EOS, or, when max_steps > 0, for exactly max_steps
 * passes (a later call continues where this one stopped).  out_tok: DEV int32 [batch, out_stride]
 * receives the emitted tokens (prompt not included), out_len: DEV int32 [batch], zeroed by the
 * first call after fm_prefill and advanced by every call; both may be NULL.  teacher and stats may
 * be NULL.  plain != 0 accepts only the main token every pass (the one-token-at-a-time baseline
 * on the same kernels).  max_faces == -1 keeps the per-sequence limits set with fm_set_max_faces
 * (tokens beyond out_stride are then not stored).  Synchronous (returns after the last pass).
 * Errors: BAD_STATE, CAPACITY (prompt + 9*max_faces + D + 2 > max_tokens, or out_stride too small). */
int fm_generate(fm_ctx* ctx, int32_t max_faces, int32_t* out_tok /*DEV*/, int32_t out_stride,
                int32_t* out_len /*DEV*/, const fm_teacher* teacher /*HOST struct, DEV arrays*/,
                int32_t plain, int64_t max_steps, fm_stats* stats /*HOST*/);

/* Algorithmic bytes one verify pass must move for the given per-sequence lengths (weights of
 * the stacks that have rows, shorten/upsample, output matrix, K and V entries visible to the
 * rows); kv_len HOST int32 [batch,3] as returned by fm_accept.  For roofline reports. */
double fm_verify_bytes(const fm_ctx* ctx, int32_t batch, const int32_t* kv_len /*HOST*/);

/* Per-kernel-class device timing for roofline reports (no counterpart in the paper).  Between
 * fm_profile_begin and fm_profile_end every weight-streaming GEMM launch and every attention
 * launch is bracketed by a CUDA event pair on the context's stream; fm_profile_end synchronises
 * and sums them.  gemm_bytes counts each launch's weight matrix once (2*M*K bytes). */
typedef struct fm_profile {
  double gemm_ms, gemm_bytes; int64_t gemm_launches;
  double attn_ms; int64_t attn_launches;
} fm_profile;
int fm_profile_begin(fm_ctx* ctx);
/* One kernel class timed alone (no counterpart in the paper): the launches of that class of one
 * verify pass over the current candidates and lengths (cls 0: the weight-streaming GEMMs, 1: the
 * attention launches; same kernels, arguments and data as in the pass) are captured as a CUDA graph
 * and replayed `reps` times after 3 warm-up replays, between two events.  out->gemm_ms /
 * out->attn_ms = milliseconds per replay, *_launches = launches per replay, gemm_bytes = weight bytes
 * per replay (2*M*K per launch).  Synchronous.  The
 * replays overwrite activations and the tentative cache rows of the pass: call fm_prefill (or
 * fm_verify) again before decoding on. */
int fm_profile_class(fm_ctx* ctx, int32_t cls, int32_t reps, fm_profile* out /*HOST*/);
int fm_profile_end(fm_ctx* ctx, fm_profile* out /*HOST*/);

/* How the attention kernel cuts a level's cache (no counterpart in the paper; for reports and
 * tests): slots per chunk, chunks per group (one CTA streams one group; fixed when the context is
 * created) and the number of groups the full cache has.  A (sequence, kv-head) whose cache holds n
 * slots, prefix included, is read by ceil(ceil(n / chunk) / chunks_per_group) CTAs, whose partial
 * results go through the scratch buffers when there is more than one.  level: 0 coordinate,
 * 1 vertex, 2 face.  HOST out pointers, any may be NULL. */
int fm_attention_layout(const fm_ctx* ctx, int32_t level, int32_t* chunk_slots, int32_t* chunks_per_group,
                        int32_t* max_groups);

/* Number of kernels launched by this context since creation (for launch accounting). */
int64_t fm_launch_count(const fm_ctx* ctx);

/* Self-check of the give-up path of the device-side waits (no counterpart in the paper).  Every
 * wait inside the kernels (on a shared-memory barrier that a copy, a tensor-core commit or a peer
 * CTA completes) polls for a bounded number of clock cycles, then records FM_ERR_TIMEOUT in the
 * device status word and lets the kernel finish without touching the data.  This call enqueues one
 * thread that runs the same wait, limited to `limit_cycles` (1 .. 1e8), on a barrier that nothing
 * completes: afterwards fm_device_status returns FM_ERR_TIMEOUT, and fm_prefill clears it.  The
 * kernel always ends by itself. */
int fm_selftest_wait_timeout(fm_ctx* ctx, int64_t limit_cycles);

const char* fm_strerror(int code);
/* Device status word: 0, or FM_ERR_TIMEOUT if a bounded wait inside a kernel gave up, or
 * FM_ERR_INVALID_ARG if a kernel met an out-of-range token id (it then used PAD), or
 * FM_ERR_CAPACITY if the attention kernel was asked to merge more cache groups than it can stage
 * (it then wrote nothing; fm_create sizes the groups so that this does not happen).  The word is
 * cleared by fm_prefill.  Synchronises the stream. */
int fm_device_status(fm_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* FLASHMESH_H */
