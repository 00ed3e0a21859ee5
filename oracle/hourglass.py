"""CPU oracle of the hourglass mesh transformer and its speculative decode loop.

THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  Only the test-suite, the smoke
check and the `cpu_baseline` / `--impl reference` legs of the benchmark may
import it.  It shares no code with the CUDA library and is deliberately plain:
numpy float64, dense masks, no blocking, no fusion.  numpy's matmul and
`scipy.special.erf` are the only library primitives used.

What it follows (FlashMesh, arXiv 2511.15618):
  * Supp. "Hourglass Transformer": 3 coordinates = 1 vertex, 3 vertices = 1 face;
    shortening layers compress, upsampling layers expand, residuals between levels.
  * Sec. 3.1: block = self-attention + conditioning + FFN; `h_s` = hidden before the last
    layer (the split node); Eq. 1 (SP-Block: Linear + residual), Eq. 2 (Upsample to 3).
  * Sec. 3.3: feed main + D drafts with causal masking, accept the main token, accept
    drafts up to the first mismatch, continue from the backbone's output there.
  * Supp. "Optimizations", rules (A) and (B): one draft source per future position.
  * Sec. 3.1 Eq. 1-5 and Supp. "Three-Level Speculative Decoding": the full SP-Block and
    HF-Blocks (`draft_heads == "full"`), the averaged merge of the levels (`avg_levels`), the
    coordinate-only variant of the supplement's ablation (`draft_levels == "coord"`); Sec. 3.2:
    the label head on the point-level features.

Readings taken where the paper is silent: pre-norm
RMSNorm, GELU(erf) FFN without biases, rotate-half RoPE on the level-local index,
conditioning folded in as per-layer prefix keys/values visible to every query,
right-aligned linear shortening of 3 concatenated hiddens, linear upsampling added to the
pre-shorten hidden, longest-matching-prefix acceptance, masked argmax with ties to the
lowest id.

Pins (tests/test_oracle_*.py): reduction to a textbook pre-norm decoder when the upsample
matrices are zero; causality at all three levels; cached multi-row forward == dense
forward == sequential single-row steps (1e-9 in float64, bound 1e-5); speculative output
== plain greedy == brute-force greedy for any draft content; window >= length == full;
RoPE shift invariance; MQA with replicated weights == MHA; bookkeeping closed forms; the
paper's worked draft-coverage example.  Draft *quality* / acceptance statistics of a
trained model: parity unpinned (no trained weights exist here).
"""
from __future__ import annotations

import math

import numpy as np
from scipy.special import erf

STACK_LEVEL = (0, 1, 2, 1, 0)     # coord_down, vertex_down, face, vertex_up, coord_up
RATIO = (1, 3, 9)


# ---------------------------------------------------------------------------------------------
# elementary pieces
# ---------------------------------------------------------------------------------------------
def rms_norm(x, g, eps):
    """RMSNorm: x / sqrt(mean(x^2) + eps) * g over the last axis."""
    return x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps) * g


def gelu(x):
    """Exact GELU, x * Phi(x)."""
    return 0.5 * x * (1.0 + erf(x / math.sqrt(2.0)))


def rope(x, pos, theta):
    """Rotate-half rotary embedding.  x[n, heads, dh], pos[n]; pairs (i, i + dh/2),
    angle = pos * theta^(-2i/dh).  theta == 0 disables it."""
    if theta == 0:
        return x
    dh = x.shape[-1]
    half = dh // 2
    freq = theta ** (-2.0 * np.arange(half, dtype=np.float64) / dh)
    ang = np.asarray(pos, dtype=np.float64)[:, None] * freq[None, :]
    c = np.cos(ang)[:, None, :].astype(x.dtype)
    s = np.sin(ang)[:, None, :].astype(x.dtype)
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def softmax_rows(s):
    m = np.max(s, axis=-1, keepdims=True)
    e = np.exp(s - m)
    return e / np.sum(e, axis=-1, keepdims=True)


def allowed_mask(cfg, target_index):
    """Ids that may be emitted as mesh token t_i: coordinate bins always; EOS only where a
    face starts (i % 9 == 0) and only if the configuration allows it; BOS/PAD never."""
    m = np.zeros(cfg.vocab, dtype=bool)
    m[:cfg.n_bins] = True
    if cfg.allow_eos and target_index % 9 == 0:
        m[cfg.eos] = True
    return m


def masked_top2(cfg, logits, target_index):
    """(argmax over allowed ids with ties to the lowest id, top1 - top2 margin)."""
    z = np.where(allowed_mask(cfg, target_index), logits, -np.inf)
    best = int(np.argmax(z))                      # numpy returns the first maximum
    rest = z.copy()
    rest[best] = -np.inf
    return best, float(z[best] - np.max(rest))


def draft_source(n, j, draft_len, levels="three"):
    """Which head predicts draft offset j (target t_{n+j}) when the pending main token is t_n.

    levels == "coord" is the variant of Supp. "Ablation on multi-level speculative decoding":
    no point- or face-level modules, coordinate head j predicts offset j.  Otherwise:

    Supp. "Optimizations".  The levels fire at their own rows: the point level where a vertex
    starts (n % 3 == 0), the face level where a face starts (n % 9 == 0); rows in between
    reuse the most recent predictions of those levels (Supp. "Integrating the three levels").
    With v* = n // 3 and f* = n // 9 the most recent point-level row is 3 v*, the most recent
    face-level row 9 f*.
      * Rule (B): offsets 1 and 2 always come from the coordinate heads; the higher levels
        drop the point that holds the main token.
      * The point level then covers the next two whole points, vertices v*+1 and v*+2,
        wherever the face boundary lies (worked step (1): predicting the first coordinate
        of a face's last vertex, the point level gives the six tokens of the next face's
        first two vertices; step (2): one token later those predictions are reused).
      * Rule (A): where the most recent point-level row was also a face-level row
        (v* % 3 == 0) the point-level predictions were removed, and the face level covers
        the rest of the face it started: face head 1 predicts the face that holds t_n.
      * Targets beyond vertex v*+2 (the paper's 9-9 model stops there and drafts 8, 7 or 6
        tokens depending on the row; a fixed draft length needs a source for them) come from
        the face level: face head e predicts face f* + e - 1.
    Every offset has exactly one source (no averaging).  Returns (level, head, slot):
    level 0 -> coordinate head `head` (1-based); level 1 -> vertex head `head` (vertex
    v* + head), slot r of its 3 upsampled features; level 2 -> face head `head` (face
    f* + head - 1), slot r of its 9 features."""
    p = n + j
    if j <= 2 or levels == "coord":
        return (0, j, 0)
    ev = p // 3 - n // 3
    if ev <= 2:
        if (n // 3) % 3 == 0 and p // 9 == n // 9:
            return (2, 1, p % 9)
        return (1, ev, p % 3)
    return (2, p // 9 - n // 9 + 1, p % 9)


# ---------------------------------------------------------------------------------------------
# the definition: dense forward over a whole prefix, no cache
# ---------------------------------------------------------------------------------------------
def _split_qkv(cfg, qkv):
    H, Hkv, dh = cfg.n_heads, cfg.n_kv_heads, cfg.head_dim
    n = qkv.shape[0]
    q = qkv[:, :H * dh].reshape(n, H, dh)
    k = qkv[:, H * dh:(H + Hkv) * dh].reshape(n, Hkv, dh)
    v = qkv[:, (H + Hkv) * dh:].reshape(n, Hkv, dh)
    return q, k, v


def _prefix_kv(cfg, lw, cond, dt):
    """Per-layer prefix keys/values: this layer's K and V projections of norm1(c), un-rotated."""
    H, Hkv, dh = cfg.n_heads, cfg.n_kv_heads, cfg.head_dim
    a = rms_norm(cond.astype(dt), lw["g1"].astype(dt), cfg.norm_eps)
    kv = a @ lw["Wqkv"][H * dh:].astype(dt).T
    P = cond.shape[0]
    return kv[:, :Hkv * dh].reshape(P, Hkv, dh), kv[:, Hkv * dh:].reshape(P, Hkv, dh)


def _attend(cfg, q, keys, vals, mask):
    """q[n,H,dh]; keys/vals[m,Hkv,dh]; mask[n,m] bool.  Softmax over visible keys, scale 1/sqrt(dh)."""
    H, Hkv, dh = cfg.n_heads, cfg.n_kv_heads, cfg.head_dim
    out = np.zeros_like(q)
    for h in range(H):
        hk = (h * Hkv) // H
        s = (q[:, h, :] @ keys[:, hk, :].T) / math.sqrt(dh)
        s = np.where(mask, s, -np.inf)
        out[:, h, :] = softmax_rows(s) @ vals[:, hk, :]
    return out


def layer_full(cfg, lw, x, cond, window, dt):
    """One pre-norm block on all positions 0..n-1 of one level."""
    n = x.shape[0]
    P = cond.shape[0]
    a = rms_norm(x, lw["g1"].astype(dt), cfg.norm_eps)
    q, k, v = _split_qkv(cfg, a @ lw["Wqkv"].astype(dt).T)
    pos = np.arange(n)
    q, k = rope(q, pos, cfg.rope_theta), rope(k, pos, cfg.rope_theta)
    kp, vp = _prefix_kv(cfg, lw, cond, dt)
    keys, vals = np.concatenate([kp, k]), np.concatenate([vp, v])
    i, j = pos[:, None], pos[None, :]
    causal = (j <= i) & ((j >= i - window + 1) if window > 0 else True)
    mask = np.concatenate([np.ones((n, P), dtype=bool), causal], axis=1)
    o = _attend(cfg, q, keys, vals, mask).reshape(n, -1)
    x = x + o @ lw["Wo"].astype(dt).T
    x = x + gelu(rms_norm(x, lw["g2"].astype(dt), cfg.norm_eps) @ lw["W1"].astype(dt).T) @ lw["W2"].astype(dt).T
    return x


def _shorten_full(S, h, dt):
    """Right-aligned 3:1 shortening: row v = S . [h_{3v-2}; h_{3v-1}; h_{3v}], zeros below 0."""
    n, d = h.shape
    m = -(-n // 3)
    out = np.zeros((m, d), dtype=dt)
    for v in range(m):
        parts = [h[i] if i >= 0 else np.zeros(d, dtype=dt) for i in (3 * v - 2, 3 * v - 1, 3 * v)]
        out[v] = S.astype(dt) @ np.concatenate(parts)
    return out


def forward_full(cfg, w, cond, u, dtype=np.float64, return_hidden=False):
    """Logits [len(u), V] of the hourglass on inputs u_0..u_{n-1} (u_0 = BOS, u_i = t_{i-1});
    row i predicts mesh token t_i."""
    dt = dtype
    d = cfg.d_model
    u = np.asarray(u)
    n = len(u)
    cond = np.asarray(cond)

    def run(x, s):
        for lw in w["stacks"][s]:
            x = layer_full(cfg, lw, x, cond, cfg.window[STACK_LEVEL[s]], dt)
        return x

    hc = run(w["E"].astype(dt)[u], 0)
    hv = run(_shorten_full(w["S_cv"], hc, dt), 1)
    hf = run(_shorten_full(w["S_vf"], hv, dt), 2)
    up_f = hf @ w["U_fv"].astype(dt).T                         # [nf, 3d]
    v1 = np.stack([hv[v] + up_f[v // 3, (v % 3) * d:(v % 3 + 1) * d] for v in range(hv.shape[0])])
    hv2 = run(v1, 3)
    up_v = hv2 @ w["U_vc"].astype(dt).T                        # [nv, 3d]
    c1 = np.stack([hc[i] + up_v[i // 3, (i % 3) * d:(i % 3 + 1) * d] for i in range(n)])
    hc2 = run(c1, 4)
    logits = rms_norm(hc2, w["g_out"].astype(dt), cfg.norm_eps) @ w["W_out"].astype(dt).T
    if return_hidden:
        return logits, {"hc": hc, "hv": hv, "hf": hf, "hv2": hv2, "hc2": hc2}
    return logits


def greedy_full(cfg, w, cond, prompt, n_tokens, dtype=np.float64):
    """Brute-force definition of the decoder's output: token-by-token greedy decoding, each
    step a dense forward over the whole prefix.  Stops at EOS or after n_tokens new tokens."""
    u = [cfg.bos] + [int(t) for t in prompt]
    out = []
    while len(out) < n_tokens:
        i = len(u) - 1
        tok, _ = masked_top2(cfg, forward_full(cfg, w, cond, u, dtype)[-1], i)
        out.append(tok)
        u.append(tok)
        if tok == cfg.eos:
            break
    return out


# ---------------------------------------------------------------------------------------------
# cached, incremental, multi-row implementation (one sequence)
# ---------------------------------------------------------------------------------------------
class OracleSeq:
    """One sequence decoded with per-level KV caches.

    State: L = inputs consumed (u_0..u_{L-1}), pending main token t_{L-1}, finished flag,
    `t_end` = index one past the last mesh token to produce.  Everything a forward pass
    writes beyond L is tentative and becomes visible only when `accept` moves L."""

    def __init__(self, cfg, w, dtype=np.float64):
        self.cfg, self.dt = cfg, dtype
        self.w = self._cast(w)
        self.L = 0
        self.main = None
        self.done = False
        self.prompt_len = 0
        self.t_end = cfg.max_tokens - cfg.draft_len - 2
        self.cand = None
        self.rows = 0
        self.o = None

    def _cast(self, w):
        dt = self.dt
        if isinstance(w, dict):
            return {k: self._cast(v) for k, v in w.items()}
        if isinstance(w, list):
            return [self._cast(v) for v in w]
        return np.asarray(w, dtype=dt)

    # -- state ------------------------------------------------------------------------------
    def _alloc(self, cond):
        cfg, dt = self.cfg, self.dt
        d, Hkv, dh = cfg.d_model, cfg.n_kv_heads, cfg.head_dim
        cap = [cfg.max_tokens, -(-cfg.max_tokens // 3) + 1, -(-cfg.max_tokens // 9) + 1]
        self.cond = np.asarray(cond, dtype=dt)
        self.K = [[np.zeros((cap[STACK_LEVEL[s]], Hkv, dh), dtype=dt) for _ in self.w["stacks"][s]] for s in range(5)]
        self.V = [[np.zeros((cap[STACK_LEVEL[s]], Hkv, dh), dtype=dt) for _ in self.w["stacks"][s]] for s in range(5)]
        self.KP = [[None] * len(self.w["stacks"][s]) for s in range(5)]
        self.VP = [[None] * len(self.w["stacks"][s]) for s in range(5)]
        for s in range(5):
            for l, lw in enumerate(self.w["stacks"][s]):
                self.KP[s][l], self.VP[s][l] = _prefix_kv(cfg, lw, self.cond, dt)
        self.hc = np.zeros((cap[0], d), dtype=dt)       # coord-down output per position
        self.hv = np.zeros((cap[1], d), dtype=dt)       # vertex-down output per vertex
        self.up_f = np.zeros((cap[2], 3 * d), dtype=dt)  # U_fv . hf_f
        self.up_v = np.zeros((cap[1], 3 * d), dtype=dt)  # U_vc . hv'_v
        self.zc = np.zeros((cap[0], d), dtype=dt)       # split-node hiddens (input of last layer)
        self.zv = np.zeros((cap[1], d), dtype=dt)
        self.zf = np.zeros((cap[2], d), dtype=dt)

    def kv_len(self):
        L = self.L
        return (L, -(-L // 3), -(-L // 9))

    # -- one stack on a run of consecutive level positions ------------------------------------
    def _stack_rows(self, s, x, p0, stash=None):
        cfg, dt = self.cfg, self.dt
        H, Hkv, dh = cfg.n_heads, cfg.n_kv_heads, cfg.head_dim
        level = STACK_LEVEL[s]
        W = cfg.window[level]
        n = x.shape[0]
        if n == 0:
            return x
        pos = np.arange(p0, p0 + n)
        P = cfg.n_prefix
        layers = self.w["stacks"][s]
        for l, lw in enumerate(layers):
            if stash is not None and l == len(layers) - 1:
                stash[p0:p0 + n] = x
            a = rms_norm(x, lw["g1"], cfg.norm_eps)
            q, k, v = _split_qkv(cfg, a @ lw["Wqkv"].T)
            q, k = rope(q, pos, cfg.rope_theta), rope(k, pos, cfg.rope_theta)
            self.K[s][l][p0:p0 + n] = k
            self.V[s][l][p0:p0 + n] = v
            lo = max(0, p0 - W + 1) if W > 0 else 0
            kpos = np.arange(lo, p0 + n)
            keys = np.concatenate([self.KP[s][l], self.K[s][l][lo:p0 + n]])
            vals = np.concatenate([self.VP[s][l], self.V[s][l][lo:p0 + n]])
            i, j = pos[:, None], kpos[None, :]
            vis = (j <= i) & ((j >= i - W + 1) if W > 0 else True)
            mask = np.concatenate([np.ones((n, P), dtype=bool), vis], axis=1)
            o = _attend(cfg, q, keys, vals, mask).reshape(n, -1)
            x = x + o @ lw["Wo"].T
            x = x + gelu(rms_norm(x, lw["g2"], cfg.norm_eps) @ lw["W1"].T) @ lw["W2"].T
        if stash is not None and len(layers) == 0:
            stash[p0:p0 + n] = x
        return x

    def _shorten_rows(self, S, h, first, count):
        d = self.cfg.d_model
        out = np.zeros((count, d), dtype=self.dt)
        for r in range(count):
            v = first + r
            parts = [h[i] if i >= 0 else np.zeros(d, dtype=self.dt) for i in (3 * v - 2, 3 * v - 1, 3 * v)]
            out[r] = S @ np.concatenate(parts)
        return out

    def forward_rows(self, u):
        """Feed inputs u at positions L..L+n-1 (causal among themselves); return logits [n,V].
        Writes tentative K/V and hourglass state beyond L; does not move L."""
        cfg, w, d = self.cfg, self.w, self.cfg.d_model
        n = len(u)
        L = self.L
        assert L + n <= cfg.max_tokens
        # coordinate level, downward
        hc = self._stack_rows(0, w["E"][np.asarray(u)], L)
        self.hc[L:L + n] = hc
        # vertex rows: multiples of 3 in [L, L+n-1]
        v0, v1 = -(-L // 3), (L + n - 1) // 3
        nv = max(0, v1 - v0 + 1)
        hv = self._stack_rows(1, self._shorten_rows(w["S_cv"], self.hc, v0, nv), v0)
        self.hv[v0:v0 + nv] = hv
        # face rows: multiples of 9
        f0, f1 = -(-L // 9), (L + n - 1) // 9
        nf = max(0, f1 - f0 + 1)
        hf = self._stack_rows(2, self._shorten_rows(w["S_vf"], self.hv, f0, nf), f0, stash=self.zf)
        if nf:
            self.up_f[f0:f0 + nf] = hf @ w["U_fv"].T
        # vertex level, upward
        x = np.stack([self.hv[v] + self.up_f[v // 3, (v % 3) * d:(v % 3 + 1) * d]
                      for v in range(v0, v0 + nv)]) if nv else np.zeros((0, d), dtype=self.dt)
        hv2 = self._stack_rows(3, x, v0, stash=self.zv)
        if nv:
            self.up_v[v0:v0 + nv] = hv2 @ w["U_vc"].T
        # coordinate level, upward
        x = np.stack([self.hc[i] + self.up_v[i // 3, (i % 3) * d:(i % 3 + 1) * d] for i in range(L, L + n)])
        hc2 = self._stack_rows(4, x, L, stash=self.zc)
        return rms_norm(hc2, w["g_out"], cfg.norm_eps) @ w["W_out"].T

    # -- the six operations -------------------------------------------------------------------
    def prefill(self, cond, prompt, max_faces=None, chunk=None):
        """Consume BOS + prompt; afterwards L = 1 + len(prompt) and the first main token is pending.
        `chunk` feeds the inputs that many rows at a time (same result as one dense pass: the
        cached rows of a later chunk see the earlier ones through the caches); long prompts
        need it to keep the score matrices small.  Returns the logits of the last chunk."""
        cfg = self.cfg
        self._alloc(cond)
        self.L = 0
        self.done = False
        self.prompt_len = len(prompt)
        if max_faces is not None:
            self.t_end = self.prompt_len + 9 * max_faces
        u = [cfg.bos] + [int(t) for t in prompt]
        step = len(u) if not chunk else int(chunk)
        for i in range(0, len(u), step):
            logits = self.forward_rows(u[i:i + step])
            self.L = min(len(u), i + step)
        self.main, self.main_margin = masked_top2(cfg, logits[-1], self.L - 1)
        if self.L - 1 >= self.t_end:
            self.done = True
        return logits

    def set_max_faces(self, max_faces):
        self.t_end = self.prompt_len + 9 * max_faces
        self.done = self.done or (self.L - 1 >= self.t_end)

    # -- draft modules (Sec. 3.1; Supp. "Three-Level Speculative Decoding") ----------------------
    def _cache_attend(self, s, q, vis_pos):
        """Attention of draft queries q[m,H,dh] (rotated) over the cache of the last layer of
        stack s: the prefix keys and the accepted entries that the row at `vis_pos` sees
        (positions max(0, vis_pos - W + 1) .. vis_pos).  Returns [m, H*dh]."""
        cfg = self.cfg
        l = len(self.w["stacks"][s]) - 1
        W = cfg.window[STACK_LEVEL[s]]
        lo = max(0, vis_pos - W + 1) if W > 0 else 0
        keys = np.concatenate([self.KP[s][l], self.K[s][l][lo:vis_pos + 1]])
        vals = np.concatenate([self.VP[s][l], self.V[s][l][lo:vis_pos + 1]])
        mask = np.ones((q.shape[0], keys.shape[0]), dtype=bool)
        return _attend(cfg, q, keys, vals, mask).reshape(q.shape[0], -1)

    def _sp_block(self, z, hw, level, pos):
        """Eq. 1: h^(d) = Linear(CA(SA(h_s), c)) + h_s for one head.  Reduced heads: the attention
        is left out, h + A rms(h).  Full heads: the attention (self-attention and conditioning in
        one softmax, as in every block of this model) reads the cache of the backbone's last
        layer at this level -- the layer whose input the split-node hiddens are -- with the
        head's own query and output projections: y = h + Wo Attn(Wq rms(h, ga)); then
        h^(d) = h + A rms(y, g)."""
        cfg = self.cfg
        y = z
        if cfg.draft_heads == "full":
            s = (4, 3, 2)[level]
            a = rms_norm(z, hw["ga"], cfg.norm_eps)
            q = rope((hw["Wq"] @ a).reshape(1, cfg.n_heads, cfg.head_dim), [pos], cfg.rope_theta)
            y = z + hw["Wo"] @ self._cache_attend(s, q, pos)[0]
        return z + hw["A"] @ rms_norm(y, hw["g"], cfg.norm_eps)

    def _hf_block(self, x, hw, level, qpos, vis_pos):
        """Eq. 3-5: an upsampled feature for level position `qpos` queries the backbone's cache
        at that level (its last layer, entries up to the last accepted position `vis_pos`) with
        the offset's own W_q, and the offset's own FFN maps the attention output back:
        x + FFN(Attn(W_q rms(x), K, V)).  Reduced heads: identity."""
        cfg = self.cfg
        if cfg.draft_heads != "full":
            return x
        s = (4, 3)[level]
        a = rms_norm(x, hw["g"], cfg.norm_eps)
        q = rope((hw["Wq"] @ a).reshape(1, cfg.n_heads, cfg.head_dim), [qpos], cfg.rope_theta)
        o = self._cache_attend(s, q, vis_pos)[0]
        return x + hw["W2"] @ gelu(hw["W1"] @ o)

    def draft_features(self):
        """Coordinate-level features of every head at the last accepted split nodes, keyed like
        draft_source's result, and the point-level features they came from (for the label head):
        points[(1, e, 0)] for vertex head e, points[(2, e, rv)] for vertex rv of face head e."""
        cfg, w, d = self.cfg, self.w, self.cfg.d_model
        n = self.L - 1
        vs, fs = n // 3, n // 9
        feats, points = {}, {}
        for k in range(1, cfg.n_coord_heads + 1):                      # coordinate level: SP only
            feats[(0, k, 0)] = self._sp_block(self.zc[n], w["heads_c"][k - 1], 0, n)
        if cfg.draft_levels != "three":
            return feats, points
        hf_vc = w.get("hf_vc", [None] * 6)
        hf_fv = w.get("hf_fv", [None] * (3 * cfg.n_face_heads))
        hf_fc = w.get("hf_fc", [None] * (9 * cfg.n_face_heads))
        for e in (1, 2):                                               # point level: SP, upsample, one HF
            yv = self._sp_block(self.zv[vs], w["heads_v"][e - 1], 1, vs)
            points[(1, e, 0)] = yv
            tri = w["U_vc"] @ yv                                       # Eq. 2: one vertex -> 3 coordinates
            for r in range(3):
                feats[(1, e, r)] = self._hf_block(tri[r * d:(r + 1) * d], hf_vc[3 * e + r - 3], 0, 3 * (vs + e) + r, n)
        for e in range(1, cfg.n_face_heads + 1):                       # face level: SP, upsample, HF, upsample, HF
            yf = self._sp_block(self.zf[fs], w["heads_f"][e - 1], 2, fs)       # head e drafts face f* + e - 1
            tri = w["U_fv"] @ yf                                       # one face -> 3 vertices
            for rv in range(3):
                xv = self._hf_block(tri[rv * d:(rv + 1) * d], hf_fv[3 * (e - 1) + rv], 1, 3 * (fs + e - 1) + rv, vs)
                points[(2, e, rv)] = xv
                sub = w["U_vc"] @ xv                                   # each vertex -> 3 coordinates
                for r in range(3):
                    feats[(2, e, 3 * rv + r)] = self._hf_block(sub[r * d:(r + 1) * d], hf_fc[9 * (e - 1) + 3 * rv + r], 0,
                                                               9 * (fs + e - 1) + 3 * rv + r, n)
        return feats, points

    def _all_sources(self, n, j):
        """Every level that predicts offset j (Supp. "Integrating the three levels", before the
        optimisation rules pick one): the coordinate head if there is one for j, the point level
        for the next two vertices, the face level for the faces its heads draft (never the
        vertex that holds the pending token: that one is the backbone's)."""
        cfg = self.cfg
        p = n + j
        out = []
        if j <= cfg.n_coord_heads:
            out.append((0, j, 0))
        if cfg.draft_levels == "three":
            ev, ef = p // 3 - n // 3, p // 9 - n // 9 + 1
            if 1 <= ev <= 2:
                out.append((1, ev, p % 3))
            if ev >= 1 and 1 <= ef <= cfg.n_face_heads:
                out.append((2, ef, p % 9))
        return out

    def draft(self):
        """Candidates [main, d_1..d_D] from the draft modules at the last accepted split nodes,
        with the draft logits [D,V] and their top-2 margins.  With cfg.avg_levels the logits of
        an offset are the logarithm of the mean of the levels' softmax distributions."""
        cfg, w = self.cfg, self.w
        D = cfg.draft_len
        if self.done:
            return [cfg.pad] * (D + 1), np.zeros((D, cfg.vocab)), [0.0] * D
        n = self.L - 1
        feats, self.points = self.draft_features()

        def logits_of(f):
            return w["W_out"] @ rms_norm(f, w["g_out"], cfg.norm_eps)

        cand, dl, margins = [self.main], [], []
        for j in range(1, D + 1):
            if cfg.avg_levels:
                probs = [softmax_rows(logits_of(feats[src])[None])[0] for src in self._all_sources(n, j)]
                logits = np.log(np.mean(probs, axis=0))
            else:
                logits = logits_of(feats[draft_source(n, j, D, cfg.draft_levels)])
            tok, mg = masked_top2(cfg, logits, n + j)
            cand.append(tok)
            dl.append(logits)
            margins.append(mg)
        return cand, np.stack(dl) if D else np.zeros((0, cfg.vocab)), margins

    def draft_labels(self):
        """Sec. 3.2: a label head (a linear layer, here behind an RMSNorm) on the point-level
        feature of every drafted point.  Slot s of the candidate row holds mesh token n + s; a
        point starts at slot s >= 1 when (n + s) % 3 == 0 and its three tokens are drafts of the
        row.  Its feature is the point-level feature in the pipeline of the head that drafts its
        last coordinate.  Returns (labels[D+1] with -1 where no point starts, margins[D+1]).
        Call after draft()."""
        cfg, w = self.cfg, self.w
        D = cfg.draft_len
        labels, margins = [-1] * (D + 1), [0.0] * (D + 1)
        if self.done or cfg.draft_levels != "three":
            return labels, margins
        n = self.L - 1
        for s in range(1, D - 1):
            if (n + s) % 3 != 0:
                continue
            level, head, slot = draft_source(n, s + 2, D)
            f = self.points[(1, head, 0)] if level == 1 else self.points[(2, head, slot // 3)]
            z = w["label"]["W"] @ rms_norm(f, w["label"]["g"], cfg.norm_eps)
            best = int(np.argmax(z))
            rest = np.delete(z, best)
            labels[s], margins[s] = best, float(z[best] - rest.max())
        return labels, margins

    def verify(self, cand):
        """One forward pass over the candidates (Sec. 3.3).  Rows fed = min(D+1, tokens left).
        Returns (argmax per row, logits, margins); rows that were not fed hold -1."""
        cfg = self.cfg
        D = cfg.draft_len
        self.cand = [int(t) for t in cand]
        if self.done:
            self.rows, self.o = 0, [-1] * (D + 1)
            return self.o, np.zeros((D + 1, cfg.vocab)), [0.0] * (D + 1)
        assert self.cand[0] == self.main, "candidate 0 must be the pending main token"
        rows = min(D + 1, self.t_end - (self.L - 1))
        logits = self.forward_rows(self.cand[:rows])
        o, mg = [-1] * (D + 1), [0.0] * (D + 1)
        for j in range(rows):
            o[j], mg[j] = masked_top2(cfg, logits[j], self.L + j)
        full = np.zeros((D + 1, cfg.vocab))
        full[:rows] = logits
        self.rows, self.o, self.o_margin = rows, o, mg
        return o, full, mg

    def accept(self, force_len=None, force_tok=None):
        """Greedy longest-matching-prefix acceptance and rollback.  Returns (n_acc, emitted, kv_len)."""
        cfg = self.cfg
        D = cfg.draft_len
        if self.done or self.rows == 0:
            return 0, [-1] * (D + 1), self.kv_len()
        o = list(self.o) if force_tok is None else [int(t) for t in force_tok]
        a = 1
        while a < self.rows and self.cand[a] == o[a - 1]:
            a += 1
        if force_len is not None:
            a = int(force_len)
        a = max(1, min(a, self.rows))
        for j in range(a):                                   # an accepted EOS ends the sequence
            if self.cand[j] == cfg.eos:
                a = j + 1
                self.done = True
                break
        emitted = self.cand[:a] + [-1] * (D + 1 - a)
        self.L += a
        self.main = o[a - 1]
        if self.L - 1 >= self.t_end:
            self.done = True
        self.rows = 0
        return a, emitted, self.kv_len()

    def generate(self, max_faces, draft_fn=None, force_plain=False):
        """Decode until EOS or 9*max_faces new tokens.  draft_fn(seq, cand) may edit the drafts."""
        self.set_max_faces(max_faces)
        out, acc = [], []
        while not self.done:
            cand, _, _ = self.draft()
            if draft_fn is not None:
                cand = draft_fn(self, list(cand))
            self.verify(cand)
            a, em, _ = self.accept(force_len=1 if force_plain else None)
            out += em[:a]
            acc.append(a)
        return out, acc
