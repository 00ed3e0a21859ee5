"""Pins of the oracle's model arithmetic against things the mathematics fixes."""
import math

import numpy as np
import pytest

import fm_synth as S
from oracle import hourglass as O


def _setup(**kw):
    cfg = S.toy_config(**kw)
    return cfg, S.make_weights(cfg), S.make_condition(cfg)


def _tokens(cfg, n, seed=0):
    rng = np.random.default_rng(seed)
    return [cfg.bos] + [int(t) for t in rng.integers(0, cfg.n_bins, n - 1)]


# ------------------------------------------------------------------------------ elementary
def test_gelu_closed_form_values():
    # GELU(x) = x * Phi(x): Phi(0)=1/2, Phi(1)=0.8413447460685429, Phi(-1)=1-Phi(1)
    x = np.array([0.0, 1.0, -1.0, 3.0])
    want = [0.0, 0.8413447460685429, -(1 - 0.8413447460685429), 3 * 0.9986501019683699]
    assert np.allclose(O.gelu(x), want, atol=1e-14)


def test_rms_norm_gives_unit_rms_and_scales_by_gain():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((5, 64)) * 7.0
    y = O.rms_norm(x, np.ones(64), 0.0)
    assert np.allclose(np.sqrt(np.mean(y * y, axis=-1)), 1.0)
    g = rng.standard_normal(64)
    assert np.allclose(O.rms_norm(x, g, 0.0), y * g)
    assert np.allclose(O.rms_norm(3.0 * x, g, 0.0), O.rms_norm(x, g, 0.0))      # scale invariance


def test_rope_is_a_rotation_and_depends_on_relative_position_only():
    rng = np.random.default_rng(2)
    q, k = rng.standard_normal((1, 1, 32)), rng.standard_normal((1, 1, 32))
    assert np.allclose(O.rope(q, [0], 10000.0), q)
    for m, n in [(5, 3), (1005, 1003), (140002, 140000)]:
        qm, kn = O.rope(q, [m], 10000.0), O.rope(k, [n], 10000.0)
        assert np.isclose(np.linalg.norm(qm), np.linalg.norm(q))
        ref = np.sum(O.rope(q, [2], 10000.0) * k)
        assert np.isclose(np.sum(qm * kn), ref, atol=1e-9)
    # first pair (i=0, i+dh/2) rotates by exactly `pos` radians, last pair by pos*theta^(-(dh-2)/dh)
    e = np.zeros((1, 1, 32)); e[0, 0, 0] = 1.0
    r = O.rope(e, [0.5], 10000.0)
    assert np.isclose(r[0, 0, 0], math.cos(0.5)) and np.isclose(r[0, 0, 16], math.sin(0.5))
    e = np.zeros((1, 1, 32)); e[0, 0, 15] = 1.0
    r = O.rope(e, [7.0], 10000.0)
    ang = 7.0 * 10000.0 ** (-30.0 / 32.0)
    assert np.isclose(r[0, 0, 15], math.cos(ang)) and np.isclose(r[0, 0, 31], math.sin(ang))


def test_masked_top2_ties_and_mask():
    cfg = S.toy_config(allow_eos=1)
    z = np.zeros(cfg.vocab); z[[3, 7]] = 2.0; z[cfg.bos] = 9.0; z[cfg.pad] = 9.0; z[cfg.eos] = 5.0
    assert O.masked_top2(cfg, z, 4) == (3, 0.0)            # tie -> lowest id; specials masked
    tok, mg = O.masked_top2(cfg, z, 9)                      # EOS allowed where a face starts
    assert tok == cfg.eos and mg == 3.0
    assert O.masked_top2(cfg.with_(allow_eos=0), z, 9)[0] == 3


# ----------------------------------------------------------- reduction to a textbook decoder
def _textbook_decoder(cfg, w, cond, u, layers, window):
    """Independent, loop-style pre-norm decoder with prefix keys/values (test-local)."""
    d, H, Hkv, dh = cfg.d_model, cfg.n_heads, cfg.n_kv_heads, cfg.head_dim
    X = [w["E"][t].astype(np.float64) for t in u]
    norm = lambda x, g: x * g / math.sqrt(float(np.dot(x, x)) / len(x) + cfg.norm_eps)

    def rot(vec, p):
        out = vec.copy()
        for i in range(dh // 2):
            a = p * cfg.rope_theta ** (-2.0 * i / dh)
            out[i] = vec[i] * math.cos(a) - vec[i + dh // 2] * math.sin(a)
            out[i + dh // 2] = vec[i + dh // 2] * math.cos(a) + vec[i] * math.sin(a)
        return out

    for lw in layers:
        Wq, Wk, Wv = np.split(lw["Wqkv"].astype(np.float64), [H * dh, (H + Hkv) * dh])
        pk = [Wk @ norm(c.astype(np.float64), lw["g1"]) for c in cond]
        pv = [Wv @ norm(c.astype(np.float64), lw["g1"]) for c in cond]
        A = [norm(x, lw["g1"]) for x in X]
        Y = []
        for i, x in enumerate(X):
            att = np.zeros(H * dh)
            for h in range(H):
                hk = h * Hkv // H
                sl, slk = slice(h * dh, (h + 1) * dh), slice(hk * dh, (hk + 1) * dh)
                q = rot((Wq @ A[i])[sl], i)
                ks = [p[slk] for p in pk]; vs = [p[slk] for p in pv]
                for j in range(i + 1):
                    if window > 0 and j < i - window + 1:
                        continue
                    ks.append(rot((Wk @ A[j])[slk], j)); vs.append((Wv @ A[j])[slk])
                sc = np.array([float(np.dot(q, kk)) / math.sqrt(dh) for kk in ks])
                pr = np.exp(sc - sc.max()); pr /= pr.sum()
                att[sl] = sum(p_ * v_ for p_, v_ in zip(pr, vs))
            y = x + lw["Wo"].astype(np.float64) @ att
            hdn = lw["W1"].astype(np.float64) @ norm(y, lw["g2"])
            act = np.array([0.5 * t * (1 + math.erf(t / math.sqrt(2))) for t in hdn])
            Y.append(y + lw["W2"].astype(np.float64) @ act)
        X = Y
    return np.stack([w["W_out"].astype(np.float64) @ norm(x, w["g_out"]) for x in X])


@pytest.mark.parametrize("window,kv", [(0, 2), (5, 2), (0, 1)])
def test_zero_upsample_reduces_to_plain_decoder(window, kv):
    cfg, w, cond = _setup(layers=(2, 1, 1, 1, 1), window=(window, 0, 0), n_kv_heads=kv)
    w["U_fv"][:] = 0.0
    w["U_vc"][:] = 0.0
    u = _tokens(cfg, 14)
    got = O.forward_full(cfg, w, cond, u)
    want = _textbook_decoder(cfg, w, cond, u, w["stacks"][0] + w["stacks"][4], window)
    assert np.abs(got - want).max() < 1e-10


def test_upsample_matrices_matter():
    cfg, w, cond = _setup()
    u = _tokens(cfg, 14)
    a = O.forward_full(cfg, w, cond, u)
    w["U_vc"][:] = 0.0
    assert np.abs(a - O.forward_full(cfg, w, cond, u)).max() > 1e-3


# ------------------------------------------------------------------------------ hourglass
def test_causality_at_all_levels():
    cfg, w, cond = _setup(layers=(1, 2, 2, 1, 1))
    u = _tokens(cfg, 30)
    base, hb = O.forward_full(cfg, w, cond, u, return_hidden=True)
    for j in (1, 9, 13, 18, 29):
        u2 = list(u); u2[j] = (u2[j] + 1) % cfg.n_bins
        got, hg = O.forward_full(cfg, w, cond, u2, return_hidden=True)
        assert np.array_equal(got[:j], base[:j])
        assert np.abs(got[j] - base[j]).max() > 0
        nv = len([v for v in range(hb["hv"].shape[0]) if 3 * v < j])
        nf = len([f for f in range(hb["hf"].shape[0]) if 9 * f < j])
        assert np.array_equal(hg["hv"][:nv], hb["hv"][:nv]) and np.array_equal(hg["hf"][:nf], hb["hf"][:nf])
        assert np.array_equal(hg["hv2"][:nv], hb["hv2"][:nv])
        if 3 * nv < hb["hv"].shape[0] * 3 and nv < hb["hv"].shape[0]:
            assert np.abs(hg["hv"][nv] - hb["hv"][nv]).max() > 0       # vertex ceil(j/3) does see input j


def test_level_lengths_and_shorten_alignment():
    cfg, w, cond = _setup()
    for n in (1, 3, 4, 9, 10, 19):
        _, h = O.forward_full(cfg, w, cond, _tokens(cfg, n), return_hidden=True)
        assert h["hv"].shape[0] == -(-n // 3) and h["hf"].shape[0] == -(-n // 9)
    # vertex row 0 pools only input 0 (zeros stand for positions -2, -1): check by linearity
    _, h = O.forward_full(cfg.with_(layers=(0, 0, 0, 0, 0)), {**w, "stacks": [[], [], [], [], []]}, cond,
                          _tokens(cfg, 4), return_hidden=True)
    d = cfg.d_model
    e = w["E"].astype(np.float64)
    u = _tokens(cfg, 4)
    S_cv = w["S_cv"].astype(np.float64)
    assert np.allclose(h["hv"][0], S_cv[:, 2 * d:] @ e[u[0]])
    assert np.allclose(h["hv"][1], S_cv[:, :d] @ e[u[1]] + S_cv[:, d:2 * d] @ e[u[2]] + S_cv[:, 2 * d:] @ e[u[3]])


def test_window_at_least_length_equals_full_attention():
    cfg, w, cond = _setup()
    u = _tokens(cfg, 20)
    full = O.forward_full(cfg, w, cond, u)
    wide = O.forward_full(cfg.with_(window=(20, 7, 3)), w, cond, u)
    assert np.abs(full - wide).max() < 1e-12
    narrow = O.forward_full(cfg.with_(window=(19, 0, 0)), w, cond, u)
    assert np.abs(full[:19] - narrow[:19]).max() < 1e-12 and np.abs(full[19] - narrow[19]).max() > 1e-9


def test_mqa_with_replicated_kv_weights_equals_mha():
    cfg1, w1, cond = _setup(n_kv_heads=1)
    cfg2 = cfg1.with_(n_kv_heads=cfg1.n_heads)
    H, dh = cfg1.n_heads, cfg1.head_dim
    w2 = S.make_weights(cfg2)
    for k in ("E", "S_cv", "S_vf", "U_fv", "U_vc", "g_out", "W_out"):
        w2[k] = w1[k]
    for s in range(5):
        for l, lw in enumerate(w1["stacks"][s]):
            Wq, Wk, Wv = np.split(lw["Wqkv"], [H * dh, (H + 1) * dh])
            w2["stacks"][s][l] = {**lw, "Wqkv": np.concatenate([Wq] + [Wk] * H + [Wv] * H)}
    u = _tokens(cfg1, 13)
    assert np.abs(O.forward_full(cfg1, w1, cond, u) - O.forward_full(cfg2, w2, cond, u)).max() < 1e-12


def test_prefix_is_visible_and_unrotated():
    cfg, w, cond = _setup()
    u = _tokens(cfg, 10)
    a = O.forward_full(cfg, w, cond, u)
    assert np.abs(a - O.forward_full(cfg, w, cond * 1.5 + 0.3, u)).max() > 1e-6
    # permuting the prefix entries cannot change anything if they carry no position
    b = O.forward_full(cfg, w, cond[::-1].copy(), u)
    assert np.abs(a - b).max() < 1e-12


# ------------------------------------------------------------- cached forward == definition
@pytest.mark.parametrize("window", [(0, 0, 0), (7, 3, 2)])
def test_cached_rows_equal_dense_forward_and_single_steps(window):
    cfg, w, cond = _setup(layers=(1, 2, 2, 1, 2), window=window)
    u = _tokens(cfg, 40)
    full = O.forward_full(cfg, w, cond, u)
    seq = O.OracleSeq(cfg, w)
    got = [seq.prefill(cond, u[1:6])]
    pos = 6
    for n in (4, 1, 10, 1, 1, 13, 4):                 # multi-row passes of assorted sizes
        got.append(seq.forward_rows(u[pos:pos + n]))
        seq.L += n
        pos += n
    got = np.concatenate(got)
    assert pos == 40 and np.abs(got - full).max() < 1e-9
    one = O.OracleSeq(cfg, w)
    rows = [one.prefill(cond, [])]
    for i in range(1, 40):                            # k fed tokens == k sequential single-token steps
        rows.append(one.forward_rows(u[i:i + 1]))
        one.L += 1
    assert np.abs(np.concatenate(rows) - full).max() < 1e-9


@pytest.mark.parametrize("chunk", [1, 7, 16])
def test_chunked_prefill_equals_the_dense_forward(chunk):
    cfg, w, cond = _setup(layers=(1, 2, 2, 1, 2), window=(11, 5, 2))
    u = _tokens(cfg, 37)
    full = O.forward_full(cfg, w, cond, u)
    seq = O.OracleSeq(cfg, w)
    last = seq.prefill(cond, u[1:], chunk=chunk)
    assert seq.L == 37 and np.abs(last - full[-last.shape[0]:]).max() < 1e-9
    nxt = seq.forward_rows([u[5]])                    # the state after a chunked prefill decodes on correctly
    assert np.abs(nxt[0] - O.forward_full(cfg, w, cond, u + [u[5]])[-1]).max() < 1e-9
    assert seq.main == O.masked_top2(cfg, full[-1], 36)[0]


def test_rejected_rows_leave_no_trace():
    cfg, w, cond = _setup(draft_len=9)
    u = _tokens(cfg, 30)
    full = O.forward_full(cfg, w, cond, u)
    seq = O.OracleSeq(cfg, w)
    seq.prefill(cond, u[1:8])
    junk = [(t + 3) % cfg.n_bins for t in u[8:18]]
    seq.forward_rows([u[8]] + junk[1:])               # only the first row will be kept
    seq.L += 1
    got = seq.forward_rows(u[9:30])
    assert np.abs(got - full[9:30]).max() < 1e-9


def test_float32_mode_agrees_with_float64():
    cfg, w, cond = _setup()
    u = _tokens(cfg, 20)
    a = O.forward_full(cfg, w, cond, u, dtype=np.float64)
    b = O.forward_full(cfg, w, cond.astype(np.float32), u, dtype=np.float32)
    assert b.dtype == np.float32 and np.abs(a - b).max() < 2e-4
