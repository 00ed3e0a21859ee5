"""Pins of the oracle's draft modules beyond the reduced heads: the full SP-Block and HF-Blocks
(Sec. 3.1, Eq. 1-5), the averaged merge of the levels, the coordinate-only variant (supplement,
ablation on multi-level decoding) and the label head (Sec. 3.2)."""
import numpy as np
import pytest

import fm_synth as S
from oracle import hourglass as O


def _prompt(cfg, faces, seed=3):
    return [int(t) for t in np.random.default_rng(seed).integers(0, cfg.n_bins, 9 * faces)]


def _seq(cfg, w, faces=2, extra=0, **kw):
    seq = O.OracleSeq(cfg, w)
    seq.prefill(S.make_condition(cfg), _prompt(cfg, faces), max_faces=6)
    for _ in range(extra):                               # move on token by token
        cand, _, _ = seq.draft()
        seq.verify(cand)
        seq.accept(force_len=1)
    return seq


def test_full_modules_with_zero_output_matrices_are_the_reduced_heads():
    """Eq. 1 with the attention's output projection zeroed is Linear + residual, and Eq. 5 with
    FFN = 0 is the identity: the full draft path then gives the reduced heads' logits."""
    full = S.toy_config(draft_len=12, draft_heads="full", layers=(1, 2, 2, 1, 2))
    w = S.make_weights(full)
    for hs in (w["heads_c"], w["heads_v"], w["heads_f"]):
        for h in hs:
            h["Wo"][:] = 0.0
    for name in ("hf_vc", "hf_fv", "hf_fc"):
        for h in w[name]:
            h["W2"][:] = 0.0
    red = full.with_(draft_heads="reduced")
    for extra in (0, 1, 4, 7):
        a, b = _seq(full, w, extra=extra), _seq(red, w, extra=extra)
        ca, la, _ = a.draft()
        cb, lb, _ = b.draft()
        assert ca == cb and np.abs(la - lb).max() < 1e-12
    # and the extra weights matter: with them back the logits differ
    w2 = S.make_weights(full)
    assert np.abs(_seq(full, w2).draft()[1] - _seq(red, w2).draft()[1]).max() > 1e-3


def test_sp_block_against_a_dense_recomputation_without_caches():
    """Coordinate head 1 of a model with one coord-up layer, recomputed from forward_full's
    hiddens: the split-node hiddens are c1_i = hc_i + (U_vc hv'_{i//3})[i%3]; the last layer's keys
    and values are its own projections of rms(c1); the head attends over the prefix and all
    positions <= n with its own query."""
    cfg = S.toy_config(draft_len=3, draft_heads="full", layers=(1, 1, 1, 1, 1))
    w = S.make_weights(cfg)
    cond = S.make_condition(cfg)
    prompt = _prompt(cfg, 2)
    seq = O.OracleSeq(cfg, w)
    seq.prefill(cond, prompt, max_faces=4)
    _, dl, _ = seq.draft()
    n, d, H, dh = seq.L - 1, cfg.d_model, cfg.n_heads, cfg.head_dim
    u = [cfg.bos] + prompt
    _, hid = O.forward_full(cfg, w, cond, u, return_hidden=True)
    f64 = lambda a: np.asarray(a, dtype=np.float64)
    up = hid["hv2"] @ f64(w["U_vc"]).T
    c1 = np.stack([hid["hc"][i] + up[i // 3, (i % 3) * d:(i % 3 + 1) * d] for i in range(len(u))])
    lw = w["stacks"][4][0]
    rms = lambda x, g: x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + cfg.norm_eps) * f64(g)
    kv = rms(c1, lw["g1"]) @ f64(lw["Wqkv"])[H * dh:].T
    k = O.rope(kv[:, :H * dh].reshape(-1, H, dh), np.arange(len(u)), cfg.rope_theta)
    v = kv[:, H * dh:].reshape(-1, H, dh)
    pkv = rms(f64(cond), lw["g1"]) @ f64(lw["Wqkv"])[H * dh:].T
    keys = np.concatenate([pkv[:, :H * dh].reshape(-1, H, dh), k])
    vals = np.concatenate([pkv[:, H * dh:].reshape(-1, H, dh), v])
    hw = w["heads_c"][0]
    z = c1[n]
    q = O.rope((f64(hw["Wq"]) @ rms(z, hw["ga"])).reshape(1, H, dh), [n], cfg.rope_theta)[0]
    o = np.zeros((H, dh))
    for h in range(H):
        sc = keys[:, h] @ q[h] / np.sqrt(dh)
        p = np.exp(sc - sc.max())
        o[h] = (p / p.sum()) @ vals[:, h]
    y = z + f64(hw["Wo"]) @ o.reshape(-1)
    feat = z + f64(hw["A"]) @ rms(y, hw["g"])
    want = f64(w["W_out"]) @ rms(feat, w["g_out"])
    assert np.abs(dl[0] - want).max() < 1e-9


@pytest.mark.parametrize("window", [(0, 0, 0), (7, 3, 2)])
def test_zero_queries_average_exactly_the_visible_cache_entries(window):
    """With W_q = 0 every score is 0 and the attention output is the plain mean of the visible
    values: the prefix entries and the accepted positions that the last accepted row sees, at the
    level of the module (SP: coordinate / vertex / face; HF: coordinate or vertex) -- nothing beyond
    the last accepted position, nothing outside the window."""
    cfg = S.toy_config(draft_len=9, draft_heads="full", layers=(1, 2, 2, 1, 2), window=window)
    w = S.make_weights(cfg)
    for hs in (w["heads_c"], w["heads_v"], w["heads_f"]):
        for h in hs:
            h["Wq"][:] = 0.0
    for name in ("hf_vc", "hf_fv", "hf_fc"):
        for h in w[name]:
            h["Wq"][:] = 0.0
    seq = _seq(cfg, w, faces=2, extra=5)
    cand, _, _ = seq.draft()
    seq.verify([cand[0]] + [3] * 9)                      # tentative rows beyond L: must stay invisible
    n = seq.L - 1
    pos = (n, n // 3, n // 9)

    def mean_visible(s, level):
        l = len(w["stacks"][s]) - 1
        W = window[level]
        lo = max(0, pos[level] - W + 1) if W > 0 else 0
        vals = np.concatenate([seq.VP[s][l], seq.V[s][l][lo:pos[level] + 1]])
        return vals.mean(axis=0).reshape(-1)

    f64 = lambda a: np.asarray(a, dtype=np.float64)
    rms = lambda x, g: x / np.sqrt(np.mean(x * x) + cfg.norm_eps) * f64(g)
    feats, points = seq.draft_features()
    z = (seq.zc[n], seq.zv[n // 3], seq.zf[n // 9])
    for level, s, hs, key in ((0, 4, w["heads_c"], (0, 1, 0)), (1, 3, w["heads_v"], (1, 1, 0))):
        hw = hs[0]
        y = z[level] + f64(hw["Wo"]) @ mean_visible(s, level)
        sp = z[level] + f64(hw["A"]) @ rms(y, hw["g"])
        got = feats[key] if level == 0 else points[key]
        assert np.abs(got - sp).max() < 1e-10
    # face head 1: SP at the face level, then HF at the vertex level (vertex rv = 0 of its face)
    hw = w["heads_f"][0]
    yf = z[2] + f64(hw["A"]) @ rms(z[2] + f64(hw["Wo"]) @ mean_visible(2, 2), hw["g"])
    x = (f64(w["U_fv"]) @ yf)[:cfg.d_model]
    hb = w["hf_fv"][0]
    want = x + f64(hb["W2"]) @ O.gelu(f64(hb["W1"]) @ mean_visible(3, 1))
    assert np.abs(points[(2, 1, 0)] - want).max() < 1e-10
    # point pipeline, offset 3 (first coordinate of vertex v*+1): HF at the coordinate level
    x = (f64(w["U_vc"]) @ points[(1, 1, 0)])[:cfg.d_model]
    hb = w["hf_vc"][0]
    want = x + f64(hb["W2"]) @ O.gelu(f64(hb["W1"]) @ mean_visible(4, 0))
    assert np.abs(feats[(1, 1, 0)] - want).max() < 1e-10


def test_hf_block_is_residual_and_linear_in_its_second_ffn_matrix():
    cfg = S.toy_config(draft_len=9, draft_heads="full")
    w = S.make_weights(cfg)
    seq = _seq(cfg, w, extra=3)
    f0, _ = seq.draft_features()
    for h in w["hf_vc"]:
        h["W2"] *= 2.0
    seq2 = _seq(cfg, w, extra=3)
    f2, _ = seq2.draft_features()
    _, pts = seq.draft_features()
    x = (np.asarray(w["U_vc"], np.float64) @ pts[(1, 1, 0)])[:cfg.d_model]
    assert np.abs((f2[(1, 1, 0)] - x) - 2.0 * (f0[(1, 1, 0)] - x)).max() < 1e-9
    assert np.abs(f0[(1, 1, 0)] - x).max() > 1e-6


def test_averaged_levels_are_a_distribution_and_reduce_to_the_single_source_where_one_level_predicts():
    cfg = S.toy_config(draft_len=9, avg_levels=1)
    w = S.make_weights(cfg)
    single = cfg.with_(avg_levels=0)
    for extra in (0, 3, 6):
        a, b = _seq(cfg, w, extra=extra), _seq(single, w, extra=extra)
        n = a.L - 1
        ca, la, _ = a.draft()
        cb, lb, _ = b.draft()
        for j in range(1, 10):
            srcs = a._all_sources(n, j)
            assert 1 <= len(srcs) <= 3 and len({s[0] for s in srcs}) == len(srcs)
            assert abs(np.exp(la[j - 1]).sum() - 1.0) < 1e-9
            if len(srcs) == 1:                           # log-softmax of the only source: same argmax, shifted logits
                assert srcs[0] == O.draft_source(n, j, 9)
                shift = la[j - 1] - lb[j - 1]
                assert np.abs(shift - shift[0]).max() < 1e-9 and ca[j] == cb[j]
            # the source the single-source rule picks is always among the averaged ones
            assert O.draft_source(n, j, 9) in srcs
        # at a face row offset 3 is predicted by the point level and by the face level
        if n % 9 == 0:
            assert [s[0] for s in a._all_sources(n, 3)] == [1, 2]


def test_coordinate_only_variant_uses_one_coordinate_head_per_offset():
    cfg = S.toy_config(draft_len=18, draft_levels="coord")
    w = S.make_weights(cfg)
    assert len(w["heads_c"]) == 18 and not w["heads_v"] and not w["heads_f"]
    seq = _seq(cfg, w, extra=2)
    _, dl, _ = seq.draft()
    n = seq.L - 1
    z = seq.zc[n]
    f64 = lambda a: np.asarray(a, dtype=np.float64)
    rms = lambda x, g: x / np.sqrt(np.mean(x * x) + cfg.norm_eps) * f64(g)
    for j in (1, 7, 18):
        assert O.draft_source(n, j, 18, "coord") == (0, j, 0)
        hw = w["heads_c"][j - 1]
        feat = z + f64(hw["A"]) @ rms(z, hw["g"])
        assert np.abs(dl[j - 1] - f64(w["W_out"]) @ rms(feat, w["g_out"])).max() < 1e-10
    # and decoding with it is still exact
    prompt = _prompt(cfg, 1)
    cond = S.make_condition(cfg)
    brute = O.greedy_full(cfg, w, cond, prompt, 18)
    s2 = O.OracleSeq(cfg, w)
    s2.prefill(cond, prompt, max_faces=2)
    out, _ = s2.generate(2)
    assert out == brute


def test_label_head_slots_and_antisymmetry():
    """Labels exist exactly at the slots where a vertex made of drafts only starts; with the three
    rows of the label matrix set to u, 2u, 3u the label is 2 where u . rms(feature) > 0 and 0
    elsewhere, so flipping the sign of u swaps the two and label 1 never appears."""
    from oracle.correct import draft_points
    cfg = S.toy_config(draft_len=12)
    w = S.make_weights(cfg)
    u = np.asarray(w["label"]["W"][0]).copy()
    w["label"]["W"][:] = np.stack([u, 2 * u, 3 * u])
    wm = {k: v for k, v in w.items()}
    wm["label"] = {"g": w["label"]["g"], "W": -w["label"]["W"]}
    seen = set()
    for extra in range(9):
        a, b = _seq(cfg, w, extra=extra), _seq(cfg, wm, extra=extra)
        a.draft(); b.draft()
        la, _ = a.draft_labels()
        lb, _ = b.draft_labels()
        starts = draft_points(a.L, 13)
        assert [s for s in range(13) if la[s] >= 0] == starts
        for s in starts:
            assert la[s] in (0, 2) and lb[s] == 2 - la[s]
            seen.add(la[s])
    assert seen == {0, 2}
