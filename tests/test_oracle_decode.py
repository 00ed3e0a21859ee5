"""Pins of the oracle's decode loop: speculative == plain greedy == brute force, bookkeeping."""
import os

import numpy as np
import pytest

import fm_synth as S
from oracle import hourglass as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _setup(**kw):
    cfg = S.toy_config(**kw)
    return cfg, S.make_weights(cfg), S.make_condition(cfg)


def _prompt(cfg, faces, seed=3):
    return [int(t) for t in np.random.default_rng(seed).integers(0, cfg.n_bins, 9 * faces)]


def _teacher(truth, upto=None, corrupt_rng=None):
    """Draft editor: fill the drafts with the true continuation `truth` (mesh-token list
    indexed by absolute position).  `upto` keeps only that many correct drafts; the next one
    is made wrong on purpose."""
    def fn(seq, cand):
        n, D = seq.L - 1, seq.cfg.draft_len
        keep = D if upto is None else (upto if corrupt_rng is None else int(corrupt_rng.integers(0, D + 1)))
        for j in range(1, D + 1):
            t = truth[n + j] if n + j < len(truth) else 0
            cand[j] = t if j <= keep else (t + 1) % seq.cfg.n_bins
        return cand
    return fn


@pytest.mark.parametrize("D", [1, 2, 3, 9, 12])
def test_speculative_equals_plain_equals_bruteforce(D):
    cfg, w, cond = _setup(draft_len=D, layers=(1, 1, 2, 1, 1))
    prompt = _prompt(cfg, 1)
    faces = 3
    brute = O.greedy_full(cfg, w, cond, prompt, 9 * faces)

    def run(draft_fn=None, plain=False):
        seq = O.OracleSeq(cfg, w)
        seq.prefill(cond, prompt, max_faces=faces)
        out, acc = seq.generate(faces, draft_fn=draft_fn, force_plain=plain)
        assert sum(acc) == len(out) and seq.done
        assert seq.kv_len() == (seq.L, -(-seq.L // 3), -(-seq.L // 9))
        return out, acc

    plain, acc = run(plain=True)
    assert plain == brute and set(acc) == {1}
    heads, _ = run()                                                   # whatever the heads draft
    assert heads == brute
    truth = prompt + brute
    wrong, acc = run(lambda s, c: [c[0]] + [(truth[s.L - 1 + j] + 1) % cfg.n_bins if s.L - 1 + j < len(truth)
                                            else 0 for j in range(1, D + 1)])
    assert wrong == brute and set(acc) == {1}                          # all drafts wrong: a = 1 every step
    teach, acc = run(_teacher(truth))
    assert teach == brute
    assert all(a == D + 1 for a in acc[:-1]) and 1 <= acc[-1] <= D + 1  # all drafts right: a = D+1
    assert len(acc) == -(-len(brute) // (D + 1))
    rnd, acc = run(_teacher(truth, upto=0, corrupt_rng=np.random.default_rng(D)))
    assert rnd == brute and (len(set(acc)) > 1 or D == 1)


def test_accept_length_is_exactly_the_number_of_leading_matches():
    cfg, w, cond = _setup(draft_len=9)
    prompt = _prompt(cfg, 1)
    truth = prompt + O.greedy_full(cfg, w, cond, prompt, 36)
    for keep in range(0, 10):
        seq = O.OracleSeq(cfg, w)
        seq.prefill(cond, prompt, max_faces=4)
        cand, _, _ = seq.draft()
        cand = _teacher(truth, upto=keep)(seq, list(cand))
        if keep < 8:                                  # a later draft that is right again must not count
            cand[keep + 2] = truth[seq.L - 1 + keep + 2]
        o, _, _ = seq.verify(cand)
        assert o[:10] == truth[seq.L - 1 + 1: seq.L - 1 + 11] or keep < 9
        L0 = seq.L
        a, em, kv = seq.accept()
        assert a == keep + 1 and em[:a] == cand[:a] and em[a:] == [-1] * (10 - a)
        assert kv == (L0 + a, -(-(L0 + a) // 3), -(-(L0 + a) // 9))
        assert seq.main == truth[seq.L - 1]


def test_verify_is_idempotent_and_does_not_move_lengths():
    cfg, w, cond = _setup(draft_len=3)
    seq = O.OracleSeq(cfg, w)
    seq.prefill(cond, _prompt(cfg, 1), max_faces=2)
    cand, _, _ = seq.draft()
    o1, l1, _ = seq.verify(cand)
    kv = seq.kv_len()
    o2, l2, _ = seq.verify(cand)
    assert o1 == o2 and np.array_equal(l1, l2) and seq.kv_len() == kv


def test_budget_clip_and_inactive_after_done():
    cfg, w, cond = _setup(draft_len=12)
    prompt = _prompt(cfg, 1)
    truth = prompt + O.greedy_full(cfg, w, cond, prompt, 18)
    seq = O.OracleSeq(cfg, w)
    seq.prefill(cond, prompt, max_faces=2)
    out, acc = seq.generate(2, draft_fn=_teacher(truth))
    assert out == truth[9:] and acc == [13, 5]            # second pass clipped to the 5 tokens left
    assert seq.accept()[0] == 0 and seq.draft()[0] == [cfg.pad] * 13
    assert seq.verify([cfg.pad] * 13)[0] == [-1] * 13


def test_eos_only_where_a_face_starts_and_it_ends_the_sequence():
    hits = 0
    for seed in range(6):
        cfg, w, cond = _setup(draft_len=3, allow_eos=1, seed=20 + seed)
        w["W_out"][cfg.eos] = 3.0 * w["W_out"][:cfg.n_bins].mean(axis=0) + w["W_out"][cfg.eos]
        seq = O.OracleSeq(cfg, w)
        seq.prefill(cond, [], max_faces=8)
        out, _ = seq.generate(8)
        assert all(0 <= t < cfg.n_bins or t == cfg.eos for t in out)
        if cfg.eos in out:
            hits += 1
            assert out.index(cfg.eos) == len(out) - 1 and (len(out) - 1) % 9 == 0
        else:
            assert len(out) == 72
        assert out == O.greedy_full(cfg, w, cond, [], 72)
    assert hits >= 1


def test_eos_inside_accepted_drafts_clips_the_accept():
    cfg, w, cond = _setup(draft_len=9, allow_eos=1)
    seq = O.OracleSeq(cfg, w)
    seq.prefill(cond, _prompt(cfg, 1), max_faces=4)
    cand, _, _ = seq.draft()
    seq.verify(cand)
    forced = list(seq.o)
    cand2 = [cand[0]] + forced[:9]
    cand2[3] = cfg.eos
    seq.verify(cand2)
    a, em, _ = seq.accept(force_len=10)
    assert a == 4 and em[3] == cfg.eos and seq.done


# ------------------------------------------------------------------ draft source assignment
def test_draft_sources_match_the_papers_worked_example():
    """Supp. "Optimizations": the row rule (A) names and the two worked steps, at the phases of
    the face the paper's indices put them at (a face row, then 6 and 7 tokens into the face)."""
    rows = [tuple(int(x) for x in ln.split()) for ln in open(os.path.join(GOLDEN, "draft_coverage_9_9.txt"))
            if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 23 and {r[0] for r in rows} == {0, 6, 7}
    for n, j, level in rows:
        for faces_before in (0, 1, 5):                # the assignment depends on the phase only
            assert O.draft_source(n + 9 * faces_before, j, 9)[0] == level


def test_draft_sources_at_every_phase_of_the_face():
    """All nine phases, offsets 1..9, against the table worked out by hand from the rules."""
    table = {}
    for ln in open(os.path.join(GOLDEN, "draft_sources_all_phases_D9.txt")):
        if ln.strip() and not ln.startswith("#"):
            f = ln.split()
            table[int(f[0])] = f[1:]
    assert sorted(table) == list(range(9)) and all(len(v) == 9 for v in table.values())
    name = {0: "c", 1: "v", 2: "f"}
    for n in range(0, 45):
        for j in range(1, 10):
            level, head, _ = O.draft_source(n, j, 9)
            assert name[level] + (str(head) if level else "") == table[n % 9][j - 1], (n, j)


@pytest.mark.parametrize("D", [3, 9, 12, 24, 27])
def test_every_offset_has_one_valid_source(D):
    cfg = S.toy_config(draft_len=D)
    for n in range(0, 40):
        for j in range(1, D + 1):
            level, head, slot = O.draft_source(n, j, D)
            p = n + j
            if level == 0:
                assert j in (1, 2) and head == j
            elif level == 1:                          # the vertex `head` after the one that holds t_n
                assert 1 <= head <= 2 and 3 * (n // 3 + head) + slot == p
                assert (n // 3) % 3 != 0 or p // 9 != n // 9      # never where rule (A) keeps the face level
            else:                                     # face head e drafts face f* + e - 1
                assert 1 <= head <= cfg.n_face_heads and 9 * (n // 9 + head - 1) + slot == p
                assert head > 1 or (n // 3) % 3 == 0


def test_draft_features_follow_the_head_formula_in_special_cases():
    """With a head's matrix A zeroed the SP feature is the split-node hidden itself, so the
    draft logits must equal the output layer applied to (upsampled) stashed hiddens."""
    cfg, w, cond = _setup(draft_len=9)
    for hs in (w["heads_c"], w["heads_v"], w["heads_f"]):
        for h in hs:
            h["A"][:] = 0.0
    W, g = w["W_out"].astype(np.float64), w["g_out"].astype(np.float64)
    out = lambda f: W @ (f / np.sqrt(np.mean(f * f) + cfg.norm_eps) * g)
    d = cfg.d_model
    U_vc, U_fv = w["U_vc"].astype(np.float64), w["U_fv"].astype(np.float64)
    seq = O.OracleSeq(cfg, w)
    seq.prefill(cond, _prompt(cfg, 1), max_faces=4)       # n = 9: a face row
    _, dl, _ = seq.draft()
    n = seq.L - 1
    assert n == 9
    assert np.allclose(dl[0], out(seq.zc[n])) and np.allclose(dl[1], out(seq.zc[n]))
    ftri = U_fv @ seq.zf[n // 9]                           # every face head sees the same z_f
    for j in range(3, 9):                                  # rule (A): the face level, slots 3..8 of this face
        sub = U_vc @ ftri[(j // 3) * d:(j // 3 + 1) * d]
        assert np.allclose(dl[j - 1], out(sub[(j % 3) * d:(j % 3 + 1) * d]))
    assert np.allclose(dl[8], out((U_vc @ ftri[:d])[:d]))  # offset 9: next face, slot 0
    # three tokens on (force the accept): a point-level row inside the face
    cand, _, _ = seq.draft()
    seq.verify(cand)
    seq.accept(force_len=3)
    _, dl, _ = seq.draft()
    n = seq.L - 1
    assert n == 12
    tri = U_vc @ seq.zv[n // 3]
    for j in range(3, 9):                                  # both vertex heads see the same z_v
        assert np.allclose(dl[j - 1], out(tri[(j % 3) * d:(j % 3 + 1) * d]))
    ftri = U_fv @ seq.zf[n // 9]
    assert np.allclose(dl[8], out((U_vc @ ftri[d:2 * d])[:d]))     # offset 9 -> t_21: next face, slot 3


def test_head_residual_and_linear_term():
    cfg, w, cond = _setup(draft_len=3)
    seq = O.OracleSeq(cfg, w)
    seq.prefill(cond, _prompt(cfg, 1), max_faces=4)
    _, dl, _ = seq.draft()
    n = seq.L - 1
    z = seq.zc[n]
    hw = w["heads_c"][0]
    y = z + hw["A"].astype(np.float64) @ (z * hw["g"] / np.sqrt(np.mean(z * z) + cfg.norm_eps))
    want = w["W_out"].astype(np.float64) @ (y * w["g_out"] / np.sqrt(np.mean(y * y) + cfg.norm_eps))
    assert np.allclose(dl[0], want)


# ------------------------------------------------------------------------ synthetic inputs
def test_inputs_are_well_formed_and_deterministic():
    for name in ("tiny", "small"):
        cfg = S.get_config(name)
        p = S.make_prompt(cfg)
        assert len(p) == 9 * cfg.prompt_faces[0] and np.array_equal(p, S.make_prompt(cfg))
        assert ((0 <= p) & (p < cfg.n_bins)).all()
        f = p.reshape(-1, 3, 3)
        for face in f:                                   # vertices ascending by (z,y,x) inside a face
            assert sorted(map(tuple, face)) == list(map(tuple, face))
        assert sorted(map(tuple, p.reshape(-1, 9))) == list(map(tuple, p.reshape(-1, 9)))
        c = S.make_condition(cfg)
        assert c.shape == (cfg.n_prefix, cfg.d_model) and c.dtype == np.float32
    assert S.icosphere_faces(1).shape == (80, 3, 3) and S.icosphere_faces(2).shape == (320, 3, 3)
    w = S.make_weights(S.toy_config())
    assert np.array_equal(S.round_to_bf16(w["W_out"]), w["W_out"])
    a = S.accept_schedule(0, 16, 4000, 9, 6.7)
    assert a.min() >= 1 and a.max() == 10 and abs(a.mean() - 7.7) < 0.1
