"""GPU parity: the CUDA library against the oracle, element by element, through the C ABI."""
import numpy as np
import pytest

import fm_synth as S

pytestmark = pytest.mark.gpu

# The toy model draws its matrices with std 0.1 (five times the workloads' 0.02) so that attention
# is sharp and an indexing mistake moves the hidden states by O(1); only the output matrix is drawn
# at the workloads' 0.02, which puts the logits on the workloads' scale (sigma = 0.02 sqrt(d), about
# 0.23 at d = 128), so the stated bound applies as it stands: logits within 2e-2, ids compared where
# the oracle's top-2 margin exceeds 0.1.  (A mistake that moves a normalised hidden state by 10 %
# still moves a logit by about 0.02 sqrt(d) * 0.1 * 3 sigma, well above the bound.)
TOY = dict(d_model=128, head_dim=64, d_ff=256, weight_std=0.1, out_std=0.02)
TOY_TOL = 2e-2
TOY_MARGIN = 0.1


def _dev(cfg, w, **kw):
    from paper_2511_15618_b200 import FlashMesh
    return FlashMesh(cfg, w, **kw)


def _setup(cfg, batch=None):
    w = S.make_weights(cfg)
    B = cfg.batch if batch is None else batch
    conds = [S.make_condition(cfg, b) for b in range(B)]
    prompts = [[int(t) for t in S.make_prompt(cfg, b)] for b in range(B)]
    return w, conds, prompts


def _oracle_greedy(cfg, w, cond, prompt, faces):
    from oracle.hourglass import OracleSeq
    s = OracleSeq(cfg, w)
    s.prefill(cond, prompt, max_faces=faces)
    out, _ = s.generate(faces, force_plain=True)
    return list(prompt) + out


@pytest.mark.parametrize("D", [0, 3, 9, 12, 18, 24, 27])
def test_toy_lockstep_all_draft_lengths(D):
    from oracle.lockstep import run_lockstep
    cfg = S.toy_config(**TOY, draft_len=D, layers=(1, 2, 2, 1, 2), max_batch=2, prompt_faces=(1, 1), gen_faces=6)
    cfg = cfg.with_(max_tokens=1 + 9 * 8 + D + 2)
    w, conds, prompts = _setup(cfg, batch=2)
    prompts[1] = prompts[1] + prompts[0]                    # ragged: 1 and 2 faces
    dev = _dev(cfg, w)
    rep = run_lockstep(cfg, w, conds, prompts, dev, [6, 5], 200, tol=TOY_TOL, margin=TOY_MARGIN)
    assert rep["done"] and rep["emitted"] == 9 * 11
    assert dev.device_status() == 0
    assert D < 5 or rep["labels"] > 0                 # the label head's labels were compared as well
    print(D, {k: rep[k] for k in ("steps", "max_logit_err", "max_draft_err", "overrides", "low_margin_rows", "rows", "labels", "label_flips")})


@pytest.mark.parametrize("D", [9, 18])
def test_toy_coordinate_only_drafting_lockstep(D):
    """The supplement's ablation variant: D coordinate heads, no point- or face-level modules."""
    from oracle.lockstep import run_lockstep
    cfg = S.toy_config(**TOY, draft_len=D, draft_levels="coord", layers=(1, 2, 2, 1, 2), max_batch=2, prompt_faces=(1, 1), gen_faces=6)
    cfg = cfg.with_(max_tokens=1 + 9 * 8 + D + 2)
    w, conds, prompts = _setup(cfg, batch=2)
    dev = _dev(cfg, w)
    rep = run_lockstep(cfg, w, conds, prompts, dev, [6, 5], 200, tol=TOY_TOL, margin=TOY_MARGIN)
    assert rep["done"] and rep["emitted"] == 9 * 11 and dev.device_status() == 0
    print(D, {k: rep[k] for k in ("steps", "max_logit_err", "max_draft_err", "overrides")})


@pytest.mark.parametrize("D,avg,window,kv", [(9, 0, (0, 0, 0), 2), (12, 0, (11, 5, 2), 2), (9, 1, (0, 0, 0), 2), (27, 0, (0, 0, 0), 1), (3, 1, (0, 0, 0), 2)])
def test_toy_full_sp_and_hf_blocks_lockstep(D, avg, window, kv):
    """The paper's draft path (Sec. 3.1 Eq. 1-5): SP-Blocks with attention over the backbone's cache,
    an HF-Block after every upsample; single-source and averaged merge; windows; shared KV head."""
    from oracle.lockstep import run_lockstep
    cfg = S.toy_config(**TOY, draft_len=D, draft_heads="full", avg_levels=avg, window=window, n_kv_heads=kv, hf_ff=192,
                       layers=(1, 2, 2, 1, 2), max_batch=2, prompt_faces=(1, 1), gen_faces=6)
    cfg = cfg.with_(max_tokens=1 + 9 * 8 + D + 2)
    w, conds, prompts = _setup(cfg, batch=2)
    prompts[1] = prompts[1] + prompts[0]
    dev = _dev(cfg, w)
    rep = run_lockstep(cfg, w, conds, prompts, dev, [6, 5], 200, tol=TOY_TOL, margin=TOY_MARGIN)
    assert rep["done"] and rep["emitted"] == 9 * 11 and dev.device_status() == 0
    print(D, avg, {k: rep[k] for k in ("steps", "max_logit_err", "max_draft_err", "overrides", "labels", "label_flips")})


def test_toy_averaged_merge_of_reduced_heads_lockstep():
    from oracle.lockstep import run_lockstep
    cfg = S.toy_config(**TOY, draft_len=12, avg_levels=1, layers=(1, 1, 2, 1, 1), max_batch=2, gen_faces=6, max_tokens=1 + 9 * 8 + 12 + 2)
    w, conds, prompts = _setup(cfg, batch=2)
    dev = _dev(cfg, w)
    rep = run_lockstep(cfg, w, conds, prompts, dev, 6, 200, tol=TOY_TOL, margin=TOY_MARGIN)
    assert rep["done"] and dev.device_status() == 0
    print({k: rep[k] for k in ("steps", "max_logit_err", "max_draft_err", "overrides")})


def test_toy_lockstep_windows_and_mqa_and_eos():
    from oracle.lockstep import run_lockstep
    cfg = S.toy_config(**TOY, draft_len=9, layers=(2, 1, 2, 2, 1), window=(11, 5, 2), n_kv_heads=1, allow_eos=1,
                       max_batch=3, gen_faces=8, max_tokens=1 + 9 * 8 + 9 + 2)
    w, conds, prompts = _setup(cfg, batch=3)
    w["W_out"][cfg.eos] += 3.0 * w["W_out"][:cfg.n_bins].mean(axis=0)
    dev = _dev(cfg, w)
    rep = run_lockstep(cfg, w, conds, prompts, dev, 8, 300, tol=TOY_TOL, margin=TOY_MARGIN)
    assert rep["done"] and dev.device_status() == 0
    print({k: rep[k] for k in ("steps", "emitted", "max_logit_err", "max_draft_err", "overrides")})


@pytest.mark.parametrize("prompt_faces", [100, 150])
def test_toy_head_dim_128_long_cache_many_groups(prompt_faces):
    """Head dimension 128 with a cache of 15 to 22 chunks: 100 faces give the largest number of
    groups the last CTA can merge from shared memory (15, one chunk each), 150 faces give groups
    of two chunks."""
    from oracle.lockstep import run_lockstep
    faces = 3
    cfg = S.toy_config(d_model=128, n_heads=1, n_kv_heads=1, head_dim=128, d_ff=256, weight_std=0.1, out_std=0.02, draft_len=3,
                       layers=(1, 1, 1, 1, 1), prompt_faces=(prompt_faces, prompt_faces), prompt_subdiv=2, gen_faces=faces,
                       max_tokens=1 + 9 * (prompt_faces + faces) + 3 + 2)
    w, conds, prompts = _setup(cfg, batch=1)
    assert len(prompts[0]) == 9 * prompt_faces
    dev = _dev(cfg, w)
    rep = run_lockstep(cfg, w, conds, prompts, dev, faces, 60, tol=TOY_TOL, margin=TOY_MARGIN)
    assert rep["done"] and rep["emitted"] == 9 * faces
    assert dev.device_status() == 0                  # in particular: the group-count guard did not fire
    print({k: rep[k] for k in ("steps", "max_logit_err", "max_draft_err", "overrides")})


def test_toy_teacher_drafts_vary_accept_lengths():
    from oracle.lockstep import run_lockstep
    cfg = S.toy_config(**TOY, draft_len=9, layers=(1, 1, 2, 1, 1), max_batch=2, gen_faces=8, max_tokens=1 + 9 * 8 + 9 + 2)
    w, conds, prompts = _setup(cfg, batch=2)
    truth = [_oracle_greedy(cfg, w, conds[b], prompts[b], 8) for b in range(2)]
    dev = _dev(cfg, w)
    rep = run_lockstep(cfg, w, conds, prompts, dev, 8, 300, truth=truth, keep_rng=np.random.default_rng(5), tol=TOY_TOL, margin=TOY_MARGIN)
    assert rep["done"] and sum(1 for a in rep["accept_hist"][2:] if a > 0) >= 4


def test_tiny_full_length_lockstep():
    from oracle.lockstep import run_lockstep
    cfg = S.get_config("tiny")
    w, conds, prompts = _setup(cfg)
    dev = _dev(cfg, w)
    rep = run_lockstep(cfg, w, conds, prompts, dev, cfg.gen_faces, 400)
    assert rep["done"] and rep["emitted"] == 288 and rep["max_logit_err"] <= 2e-2
    print(rep)


def test_tiny_and_small_full_draft_modules_lockstep():
    from oracle.lockstep import run_lockstep
    for name, faces in (("tiny", 8), ("small", 6)):
        cfg = S.get_config(name).with_(draft_heads="full")
        w, conds, prompts = _setup(cfg)
        dev = _dev(cfg, w)
        rep = run_lockstep(cfg, w, conds, prompts, dev, faces, 100)
        assert rep["done"] and rep["emitted"] == 9 * faces and rep["max_draft_err"] <= 2e-2 and dev.device_status() == 0
        print(name, {k: rep[k] for k in ("steps", "max_logit_err", "max_draft_err", "overrides", "labels", "label_flips")})


def test_small_lockstep_with_teacher_drafts():
    from oracle.lockstep import run_lockstep
    cfg = S.get_config("small")
    w, conds, prompts = _setup(cfg)
    faces = 24
    truth = [_oracle_greedy(cfg, w, conds[0], prompts[0], faces)]
    dev = _dev(cfg, w)
    rep = run_lockstep(cfg, w, conds, prompts, dev, faces, 400, truth=truth, keep_rng=np.random.default_rng(1))
    assert rep["done"] and rep["emitted"] == 9 * faces
    print(rep)


@pytest.mark.parametrize("variant", [{}, {"draft_heads": "full"}, {"draft_levels": "coord"}, {"avg_levels": 1}])
def test_generate_speculative_equals_plain_on_device(variant):
    """Row-invariant numerics: speculative decoding on the GPU emits exactly what one-token-at-a-
    time decoding on the same kernels emits, whatever the drafts are (and whichever draft modules
    produce them)."""
    cfg = S.get_config("tiny").with_(**variant)
    w, conds, prompts = _setup(cfg)
    dev = _dev(cfg, w)
    dev.prefill(np.stack(conds), prompts)
    plain, plen, st0 = dev.generate(cfg.gen_faces, plain=True)
    dev.prefill(np.stack(conds), prompts)
    spec, slen, st1 = dev.generate(cfg.gen_faces)
    assert int(plen[0]) == 288 and int(slen[0]) == 288
    assert (plain == spec).all()
    assert st0.steps == 288 and st1.emitted == 288
    truth = np.concatenate([np.asarray(prompts[0], np.int32), plain[0].cpu().numpy()])[None]
    dev.prefill(np.stack(conds), prompts)
    teach, tlen, st2 = dev.generate(cfg.gen_faces, truth=truth)
    assert (teach == plain).all() and st2.steps == 288 // 4 and st2.accept_hist[4] == 72


def test_stepwise_calls_replayed_as_graphs_give_the_same_results(monkeypatch):
    """fm_draft / fm_verify with the same pointer arguments every pass are captured and replayed as
    CUDA graphs from the second call on; results must be those of the plain launches, bit for bit."""
    import torch
    cfg = S.get_config("tiny")
    w, conds, prompts = _setup(cfg)

    def run(dev, reuse):
        dev.prefill(np.stack(conds), prompts)
        out = []
        for step in range(10):
            cand, dl, _ = dev.draft(want_logits=True, reuse=reuse)
            o, lg, mg = dev.verify(cand, want_logits=True, reuse=reuse)
            out.append((cand.clone(), dl.clone(), o.clone(), lg.clone(), mg.clone()))
            dev.accept(force_len=np.array([1 + step % (cfg.draft_len + 1)], dtype=np.int32), reuse=reuse)
        return out

    dev_g = _dev(cfg, w)
    l0 = dev_g.launch_count()
    got = run(dev_g, True)
    n_graph = dev_g.launch_count() - l0
    monkeypatch.setenv("FM_NO_CALL_GRAPH", "1")
    dev_p = _dev(cfg, w)
    l0 = dev_p.launch_count()
    want = run(dev_p, False)
    assert dev_p.launch_count() - l0 == n_graph          # a replayed pass counts the launches it holds
    for a, b in zip(got, want):
        for x, y in zip(a, b):
            assert torch.equal(x, y)
    assert dev_g.device_status() == 0


def test_error_codes():
    from paper_2511_15618_b200 import FmError
    cfg = S.toy_config(**TOY)
    w, conds, prompts = _setup(cfg)
    dev = _dev(cfg, w)
    with pytest.raises(FmError) as e:
        dev.batch = 1
        dev.draft()
    assert e.value.code == -2                                     # BAD_STATE before prefill
    with pytest.raises(FmError) as e:
        dev.prefill(np.stack(conds * 3), prompts * 3)
    assert e.value.code == -3                                     # batch > max_batch
    with pytest.raises(FmError) as e:
        dev.prefill(np.stack(conds), [[1, 2, 3]])
    assert e.value.code == -1                                     # prompt not a multiple of 9
    dev.prefill(np.stack(conds), prompts)
    with pytest.raises(FmError) as e:
        dev.accept()
    assert e.value.code == -2                                     # accept without verify
    with pytest.raises(FmError) as e:
        dev.generate(1000)
    assert e.value.code == -3


def test_bounded_wait_gives_up_and_prefill_recovers():
    """The give-up path of the device-side waits: a wait on a barrier that nothing completes runs
    out after its cycle limit, the kernel ends by itself and the status word reads FM_ERR_TIMEOUT;
    a new fm_prefill clears it and the next passes are correct."""
    from oracle.lockstep import run_lockstep
    from paper_2511_15618_b200 import fm_selftest_wait_timeout
    cfg = S.get_config("tiny", gen_faces=2)
    w, conds, prompts = _setup(cfg)
    dev = _dev(cfg, w)
    dev.prefill(np.stack(conds), prompts)
    assert dev.device_status() == 0
    assert fm_selftest_wait_timeout(dev.ctx, 200000) == 0          # about a tenth of a millisecond of polling
    assert dev.device_status() == -5                               # FM_ERR_TIMEOUT
    assert fm_selftest_wait_timeout(dev.ctx, 0) == -1              # limit out of range: nothing is launched
    rep = run_lockstep(cfg, w, conds, prompts, dev, 2, 40)         # starts with fm_prefill
    assert rep["done"] and rep["emitted"] == 18 and dev.device_status() == 0


def test_step_host_equals_the_stepwise_calls():
    """fm_step_host (one call per pass, host buffers) gives what fm_draft / fm_verify / fm_accept
    give, with the host's candidates where it supplies them and the draft modules' elsewhere."""
    import torch
    cfg = S.get_config("tiny")
    w, conds, prompts = _setup(cfg)
    D = cfg.draft_len
    a, b = _dev(cfg, w), _dev(cfg, w)
    a.prefill(np.stack(conds), prompts)
    b.prefill(np.stack(conds), prompts)
    truth = _oracle_greedy(cfg, w, conds[0], prompts[0], 6)
    cand_h = torch.full((1, D + 1), -1, dtype=torch.int32).pin_memory()
    nacc_h = torch.zeros((1,), dtype=torch.int32).pin_memory()
    em_h = torch.zeros((1, D + 1), dtype=torch.int32).pin_memory()
    kv_h = torch.zeros((1, 3), dtype=torch.int32).pin_memory()
    L = 1 + len(prompts[0])
    for step in range(12):
        cand, _, _ = a.draft()
        c = cand.cpu().numpy()
        edit = np.full((1, D + 1), -1, dtype=np.int32)
        if step % 3 != 2:                                 # some passes keep the draft modules' own candidates
            k = step % (D + 1)
            for j in range(1, k + 1):
                edit[0, j] = truth[L - 1 + j]
            c[edit >= 0] = edit[edit >= 0]
        a.verify(c)
        n_a, em_a, kv_a = a.accept()
        cand_h.copy_(torch.as_tensor(edit))
        b.step_host(cand_h if step % 3 != 2 else None, nacc_h, em_h, kv_h)
        assert int(n_a[0]) == int(nacc_h[0]) and em_a.cpu().tolist() == em_h.tolist() and kv_a.cpu().tolist() == kv_h.tolist()
        L += int(nacc_h[0])
    assert a.device_status() == 0 and b.device_status() == 0


@pytest.mark.parametrize("switch", ["FM_NO_FUSE", "FM_NO_PDL", "FM_NO_CALL_GRAPH"])
def test_toy_lockstep_with_a_fallback_switch(switch, monkeypatch):
    """The environment switches select other launch forms of the same arithmetic (shorten gather
    and upsample add as row-wise kernels; launches without programmatic dependent launch; stepwise
    calls never replayed as graphs): each must pass the same lock-step check, with accept lengths
    that vary so that rows cross passes."""
    from oracle.lockstep import run_lockstep
    monkeypatch.setenv(switch, "1")
    cfg = S.toy_config(**TOY, draft_len=9, layers=(1, 1, 2, 1, 1), max_batch=2, gen_faces=8, max_tokens=1 + 9 * 8 + 9 + 2)
    w, conds, prompts = _setup(cfg, batch=2)
    truth = [_oracle_greedy(cfg, w, conds[b], prompts[b], 8) for b in range(2)]
    dev = _dev(cfg, w)
    rep = run_lockstep(cfg, w, conds, prompts, dev, 8, 300, truth=truth, keep_rng=np.random.default_rng(5), tol=TOY_TOL, margin=TOY_MARGIN)
    assert rep["done"] and dev.device_status() == 0


def test_toy_lockstep_width_not_a_multiple_of_128():
    """d = 192 (two heads of 64, d_ff = 320): the last tile of most projections is partly empty and
    the hourglass steps run as row-wise kernels (the fused epilogues want d to be a multiple of 128)."""
    from oracle.lockstep import run_lockstep
    cfg = S.toy_config(d_model=192, n_heads=2, n_kv_heads=2, head_dim=64, d_ff=320, weight_std=0.1, out_std=0.02, draft_len=9,
                       layers=(1, 1, 2, 1, 1), max_batch=2, gen_faces=6, max_tokens=1 + 9 * 8 + 9 + 2)
    w, conds, prompts = _setup(cfg, batch=2)
    truth = [_oracle_greedy(cfg, w, conds[b], prompts[b], 6) for b in range(2)]
    dev = _dev(cfg, w)
    rep = run_lockstep(cfg, w, conds, prompts, dev, 6, 300, truth=truth, keep_rng=np.random.default_rng(3), tol=TOY_TOL, margin=TOY_MARGIN)
    assert rep["done"] and dev.device_status() == 0


@pytest.mark.parametrize("heads", ["reduced", "full"])
def test_toy_lockstep_forty_sequences(heads):
    """More than 32 sequences: the stacked draft projections run one launch per head, the verify
    pass has several row tiles per projection, and accept lengths differ per sequence."""
    from oracle.lockstep import run_lockstep
    B = 40
    cfg = S.toy_config(**TOY, draft_len=3, draft_heads=heads, layers=(1, 1, 1, 1, 1), max_batch=B, batch=B, gen_faces=3,
                       prompt_faces=(1, 1), max_tokens=1 + 9 * 8 + 3 + 2)
    w, conds, prompts = _setup(cfg, batch=B)
    for b in range(0, B, 3):
        prompts[b] = prompts[b] + prompts[(b + 1) % B]           # ragged: 1 and 2 faces
    truth = [_oracle_greedy(cfg, w, conds[b], prompts[b], 3) for b in range(B)]
    dev = _dev(cfg, w)
    rep = run_lockstep(cfg, w, conds, prompts, dev, 3, 120, truth=truth, keep_rng=np.random.default_rng(11), tol=TOY_TOL, margin=TOY_MARGIN)
    assert rep["done"] and rep["emitted"] == 27 * B
    assert dev.device_status() == 0
