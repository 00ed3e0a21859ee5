"""GPU parity on the full-size models of the benchmark workloads (Medium, Batched ragged, Large):
a few lock-step passes each against the oracle, through the C ABI -- right after a short prompt,
and with the caches filled the way the benchmark fills them (a 1000-face prefix: the coordinate
ring of the 8192-token window has wrapped, every head's cache is read by many CTAs), at batch 1
and at batch 16 with ragged fills.  The oracle cannot run these models for thousands of passes;
full-length behaviour is covered by the properties checked in test_gpu_full_size.py."""
import numpy as np
import pytest

import fm_synth as S

pytestmark = pytest.mark.gpu


def _dev(cfg, w, **kw):
    from paper_2511_15618_b200 import FlashMesh
    return FlashMesh(cfg, w, **kw)


def _greedy(cfg, w, cond, prompt, faces, dtype):
    from oracle.hourglass import OracleSeq
    s = OracleSeq(cfg, w, dtype)
    s.prefill(cond, prompt, max_faces=faces)
    out, _ = s.generate(faces, force_plain=True)
    return list(prompt) + out


def test_medium_model_lockstep_with_teacher_drafts():
    from oracle.lockstep import run_lockstep
    faces = 4
    cfg = S.get_config("medium").with_(gen_faces=faces, max_tokens=1 + 9 * (8 + faces) + 9 + 2)
    w = S.make_weights(cfg)
    conds = [S.make_condition(cfg)]
    prompts = [[int(t) for t in S.make_prompt(cfg)]]
    truth = [_greedy(cfg, w, conds[0], prompts[0], faces, np.float64)]
    dev = _dev(cfg, w)
    rep = run_lockstep(cfg, w, conds, prompts, dev, faces, 100, truth=truth, keep_rng=np.random.default_rng(3))
    assert rep["done"] and rep["emitted"] == 9 * faces and rep["max_logit_err"] <= 2e-2
    assert dev.device_status() == 0
    print(rep)


def test_medium_model_full_draft_modules_lockstep():
    """Medium with the full SP-Blocks and HF-Blocks: draft logits of all three pipelines against the
    oracle for a few passes behind a 40-face prefix."""
    from oracle.lockstep import run_lockstep
    fill, faces = 40, 2
    cfg = S.get_config("medium").with_(draft_heads="full", gen_faces=faces, max_tokens=1 + 9 * (fill + faces) + 9 + 2)
    w = S.make_weights(cfg)
    conds = [S.make_condition(cfg)]
    prompts = [S.fill_prompt(cfg, 0, fill)]
    dev = _dev(cfg, w)
    rep = run_lockstep(cfg, w, conds, prompts, dev, faces, 6, prefill_chunk=512)
    assert rep["steps"] == 6 and rep["max_logit_err"] <= 2e-2 and rep["max_draft_err"] <= 2e-2
    assert dev.device_status() == 0
    print(rep)


def test_batched_ragged_lockstep():
    from oracle.lockstep import run_lockstep
    B = 4
    cfg = S.get_config("batched").with_(max_batch=B, batch=B, max_tokens=1 + 9 * (64 + 3) + 9 + 2)
    w = S.make_weights(cfg)
    conds = [S.make_condition(cfg, b) for b in range(B)]
    prompts = [[int(t) for t in S.make_prompt(cfg, b)] for b in range(B)]
    assert len({len(p) for p in prompts}) > 1                  # ragged prompt lengths
    dev = _dev(cfg, w)
    # per-sequence limits differ, so rows go inactive at different passes
    rep = run_lockstep(cfg, w, conds, prompts, dev, [1, 2, 1, 2], 12)
    assert rep["steps"] >= 9 and rep["max_logit_err"] <= 2e-2 and rep["max_draft_err"] <= 2e-2
    assert dev.device_status() == 0
    print(rep)


def test_large_model_lockstep_head_dim_128():
    from oracle.lockstep import run_lockstep
    B = 2
    cfg = S.get_config("large").with_(max_batch=B, batch=B, max_tokens=1 + 9 * (8 + 2) + 12 + 2)
    w = S.make_weights(cfg)
    conds = [S.make_condition(cfg, b) for b in range(B)]
    prompts = [[int(t) for t in S.make_prompt(cfg, b)] for b in range(B)]
    dev = _dev(cfg, w)
    # float32 oracle: the float64 copy of 2 G parameters would need 16 GB; the two modes agree to 1e-4
    rep = run_lockstep(cfg, w, conds, prompts, dev, 1, 6, dtype=np.float32)
    assert rep["steps"] == 6 and rep["max_logit_err"] <= 2e-2 and rep["max_draft_err"] <= 2e-2
    assert dev.device_status() == 0
    print(rep)


def test_medium_lockstep_with_the_benchmarks_cache_fill():
    """Medium at batch 1 behind a 1000-face prefix (9001 coordinate positions: beyond the 8192
    window, so the ring has wrapped and old chunks are fully visible while the newest are masked;
    69 chunks at the coordinate level, 28 at the vertex level), teacher drafts, 7 passes."""
    from oracle.lockstep import run_lockstep
    fill, faces = 1000, 3
    cfg = S.get_config("medium").with_(gen_faces=faces, max_tokens=1 + 9 * (fill + faces) + 9 + 2)
    w = S.make_weights(cfg)
    conds = [S.make_condition(cfg)]
    prompts = [S.fill_prompt(cfg, 0, fill)]
    from oracle.hourglass import OracleSeq
    ref = OracleSeq(cfg, w)
    ref.prefill(conds[0], prompts[0], max_faces=faces, chunk=512)
    w64 = ref.w                                           # float64 copies, shared with the lock-step run
    out, _ = ref.generate(faces, force_plain=True)
    truth = [list(prompts[0]) + out]
    del ref
    dev = _dev(cfg, w)
    from paper_2511_15618_b200 import fm_attention_layout
    _, (chunk, per_group, _) = fm_attention_layout(dev.ctx, 0)
    assert -(-(-(-(cfg.n_prefix + cfg.window[0]) // chunk)) // per_group) >= 9      # groups per head at the coordinate level
    rep = run_lockstep(cfg, w64, conds, prompts, dev, faces, 7, truth=truth, keep_rng=np.random.default_rng(11),
                       prefill_chunk=512)
    assert rep["steps"] >= 6 and rep["max_logit_err"] <= 2e-2 and rep["max_draft_err"] <= 2e-2
    assert sum(1 for a in rep["accept_hist"][2:] if a > 0) >= 2            # accept lengths varied
    assert dev.device_status() == 0
    print(rep)


def test_batch16_ragged_lockstep_with_long_and_short_caches():
    """The batched workload at its full batch of 16: ragged fills from 30 to 960 faces (two
    sequences beyond the coordinate window), 4 passes.  float32 oracle (sixteen float64 caches
    would not fit comfortably in host memory; the two modes agree to 1e-4)."""
    from oracle.lockstep import run_lockstep
    B = 16
    fills = [960, 30, 55, 80, 120, 40, 200, 64, 930, 33, 150, 47, 300, 72, 90, 500]
    cfg = S.get_config("batched").with_(max_tokens=1 + 9 * (max(fills) + 5) + 9 + 2)
    w = S.make_weights(cfg)
    conds = [S.make_condition(cfg, b) for b in range(B)]
    prompts = [S.fill_prompt(cfg, b, fills[b]) for b in range(B)]
    dev = _dev(cfg, w)
    caps = [1 + 9 * (f + 5) + 9 + 2 for f in fills]
    rep = run_lockstep(cfg, w, conds, prompts, dev, 4, 4, dtype=np.float32, prefill_chunk=512, seq_max_tokens=caps)
    assert rep["steps"] == 4 and rep["max_logit_err"] <= 2e-2 and rep["max_draft_err"] <= 2e-2
    assert dev.device_status() == 0
    print(rep)
