"""GPU parity on the full-size models of the benchmark workloads (Medium, Batched ragged, Large):
a few lock-step passes each against the oracle, through the C ABI.  The oracle cannot run these
models for thousands of passes; full-length behaviour is covered by the properties checked in
test_gpu_parity.py (speculative == plain on the device) and by bench.py's own assertion."""
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
