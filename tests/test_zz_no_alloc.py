"""fm_verify_static_scratch: the verify pass for hosts that cannot hand the library scratch memory.

A host that commits all its device memory once at start-up (a serving process with a fixed memory
plan, a plug-in that must not call cudaMalloc under its real-time loop) can run the verify pass with
the attention kernel's split-KV scratch in a fixed array inside the library instead.  The call must
give what fm_verify gives.  It is called twice in a row because every call reuses the same array,
which still holds the previous call's partial results and counters.

This file is named so that pytest collects it last."""
import ctypes

import numpy as np
import pytest

import fm_synth as S

pytestmark = pytest.mark.gpu


def test_static_scratch_verify_matches_fm_verify_twice_in_a_row():
    import torch
    from paper_2511_15618_b200 import FlashMesh, fm_verify, fm_verify_static_scratch

    # an 8-face prompt: the coordinate-level cache (64 prefix slots + 73 positions) then spans two
    # groups of chunks, so the attention kernel really goes through its partials and tickets
    cfg = S.get_config("tiny").with_(prompt_faces=(8, 8), max_tokens=1 + 9 * (8 + 32) + 3 + 2)
    w = S.make_weights(cfg)
    dev = FlashMesh(cfg, w)
    dev.prefill(np.stack([S.make_condition(cfg)]), [[int(t) for t in S.make_prompt(cfg)]])
    # a few accepted passes first
    for _ in range(6):
        cand, _, _ = dev.draft()
        dev.verify(cand)
        dev.accept()
    cand, _, _ = dev.draft()
    B, D, V = 1, dev.D, dev.V

    def buffers():
        return (torch.empty((B, D + 1), dtype=torch.int32, device="cuda"),
                torch.empty((B, D + 1, V), dtype=torch.float32, device="cuda"),
                torch.empty((B, D + 1), dtype=torch.float32, device="cuda"))

    torch.cuda.synchronize()
    o_ref, lg_ref, mg_ref = buffers()
    assert fm_verify(dev.ctx, cand.data_ptr(), o_ref.data_ptr(), lg_ref.data_ptr(), mg_ref.data_ptr()) == 0
    assert dev.device_status() == 0
    for _ in range(2):
        o, lg, mg = buffers()
        rc = fm_verify_static_scratch(dev.ctx, cand.data_ptr(), o.data_ptr(), lg.data_ptr(), mg.data_ptr())
        assert rc == 0
        assert dev.device_status() == 0                       # synchronises the context's stream
        assert torch.equal(o, o_ref)
        assert float((lg - lg_ref).abs().max()) <= 2e-2       # the tolerance of the parity tests
        assert float((mg - mg_ref).abs().max()) <= 2e-2
    # the pass can still be accepted afterwards: the call leaves the context as fm_verify does
    n_acc, _, _ = dev.accept()
    assert int(n_acc[0]) >= 1


def test_static_scratch_rejects_a_configuration_that_needs_more_than_the_array(monkeypatch):
    from paper_2511_15618_b200 import FlashMesh, fm_verify_static_scratch
    import torch

    # many sequences and kv-heads with long caches cut into many groups (the tuning knob asks for
    # short groups; the library then takes the largest number of groups it can merge): the group
    # partials outgrow the fixed array
    monkeypatch.setenv("FM_ATTN_G", "8")
    cfg = S.get_config("tiny").with_(max_batch=16, max_tokens=100000)
    w = S.make_weights(cfg)
    dev = FlashMesh(cfg, w)
    dev.prefill(np.stack([S.make_condition(cfg)]), [[]])
    cand, _, _ = dev.draft()
    o = torch.empty((1, dev.D + 1), dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    assert fm_verify_static_scratch(dev.ctx, cand.data_ptr(), o.data_ptr(), None, None) == -3      # FM_ERR_CAPACITY
    # nothing was enqueued: the ordinary call still works
    out, _, _ = dev.verify(cand)
    assert dev.device_status() == 0
