"""fm_verify_static_scratch: the verify pass for hosts that cannot hand the library scratch memory.

A host that commits all its device memory once at start-up (a serving process with a fixed memory
plan, a plug-in that must not call cudaMalloc under its real-time loop) can run the verify pass with
the attention kernel's split-KV scratch in a fixed array inside the library instead.  The call must
give what fm_verify gives.  It is called twice in a row because every call reuses the same array,
which still holds the previous call's partial results and counters.

This file is named so that pytest collects it last."""
import numpy as np
import pytest

import fm_synth as S

pytestmark = pytest.mark.gpu


def test_static_scratch_verify_matches_fm_verify_twice_in_a_row(monkeypatch):
    import torch
    from paper_2511_15618_b200 import FlashMesh, fm_attention_layout, fm_verify, fm_verify_static_scratch

    # One chunk per group (the library's tuning knob, read when the context is created), so that the
    # 72-face prompt spreads a head's cache over several CTAs at all three levels: only then do the
    # partial results and the ticket counters, i.e. the static array, come into play.
    monkeypatch.setenv("FM_ATTN_G", "1")
    cfg = S.get_config("tiny").with_(prompt_faces=(72, 72), max_tokens=1 + 9 * (72 + 32) + 3 + 2)
    w = S.make_weights(cfg)
    dev = FlashMesh(cfg, w)
    dev.prefill(np.stack([S.make_condition(cfg)]), [[int(t) for t in S.make_prompt(cfg)]])
    # a few accepted passes first
    for _ in range(6):
        cand, _, _ = dev.draft()
        dev.verify(cand)
        _, _, kv = dev.accept()
    cand, _, _ = dev.draft()
    B, D, V = 1, dev.D, dev.V
    # groups a head's cache is cut into right now, by the library's own arithmetic: at every level
    # more than one, so every attention launch of the pass merges through the scratch array
    kv = kv.cpu().numpy()[0]
    for level in range(3):
        rc, (chunk, per_group, max_groups) = fm_attention_layout(dev.ctx, level)
        assert rc == 0 and per_group == 1
        slots = cfg.n_prefix + int(kv[level]) + 1
        groups = -(-(-(-slots // chunk)) // per_group)
        assert 2 <= groups <= max_groups, (level, slots, chunk, groups)

    def buffers():
        return (torch.empty((B, D + 1), dtype=torch.int32, device="cuda"),
                torch.empty((B, D + 1, V), dtype=torch.float32, device="cuda"),
                torch.empty((B, D + 1), dtype=torch.float32, device="cuda"))

    def plain_verify():
        o, lg, mg = buffers()
        assert fm_verify(dev.ctx, cand.data_ptr(), o.data_ptr(), lg.data_ptr(), mg.data_ptr()) == 0
        assert dev.device_status() == 0                       # synchronises the context's stream
        return o, lg, mg

    torch.cuda.synchronize()
    o_ref, lg_ref, mg_ref = plain_verify()
    outs = [buffers() for _ in range(2)]
    for i, (o, lg, mg) in enumerate(outs):
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        rc = fm_verify_static_scratch(dev.ctx, cand.data_ptr(), o.data_ptr(), lg.data_ptr(), mg.data_ptr())
        assert rc == 0
        assert dev.device_status() == 0
        assert torch.cuda.mem_get_info()[0] == free_before    # the call took no device memory
        # same kernels, same reduction order, only the scratch lives elsewhere: identical bits
        assert torch.equal(o, o_ref) and torch.equal(lg, lg_ref) and torch.equal(mg, mg_ref)
        if i == 0:
            # the context's own scratch is untouched by the call: the ordinary pass still gives the same
            o2, lg2, mg2 = plain_verify()
            assert torch.equal(o2, o_ref) and torch.equal(lg2, lg_ref) and torch.equal(mg2, mg_ref)
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
