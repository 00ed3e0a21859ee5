"""GPU parity of the correction stage (fm_correct) against its oracle: bit-exact, through the C ABI,
at every phase of the face (the row starts at an arbitrary coordinate of an arbitrary vertex)."""
import numpy as np
import pytest

import fm_synth as S

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("D", [9, 12, 24, 27])
def test_correct_matches_oracle_at_every_phase(D):
    import torch
    from oracle.correct import correct_row
    from paper_2511_15618_b200 import FlashMesh

    B = 3
    cfg = S.toy_config(d_model=128, head_dim=64, d_ff=256, draft_len=D, layers=(1, 1, 1, 1, 1), max_batch=B, n_bins=16,
                       prompt_faces=(1, 1), gen_faces=60, max_tokens=1 + 9 * 64 + D + 2)
    w = S.make_weights(cfg)
    conds = [S.make_condition(cfg, b) for b in range(B)]
    prompts = [[int(t) for t in S.make_prompt(cfg, b)] for b in range(B)]
    dev = FlashMesh(cfg, w)
    dev.prefill(np.stack(conds), prompts)
    rng = np.random.default_rng(D)
    L = np.array([1 + len(p) for p in prompts])
    hist = [list(p) for p in prompts]                # accepted mesh tokens t_0 .. t_{L-2} per sequence
    checked = moved = 0
    phases = set()
    for step in range(14):
        phases |= {int(x) % 9 for x in L}
        cand, _, _ = dev.draft()
        base = cand.cpu().numpy()
        # random drafts (few distinct values so that coincidences happen; now and then a token that
        # is not a coordinate bin), random labels; the main token stays what the library drafted
        rows = rng.integers(0, 5, size=(B, D + 1)).astype(np.int32)
        rows[rng.random((B, D + 1)) < 0.03] = cfg.n_bins + 1
        rows[:, 0] = base[:, 0]
        labels = rng.integers(0, 3, size=(B, D + 1)).astype(np.int32)
        d_rows = torch.as_tensor(rows).cuda()
        d_lab = torch.as_tensor(labels).cuda()
        out = dev.correct(d_rows, d_lab).cpu().numpy()
        out_h = dev.correct(torch.as_tensor(rows).cuda(), d_lab, use_history=True).cpu().numpy()
        # ... and with the label head's own labels (compared with the oracle's in the lock-step tests)
        own = dev.draft_labels()[0]
        out_own = dev.correct(torch.as_tensor(rows).cuda(), None, use_history=True).cpu().numpy()
        own = own.cpu().numpy()
        for b in range(B):
            assert len(hist[b]) == int(L[b]) - 1
            want = correct_row(rows[b].tolist(), labels[b].tolist(), int(L[b]), cfg.n_bins)
            assert out[b].tolist() == want, (step, b, int(L[b]), rows[b].tolist(), labels[b].tolist())
            want_h = correct_row(rows[b].tolist(), labels[b].tolist(), int(L[b]), cfg.n_bins, history=hist[b])
            assert out_h[b].tolist() == want_h, (step, b, int(L[b]), rows[b].tolist(), labels[b].tolist(), hist[b][-18:])
            want_own = correct_row(rows[b].tolist(), own[b].tolist(), int(L[b]), cfg.n_bins, history=hist[b])
            assert out_own[b].tolist() == want_own
            moved += int(want_h != want)
            checked += 1
        # move every sequence on by a different number of tokens: all nine phases get visited
        dev.verify(cand)
        force = np.array([1 + (step + b) % min(D + 1, 4) for b in range(B)], dtype=np.int32)
        n_acc, em, kv = dev.accept(force_len=force)
        em, n_acc = em.cpu().numpy(), n_acc.cpu().numpy()
        for b in range(B):
            hist[b] += [int(t) for t in em[b, :n_acc[b]]]
        L = kv.cpu().numpy()[:, 0]
    assert checked == 14 * B
    assert phases == set(range(9))                   # the rows started at every coordinate of the face
    assert moved > 0                                 # the historical rule did change rows
    assert dev.device_status() == 0


def test_correct_argument_checks():
    import torch
    from paper_2511_15618_b200 import FlashMesh, fm_correct
    cfg = S.toy_config(d_model=128, head_dim=64, d_ff=256)
    dev = FlashMesh(cfg, S.make_weights(cfg))
    x = torch.zeros((1, dev.D + 1), dtype=torch.int32, device="cuda")
    assert fm_correct(dev.ctx, x.data_ptr(), x.data_ptr()) == -2          # before fm_prefill
    assert fm_correct(dev.ctx, None, x.data_ptr()) == -1
