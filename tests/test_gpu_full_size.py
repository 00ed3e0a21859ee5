"""Full-size checks in the launch configuration the benchmark times (Medium at batch 1 with 2000
faces in the caches; the same model at batch 16 with ragged fills): the oracle cannot run these
sizes, so what is checked are properties that hold at any size -- speculative output == plain
decoding on the same kernels (bit-exact), logits of a position independent of the row it is fed
in (bit-exact), bookkeeping closed forms, tokens in range."""
import numpy as np
import pytest

import fm_synth as S

pytestmark = pytest.mark.gpu


def _setup(workload, start_faces, passes):
    import torch
    from bench import MEAN_DRAFTS
    from paper_2511_15618_b200 import FlashMesh
    cfg = S.get_config(workload)
    B, D = cfg.batch, cfg.draft_len
    need_faces = -(-(passes + 8) * (D + 1) // 9) + 1
    max_tokens = 1 + 9 * (start_faces + cfg.prompt_faces[1] + need_faces) + D + 2
    w = S.make_weights(cfg)
    conds = np.stack([S.make_condition(cfg, b) for b in range(B)])
    rng = np.random.default_rng([cfg.seed, 77, 0])
    prompts = []
    for b in range(B):
        f = start_faces if B == 1 else max(1, int(start_faces * rng.uniform(0.5, 1.0)))
        prompts.append(S.fill_prompt(cfg, b, f))
    dev = FlashMesh(cfg, w, max_tokens=max_tokens)
    del w
    keep = (S.accept_schedule(cfg.seed, B, 4096, D, MEAN_DRAFTS) - 1).astype(np.int32)
    return cfg, dev, conds, prompts, need_faces, torch.as_tensor(keep).cuda()


@pytest.mark.parametrize("workload,start_faces", [("medium", 2000), ("batched", 2000)])
def test_speculative_equals_plain_at_benchmark_size(workload, start_faces):
    import torch
    passes = 24
    cfg, dev, conds, prompts, need_faces, keep = _setup(workload, start_faces, passes)
    B, D = cfg.batch, cfg.draft_len
    dev.prefill(conds, prompts)
    plain, plen, st0 = dev.generate(need_faces, plain=True)
    pt = plain.cpu().numpy()
    assert (pt[:, :int(plen.min())] >= 0).all() and (pt[:, :int(plen.min())] < cfg.n_bins).all()     # EOS is masked in these runs
    truth = np.zeros((B, max(len(p) for p in prompts) + 9 * need_faces), dtype=np.int32)
    for b in range(B):
        seq = np.concatenate([np.asarray(prompts[b], np.int32), pt[b]])
        truth[b, :len(seq)] = seq
    truth_d = torch.as_tensor(truth).cuda()
    dev.prefill(conds, prompts)
    tok, ln, st = dev.generate(need_faces, truth=truth_d, keep=keep, max_steps=passes)
    got, n = tok.cpu().numpy(), ln.cpu().numpy()
    assert st.steps == passes and (n >= passes).all()
    for b in range(B):
        assert (got[b, :n[b]] == pt[b, :n[b]]).all()              # same tokens as one-at-a-time decoding
    assert st.emitted == int(n.sum())
    assert 0.5 * (1 + 6.7) < st.emitted / (passes * B) <= D + 1    # the teacher schedule's accept lengths
    # bookkeeping closed forms after the run
    cand, _, _ = dev.draft()
    dev.verify(cand)
    _, _, kv = dev.accept()
    kv = kv.cpu().numpy()
    assert (kv[:, 1] == -(-kv[:, 0] // 3)).all() and (kv[:, 2] == -(-kv[:, 0] // 9)).all()
    assert dev.device_status() == 0


def test_logits_do_not_depend_on_the_row_at_benchmark_size():
    """A position's logits are bit-identical whether it is verified as row j of one pass or as row
    j - 1 of the next (after one token was accepted): chunking, grouping and reduction orders are
    fixed by slot and column, not by the launch's rows or the cache length."""
    import torch
    cfg, dev, conds, prompts, need_faces, _ = _setup("medium", 2000, 8)
    D = cfg.draft_len
    dev.prefill(conds, prompts)
    plain, plen, _ = dev.generate(3, plain=True)
    pt = plain.cpu().numpy()[0]
    dev.prefill(conds, prompts)
    # candidates = the true continuation: main token, then the next D tokens of plain decoding
    cand, _, _ = dev.draft()
    c = cand.cpu().numpy()
    assert c[0, 0] == pt[0]
    c[0, 1:] = pt[1:D + 1]
    cand_a = torch.as_tensor(c).cuda()
    _, lg_a, _ = dev.verify(cand_a, want_logits=True)
    lg_a = lg_a.clone()
    dev.accept(force_len=np.array([1], dtype=np.int32))
    cand, _, _ = dev.draft()
    c2 = cand.cpu().numpy()
    assert c2[0, 0] == pt[1]
    c2[0, 1:] = pt[2:D + 2]
    _, lg_b, _ = dev.verify(torch.as_tensor(c2).cuda(), want_logits=True)
    assert torch.equal(lg_a[0, 1:], lg_b[0, :D])


@pytest.mark.parametrize("workload,n_tok", [("medium", 130), ("batched", 70), ("large", 60)])
def test_every_accept_pattern_leaves_the_logits_of_plain_decoding(workload, n_tok):
    """Bit-exact losslessness (Sec. 3.3) at benchmark size.  A position's hidden states reach the
    upper stacks along different code paths depending on where the passes happen to start: with its
    parent vertex or face computed in the same pass, or in an earlier one (stored upsampled slot).
    Decoding one token per pass takes the second path almost always, accepting whole passes takes
    the first.  The logits of every position must not depend on that, to the last bit -- a
    difference of one rounding in an operand row is enough to flip a near-tie thousands of tokens
    later and let speculative output drift away from plain decoding."""
    import torch
    from paper_2511_15618_b200 import FlashMesh
    cfg = S.get_config(workload)
    faces = n_tok // 9 + 8
    cfg = cfg.with_(gen_faces=faces, max_tokens=1 + 9 * (cfg.prompt_faces[1] + faces) + cfg.draft_len + 1)
    B, D = cfg.batch, cfg.draft_len
    w = S.make_weights(cfg)
    conds = np.stack([S.make_condition(cfg, b) for b in range(B)])
    prompts = [[int(t) for t in S.make_prompt(cfg, b)] for b in range(B)]
    dev = FlashMesh(cfg, w)
    del w
    dev.prefill(conds, prompts)
    plain, _, _ = dev.generate(faces, plain=True)
    pt = plain.cpu().numpy()

    def walk(pattern):
        dev.prefill(conds, prompts)
        got, n, step = {}, 0, 0
        while n + D + 1 < n_tok:
            cand, _, _ = dev.draft()
            c = cand.cpu().numpy()
            assert (c[:, 0] == pt[:, n]).all()
            c[:, 1:] = pt[:, n + 1:n + 1 + D]                  # drafts = the true continuation
            _, lg, _ = dev.verify(torch.as_tensor(c).cuda(), want_logits=True)
            a = pattern[step % len(pattern)]
            for j in range(a):
                got[n + j] = lg[:, j].clone()
            dev.accept(force_len=np.full(B, a, dtype=np.int32))
            n += a
            step += 1
        return got

    ref = walk([1])
    for pattern in ([D + 1], [2], [4, 7, 1, D + 1, 2, 9, 5]):
        got = walk(pattern)
        common = [k for k in sorted(got) if k in ref]
        assert len(common) > n_tok - 2 * (D + 1)
        bad = [k for k in common if not torch.equal(got[k], ref[k])]
        assert not bad, (pattern, bad[:5])
    assert dev.device_status() == 0
