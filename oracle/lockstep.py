"""Lock-step comparison of a device implementation against the oracle.  TEST INFRASTRUCTURE.

The history is always the oracle's: at every pass the device gets the oracle's candidates,
its verify logits / argmax / margins are compared, and acceptance is either left to the
device (when every compared row agreed) or overridden with the oracle's argmax (allowed only
where the oracle's top-2 margin is <= `margin`, where bfloat16 may legitimately flip it).
The device object is passed in (duck-typed: prefill, draft, verify, accept); this module
imports nothing from the CUDA package.
"""
from __future__ import annotations

import numpy as np

from .hourglass import OracleSeq


def _np(x):
    return x.detach().cpu().numpy() if hasattr(x, "detach") else np.asarray(x)


def run_lockstep(cfg, w, conds, prompts, dev, max_faces, max_steps, *, tol=2e-2, margin=0.1, truth=None,
                 keep_rng=None, check_drafts=True, dtype=np.float64, prefill_chunk=None, seq_max_tokens=None):
    """Returns a report dict; raises AssertionError on a parity failure.

    truth: optional per-sequence known continuation (mesh tokens, prompt included) used to
    overwrite drafts so that accept lengths vary (keep_rng draws how many are kept).
    prefill_chunk: the oracle consumes the prompts that many rows at a time (long prompts).
    seq_max_tokens: per-sequence cache capacity of the oracle's sequences (default: cfg's)."""
    B, D, V = len(prompts), cfg.draft_len, cfg.vocab
    seqs = []
    for b in range(B):
        c = cfg if seq_max_tokens is None else cfg.with_(max_tokens=int(seq_max_tokens[b]))
        # the first sequence converts the weights to `dtype`; the others share those arrays
        seqs.append(OracleSeq(c, w if b == 0 else seqs[0].w, dtype))
    for b in range(B):
        seqs[b].prefill(conds[b], prompts[b], max_faces=max_faces[b] if hasattr(max_faces, "__len__") else max_faces,
                        chunk=prefill_chunk)
    dev.prefill(np.stack(conds), prompts)
    dev.set_max_faces([max_faces[b] if hasattr(max_faces, "__len__") else max_faces for b in range(B)])
    rep = dict(steps=0, emitted=0, overrides=0, max_logit_err=0.0, max_draft_err=0.0, rows=0, low_margin_rows=0,
               argmax_flips=0, draft_flips=0, accept_hist=[0] * (D + 2), labels=0, label_flips=0)
    check_labels = check_drafts and D > 0 and cfg.draft_levels == "three" and hasattr(dev, "draft_labels")
    for _ in range(max_steps):
        if all(s.done for s in seqs):
            break
        # ---- draft
        o_d = [s.draft() for s in seqs]
        cand_g, dl_g, dm_g = dev.draft(want_logits=check_drafts)
        cand_g = _np(cand_g)
        if check_drafts and D > 0:
            dl_g = _np(dl_g)
            for b, s in enumerate(seqs):
                if s.done:
                    assert (cand_g[b] == cfg.pad).all()
                    continue
                err = float(np.abs(dl_g[b] - o_d[b][1]).max())
                rep["max_draft_err"] = max(rep["max_draft_err"], err)
                assert err <= tol, f"draft logits off by {err}"
                for j in range(1, D + 1):
                    if o_d[b][2][j - 1] > margin:
                        assert cand_g[b, j] == o_d[b][0][j], "draft id differs at a decisive margin"
                    elif cand_g[b, j] != o_d[b][0][j]:
                        rep["draft_flips"] += 1
        # ---- labels of the drafted points (Sec. 3.2): equal where the oracle's margin is decisive
        if check_labels:
            lab_g = _np(dev.draft_labels()[0])
            for b, s in enumerate(seqs):
                if s.done:
                    assert (lab_g[b] == -1).all()
                    continue
                lab_o, lmg_o = s.draft_labels()
                for sl in range(D + 1):
                    assert (lab_g[b, sl] == -1) == (lab_o[sl] == -1), "label slots differ"
                    if lab_o[sl] >= 0:
                        rep["labels"] += 1
                        if lmg_o[sl] > margin:
                            assert lab_g[b, sl] == lab_o[sl], "label differs at a decisive margin"
                        elif lab_g[b, sl] != lab_o[sl]:
                            rep["label_flips"] += 1
        # ---- candidates: the oracle's, optionally teacher-edited
        cands = []
        for b, s in enumerate(seqs):
            c = list(o_d[b][0])
            if truth is not None and not s.done:
                n = s.L - 1
                keep = int(keep_rng.integers(0, D + 1)) if keep_rng is not None else D
                for j in range(1, D + 1):
                    t = truth[b][n + j] if n + j < len(truth[b]) else 0
                    c[j] = t if j <= keep else ((t + 1) % cfg.n_bins if j == keep + 1 else c[j])
            cands.append(c)
        # ---- verify
        o_v = [s.verify(cands[b]) for b, s in enumerate(seqs)]
        og, lg, mg = dev.verify(np.asarray(cands, dtype=np.int32), want_logits=True)
        og, lg = _np(og), _np(lg)
        agree = True
        for b, s in enumerate(seqs):
            rows = s.rows
            assert (og[b, rows:] == -1).all()
            if rows == 0:
                continue
            err = float(np.abs(lg[b, :rows] - o_v[b][1][:rows]).max())
            rep["max_logit_err"] = max(rep["max_logit_err"], err)
            assert err <= tol, f"verify logits off by {err} (sequence {b}, L={s.L})"
            for j in range(rows):
                rep["rows"] += 1
                if o_v[b][2][j] > margin:
                    assert og[b, j] == o_v[b][0][j], "argmax differs at a decisive margin"
                else:
                    rep["low_margin_rows"] += 1
                    if og[b, j] != o_v[b][0][j]:
                        rep["argmax_flips"] += 1
                        agree = False
        # ---- accept
        force = None if agree else np.asarray([o_v[b][0] for b in range(B)], dtype=np.int32)
        if not agree:
            rep["overrides"] += 1
        n_g, em_g, kv_g = (_np(x) for x in dev.accept(force_tok=force))
        for b, s in enumerate(seqs):
            a, em, kv = s.accept()
            assert int(n_g[b]) == a, f"accept length {int(n_g[b])} != {a}"
            assert list(em_g[b]) == em and tuple(kv_g[b]) == kv
            rep["emitted"] += a
            rep["accept_hist"][a] += 1
        rep["steps"] += 1
    rep["done"] = all(s.done for s in seqs)
    return rep
