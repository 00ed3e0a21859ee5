#!/usr/bin/env python
"""Benchmark of the speculative decode step (draft -> verify -> accept) on synthetic inputs.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload medium]

A step is one pass of the whole hot path over the batch.  The metric is mesh tokens/s.  The
timed region starts with the model, the KV caches (filled to the middle of the configured run)
and the teacher schedule resident in HBM.  One JSON line is printed by rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import fm_synth as S  # noqa: E402

METRIC = "mesh_tokens_per_s"
MEAN_DRAFTS = 6.7          # accepted drafts per pass of the paper's 9-9 row (6.43 .. 6.97 of 9)


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def _fill_prompt(cfg, seq, n_faces):
    return S.fill_prompt(cfg, seq, n_faces)


def reduce_over_ranks(maxed, summed, device):
    """Whole-job figures from per-rank ones: element-wise MAX of `maxed` (times) and SUM of
    `summed` (tokens, launches) over the ranks of the default process group.  Sequences are
    independent, so this reduction of the report is the only communication of a multi-GPU run."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return list(maxed), list(summed)
    tm = torch.tensor(list(maxed), dtype=torch.float64, device=device)
    ts = torch.tensor(list(summed), dtype=torch.float64, device=device)
    dist.all_reduce(tm, op=dist.ReduceOp.MAX)
    dist.all_reduce(ts, op=dist.ReduceOp.SUM)
    return tm.tolist(), ts.tolist()


def rank_sequences(rank, batch_per_rank):
    """Global sequence ids (seeds of conditioning and prompts) owned by a rank: weak scaling, every
    rank decodes its own `batch_per_rank` sequences."""
    return [rank * batch_per_rank + b for b in range(batch_per_rank)]


# DRAM traffic of the dominant kernel per launch from ncu (dram__bytes_read.sum +
# dram__bytes_write.sum), keyed by workload, each with the summary under profiles/ that holds the
# capture; None where the kernel changed since the capture or none was taken.
NCU_TRAFFIC = {"medium": {"bytes_per_launch": 6.46e6, "summary": "profiles/gemm_and_attention_dram_traffic_medium.md"}}


class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.path = index, None, None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.index)], stdout=open(self.path, "w"),
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, reasons = [], set()
        for ln in open(self.path):
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                out["sm_max_mhz"] = float(f[2])
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        os.unlink(self.path)
        if sm:
            out["sm_mhz"] = float(np.median(sm))
        out["reasons"] = sorted(reasons)
        return out


# -------------------------------------------------------------------------------------------
# our arm
# -------------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2511_15618_b200 import FlashMesh
    from paper_2511_15618_b200.build import build

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    torch.cuda.set_device(local)
    if rank == 0:
        build()
    if world > 1:
        dist.barrier()
    cfg = S.get_config(args.workload)
    if args.draft_len >= 0:               # cost curve of the pass against the number of drafts
        cfg = cfg.with_(draft_len=args.draft_len)
    cfg = cfg.with_(draft_heads=args.draft_heads, draft_levels=args.draft_levels)
    if args.kv_heads > 0:
        cfg = cfg.with_(n_kv_heads=args.kv_heads)
    if args.full_run:
        return run_full_length(args, cfg, rank, local)
    B, D = cfg.batch, cfg.draft_len
    K, W = args.steps, args.warmup
    start_faces = int(cfg.gen_faces * args.start_frac)
    need_faces = -(-(K + W + 8) * (D + 1) // 9) + 1
    max_tokens = 1 + 9 * (start_faces + cfg.prompt_faces[1] + need_faces) + D + 2
    w = S.make_weights(cfg)
    seqs = rank_sequences(rank, B)
    conds = np.stack([S.make_condition(cfg, q) for q in seqs])
    rng = np.random.default_rng([cfg.seed, 77, rank])
    prompts = []
    for b in range(B):                    # ragged fills around the target (exact for batch 1)
        f = start_faces if B == 1 else max(1, int(start_faces * rng.uniform(0.5, 1.0)))
        prompts.append(_fill_prompt(cfg, seqs[b], f))
    dev = FlashMesh(cfg, w, device=f"cuda:{local}", max_tokens=max_tokens)
    del w

    # untimed set-up: the continuation the teacher drafts come from (plain decoding on the same kernels)
    dev.prefill(conds, prompts)
    plain_tok, plain_len, st_plain = dev.generate(need_faces, plain=True)
    t_ori_ms = st_plain.ms / max(1, st_plain.steps)
    truth = np.full((B, max(len(p) for p in prompts) + 9 * need_faces), 0, dtype=np.int32)
    pt = plain_tok.cpu().numpy()
    for b in range(B):
        seq = np.concatenate([np.asarray(prompts[b], np.int32), pt[b]])
        truth[b, :len(seq)] = seq
    keep = (S.accept_schedule(cfg.seed + rank, B, 4096, D, MEAN_DRAFTS) - 1).astype(np.int32)
    if args.pin_accept > 0:               # every pass accepts exactly this many tokens (main + drafts)
        keep[:] = min(D, args.pin_accept - 1)
    truth_d = torch.as_tensor(truth).cuda()
    keep_d = torch.as_tensor(keep).cuda()

    def sync_all():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- timed: K passes, inputs resident in HBM
    dev.prefill(conds, prompts)
    out = None
    if W > 0:
        tok, ln, _ = dev.generate(need_faces, truth=truth_d, keep=keep_d, max_steps=W)
        out = (tok, ln)
    sampler = ClockSampler(local)
    sampler.start()
    l0 = dev.launch_count()
    sync_all()
    torch.cuda.profiler.start()           # lets `ncu --profile-from-start off` see only the timed passes
    tok, ln, st = dev.generate(need_faces, truth=truth_d, keep=keep_d, max_steps=K, out=out)
    sync_all()
    torch.cuda.profiler.stop()
    launches = dev.launch_count() - l0
    clocks = sampler.stop()
    ms, emitted, steps = float(st.ms), int(st.emitted), int(st.steps)
    # generated tokens must be the plain-decoding continuation (teacher drafts change speed, not output)
    got = tok.cpu().numpy()
    n_chk = int(ln.cpu().numpy().min())
    assert (got[:, :n_chk] == pt[:, :n_chk]).all(), "speculative output differs from plain decoding"

    if args.timed_only:
        cand, _, _ = dev.draft()
        dev.verify(cand)
        _, _, kv = dev.accept()
        sb = dev.verify_bytes(kv.cpu().numpy().tolist())
        peak, _ = _peaks()
        cand, _, _ = dev.draft()
        dev.verify(cand)
        g_ms, g_n, g_b = dev.profile_class(0, 20)
        a_ms, a_n, _ = dev.profile_class(1, 20)
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": emitted / (ms * 1e-3), "unit": "tokens/s", "workload": args.workload,
                              "gemm": {"launches": g_n, "us_per_launch": 1e3 * g_ms / max(1, g_n), "weight_bytes": g_b},
                              "attention": {"launches": a_n, "us_per_launch": 1e3 * a_ms / max(1, a_n)},
                              "batch": B, "ms_per_step": ms / max(1, steps), "steps": steps, "gpu_launches": launches,
                              "mean_accept_len": emitted / max(1, steps * B),
                              "verify_step_frac_of_hbm_peak": sb / (ms / max(1, steps) * 1e-3) / 1e9 / peak,
                              "note": "timed passes only"}), flush=True)
        return

    # ---- lengths at the end of the timed passes -> algorithmic bytes of a verify pass there
    cand, _, _ = dev.draft()
    dev.verify(cand)
    _, _, kv = dev.accept()
    kv_len = kv.cpu().numpy().tolist()
    step_bytes = dev.verify_bytes(kv_len)
    # ---- the dominant kernels timed alone, live: the GEMM launches (resp. the attention launches) of
    # one verify pass at these lengths, same arguments and data, replayed as a CUDA graph between two
    # events on the context's stream
    cand, _, _ = dev.draft()
    dev.verify(cand)
    gemm_ms, gemm_n, gemm_bytes = dev.profile_class(0, 30)
    attn_ms, attn_n, _ = dev.profile_class(1, 30)

    # ---- natural acceptance of the (random-weight) heads, same state
    dev.prefill(conds, prompts)
    _, _, st_nat = dev.generate(need_faces, max_steps=max(8, K // 4))

    # ---- end to end: host in the loop (stepwise C ABI, pinned host buffers, copies inside the timing)
    dev.prefill(conds, prompts)
    e2e = run_e2e(dev, cfg, truth, keep, prompts, max(8, min(K, 64)))

    peak, peak_kind = _peaks()
    (ms, e2e_s), (emitted, launches, e2e_tok) = reduce_over_ranks(
        [ms, e2e["seconds"]], [float(emitted), float(launches), e2e["tokens"]], "cuda")
    emitted, launches = int(emitted), int(launches)
    e2e["tokens"], e2e["seconds"] = e2e_tok, e2e_s
    value = emitted / (ms * 1e-3)
    gemm_gbs = gemm_bytes / (gemm_ms * 1e-3) / 1e9 if gemm_ms > 0 else 0.0
    kv_bytes = step_bytes - gemm_bytes                     # what the attention launches must read
    step_ms = ms / max(1, steps)
    line = {
        "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "batch_per_gpu": B, "draft_len": D,
                   "kv_fill": f"prefix of {start_faces} faces per sequence already in the caches "
                              f"(middle of the {cfg.gen_faces}-face run)",
                   "acceptance": f"teacher drafts, seeded schedule, mean {MEAN_DRAFTS} drafts kept per pass",
                   "l2": "weights streamed per pass exceed the 126 MB L2; no flush between passes",
                   "parallelism": f"replicas x{world}"},
        "mean_accept_len": emitted / max(1, steps * B * world),
        "natural_accept_len": st_nat.emitted / max(1, st_nat.steps * B),
        "natural_tokens_per_s": st_nat.emitted / (st_nat.ms * 1e-3),
        # the same D-draft pass with acceptance forced to one token (NOT T_ori of Sec. 4.1, which is
        # the D = 0 run reported under "plain_decoding")
        "single_accept_tokens_per_s": B / (t_ori_ms * 1e-3), "single_accept_ms_per_step": t_ori_ms,
        "clocks": clocks,
        "e2e": {"value": e2e["tokens"] / e2e["seconds"], "unit": "tokens/s",
                "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                "what": "fm_step_host once per pass with the host in the loop: candidates from pinned host memory "
                        "in, draft + verify + accept, accepted tokens copied back, per pass"},
        "gpu_launches": launches,
        "roofline": {"bound": "hbm", "kernel": "tc::gemm_tc_kernel (all GEMM launches of one verify pass, timed alone as a graph)",
                     "achieved": gemm_gbs, "peak": peak, "unit": "GB/s", "frac": gemm_gbs / peak,
                     "peak_kind": peak_kind + " copy bandwidth (burst figure: the kernel is timed alone)",
                     "traffic": NCU_TRAFFIC.get(args.workload, {}).get("bytes_per_launch"),
                     "traffic_source": NCU_TRAFFIC.get(args.workload, {}).get("summary"),
                     "algorithmic_bytes_per_launch": gemm_bytes / max(1, gemm_n),
                     "launches_per_pass": int(gemm_n), "us_per_launch": gemm_ms * 1e3 / max(1, gemm_n),
                     "second_kernel": {"kernel": "attn_stream_kernel (all attention launches of one verify pass)",
                                       "achieved": kv_bytes / (attn_ms * 1e-3) / 1e9 if attn_ms > 0 else 0.0,
                                       "frac": kv_bytes / (attn_ms * 1e-3) / 1e9 / peak if attn_ms > 0 else 0.0,
                                       "launches_per_pass": int(attn_n), "us_per_launch": attn_ms * 1e3 / max(1, attn_n)}},
        "verify_step": {"algorithmic_bytes": step_bytes, "ms": step_ms, "GB/s": step_bytes / (step_ms * 1e-3) / 1e9,
                        "frac_of_hbm_peak": step_bytes / (step_ms * 1e-3) / 1e9 / peak, "kv_len": kv_len[0],
                        "note": "whole pass (draft heads + verify + accept) against the verify bytes"},
    }
    # ---- the correction stage between draft and verify (an integer kernel, outside the timed passes):
    # random labels on the drafts of the current state, 200 calls between two events
    cand, _, _ = dev.draft()
    lab = torch.randint(0, 3, cand.shape, dtype=torch.int32, device=cand.device)
    for _ in range(5):
        dev.correct(cand.clone(), lab)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    work = [cand.clone() for _ in range(200)]
    e0.record()
    for w_ in work:
        dev.correct(w_, lab)
    e1.record()
    torch.cuda.synchronize()
    line["correct_stage"] = {"us_per_call": 1e3 * e0.elapsed_time(e1) / 200, "batch": B, "slots_per_row": D + 1,
                             "note": "fm_correct on random labels; host bound (binding call + launch per call); not part of the timed passes"}
    if rank == 0:
        if world == 1 and args.workload == "medium" and not args.no_batched:
            # the metric also asks for batch 16: the batched-ragged workload, timed passes only
            dev.close()
            del dev
            torch.cuda.empty_cache()
            r = subprocess.run([sys.executable, os.path.abspath(__file__), "--workload", "batched", "--steps", "30", "--warmup", "3",
                                "--timed-only", "--no-cpu"], capture_output=True, text=True)
            try:
                line["batch16"] = json.loads(r.stdout.strip().splitlines()[-1])
            except Exception:
                line["batch16"] = {"error": (r.stderr or r.stdout)[-300:]}
        if world == 1 and args.draft_len < 0 and not args.no_batched:
            # T_ori of Sec. 4.1: the same model decoding one token per pass (D = 0, so the vertex and
            # face stacks only run at multiples of 3 and 9), same kernels, same cache fill
            try:
                dev.close()
                del dev
                torch.cuda.empty_cache()
            except NameError:
                pass
            r = subprocess.run([sys.executable, os.path.abspath(__file__), "--workload", args.workload, "--steps", "90", "--warmup", "9",
                                "--draft-len", "0", "--timed-only", "--no-cpu"], capture_output=True, text=True)
            try:
                p0 = json.loads(r.stdout.strip().splitlines()[-1])
                line["plain_decoding"] = {"tokens_per_s": p0["value"], "ms_per_token": p0["ms_per_step"], "draft_len": 0,
                                          "speed_up": line["value"] / p0["value"],
                                          "note": "S = T_ori * m / T_ours (Sec. 4.1) with T_ori from this run"}
            except Exception:
                line["plain_decoding"] = {"error": (r.stderr or r.stdout)[-300:]}
        if world == 1 and args.workload == "medium" and args.draft_len < 0 and not args.no_batched:
            # the small workloads, timed passes only (the Large line, which needs minutes of prefill,
            # is in profiles/workload_lines_and_draft_variants.md with its command)
            line["other_workloads"] = {}
            for wl, st_ in (("tiny", "50"), ("small", "100")):
                r = subprocess.run([sys.executable, os.path.abspath(__file__), "--workload", wl, "--steps", st_, "--warmup", "5",
                                    "--timed-only", "--no-cpu"], capture_output=True, text=True)
                try:
                    line["other_workloads"][wl] = json.loads(r.stdout.strip().splitlines()[-1])
                except Exception:
                    line["other_workloads"][wl] = {"error": (r.stderr or r.stdout)[-300:]}
        if world == 1 and not args.no_cpu:
            line["cpu_baseline"] = cpu_baseline(args.workload, budget_s=args.cpu_seconds)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_full_length(args, cfg, rank, local):
    """The workload as configured: its own prompts, generation to gen_faces faces per sequence (or to
    per-sequence stop lengths), teacher drafts from a plain run on the same kernels.  Reports
    tokens/s over the whole run and the verify-step fraction of the HBM peak in three windows."""
    import torch
    from paper_2511_15618_b200 import FlashMesh
    B, D = cfg.batch, cfg.draft_len
    w = S.make_weights(cfg)
    conds = np.stack([S.make_condition(cfg, b) for b in range(B)])
    prompts = [[int(t) for t in S.make_prompt(cfg, b)] for b in range(B)]
    faces = cfg.gen_faces
    stops = S.stop_lengths(cfg.seed, B, faces).tolist() if args.stop_lengths else [faces] * B
    dev = FlashMesh(cfg, w, device=f"cuda:{local}")
    del w
    stride = 9 * faces
    dev.prefill(conds, prompts)
    dev.set_max_faces(stops)
    plain_tok, plain_len, st_plain = dev.generate(-1, plain=True, stride=stride)
    pt, pl = plain_tok.cpu().numpy(), plain_len.cpu().numpy()
    truth = np.zeros((B, max(len(p) for p in prompts) + stride), dtype=np.int32)
    for b in range(B):
        seq = np.concatenate([np.asarray(prompts[b], np.int32), pt[b, :pl[b]]])
        truth[b, :len(seq)] = seq
    keep = (S.accept_schedule(cfg.seed + rank, B, 4096, D, MEAN_DRAFTS) - 1).astype(np.int32)
    truth_d, keep_d = torch.as_tensor(truth).cuda(), torch.as_tensor(keep).cuda()
    dev.prefill(conds, prompts)
    dev.set_max_faces(stops)
    peak, peak_kind = _peaks()
    est_steps = max(1, int(sum(stops) * 9 / B / (1 + MEAN_DRAFTS)))
    seg = max(20, est_steps // 40)
    out, windows, total_ms, total_tok, total_steps = None, [], 0.0, 0, 0
    for _ in range(100000):
        tok, ln, st = dev.generate(-1, truth=truth_d, keep=keep_d, max_steps=seg, out=out, stride=stride)
        out = (tok, ln)
        total_ms += float(st.ms); total_tok += int(st.emitted); total_steps += int(st.steps)
        cand, _, _ = dev.draft()
        o, _, _ = dev.verify(cand)
        act = (o[:, 0] >= 0).cpu().numpy()
        active = int(act.sum())
        lens = ln.cpu().numpy()
        kv = [[int(1 + len(prompts[b]) + lens[b]), -(-int(1 + len(prompts[b]) + lens[b]) // 3), -(-int(1 + len(prompts[b]) + lens[b]) // 9)]
              for b in range(B) if act[b]]
        ms_step = float(st.ms) / max(1, int(st.steps))
        frac = dev.verify_bytes(kv) / (ms_step * 1e-3) / 1e9 / peak if kv else 0.0
        windows.append((total_steps, ms_step, int(st.emitted), active, frac))
        if active == 0 or int(st.emitted) == 0:
            break
    got, n = tok.cpu().numpy(), ln.cpu().numpy()
    for b in range(B):
        assert n[b] == pl[b] and (got[b, :n[b]] == pt[b, :n[b]]).all(), "speculative output differs from plain decoding"
    line = {"metric": METRIC, "mode": "full_run", "value": total_tok / (total_ms * 1e-3), "unit": "tokens/s", "workload": cfg.name,
            "batch": B, "draft_len": D, "draft_heads": cfg.draft_heads, "n_kv_heads": cfg.n_kv_heads,
            "faces_per_sequence": stops, "steps": total_steps, "emitted": total_tok, "ms_total": total_ms,
            "tokens_per_pass": total_tok / max(1, total_steps),
            "plain_run": {"tokens_per_s": float(pl.sum()) / (st_plain.ms * 1e-3), "ms_per_pass": st_plain.ms / max(1, st_plain.steps)},
            "windows": [{"after_steps": a, "ms_per_step": m, "emitted": e, "active_sequences": act, "verify_step_frac_of_hbm_peak": fr}
                        for a, m, e, act, fr in (windows[0], windows[len(windows) // 2], windows[-2] if len(windows) > 1 else windows[-1])],
            "peak_GBps": peak, "peak_kind": peak_kind}
    print(json.dumps(line), flush=True)


def run_e2e(dev, cfg, truth, keep, prompts, steps):
    """Host-in-the-loop decode through the C ABI's host-buffer call (fm_step_host): per pass the
    host builds the edited candidates from the transcript (it knows L from the previous pass) in
    pinned memory; the call copies them in, runs draft, verify and accept, and copies the accepted
    tokens back before it returns."""
    import torch
    B, D = len(prompts), cfg.draft_len
    L = np.array([1 + len(p) for p in prompts])
    cand_h = torch.full((B, D + 1), -1, dtype=torch.int32).pin_memory()
    nacc_h = torch.zeros((B,), dtype=torch.int32).pin_memory()
    em_h = torch.zeros((B, D + 1), dtype=torch.int32).pin_memory()
    cand_np, nacc_np = cand_h.numpy(), nacc_h.numpy()
    for _ in range(3):                                            # untimed: the call's graphs get captured
        dev.step_host(None, nacc_h, em_h)
        L = L + nacc_np
    tokens = 0
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for s in range(steps):
        for b in range(B):
            n = L[b] - 1
            k = int(keep[s % keep.shape[0], b])
            row = truth[b, n:n + D + 1]
            cand_np[b, :len(row)] = row
            if k < D and k + 1 < len(row):
                cand_np[b, k + 1] = (row[k + 1] + 1) % cfg.n_bins
        dev.step_host(cand_h, nacc_h, em_h)                       # returns after the copies back
        L = L + nacc_np
        tokens += int(nacc_np.sum())
    dt = time.perf_counter() - t0
    return {"tokens": float(tokens), "seconds": dt, "h2d": B * (D + 1) * 4, "d2h": B * (D + 2) * 4}


# -------------------------------------------------------------------------------------------
# the oracle as CPU baseline / reference arm
# -------------------------------------------------------------------------------------------
def _oracle_passes(workload, n_steps, budget_s):
    """Time the oracle, as it stands, on a bounded sample: prefill of the workload's own short
    prompt, then speculative passes with the seeded acceptance schedule (forced lengths)."""
    from oracle.hourglass import OracleSeq
    cfg = S.get_config(workload)
    B, D = cfg.batch, cfg.draft_len
    w = S.make_weights(cfg)
    B_run = min(B, 2)
    sched = S.accept_schedule(cfg.seed, B_run, 4096, D, MEAN_DRAFTS)
    seqs = []
    for b in range(B_run):
        s = OracleSeq(cfg.with_(max_tokens=2048), w)
        s.prefill(S.make_condition(cfg, b), [int(t) for t in S.make_prompt(cfg, b)], max_faces=200)
        seqs.append(s)
    t0 = time.perf_counter()
    tokens = steps = 0
    while steps < n_steps and time.perf_counter() - t0 < budget_s:
        for b, s in enumerate(seqs):
            cand, _, _ = s.draft()
            s.verify(cand)
            a, _, _ = s.accept(force_len=int(sched[steps % 4096, b]))
            tokens += a
        steps += 1
    dt = time.perf_counter() - t0
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count() or 1
    return tokens, steps, dt, cores, B_run


def cpu_baseline(workload, budget_s=20.0):
    tokens, steps, dt, cores, b_run = _oracle_passes(workload, 10 ** 9, budget_s)
    return {"value": tokens / dt, "unit": "tokens/s", "cores": cores, "kind": "oracle",
            "sample": f"{steps} speculative passes of {b_run} sequence(s) right after the prompt (short KV caches), "
                      f"forced acceptance schedule with mean {MEAN_DRAFTS} drafts; numpy float64",
            "ms_per_step": dt / max(1, steps) * 1e3}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    world = int(os.environ.get("WORLD_SIZE", "1"))
    cfg = S.get_config(args.workload)
    for _ in range(1):
        _oracle_passes(args.workload, min(args.warmup, 1), 120.0)          # warm-up (weights cast, BLAS threads)
    tokens, steps, dt, cores, b_run = _oracle_passes(args.workload, args.steps, 150.0)
    value = tokens / dt
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world,
            "steps": steps, "warmup": args.warmup, "ms_per_step": dt / max(1, steps) * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "batch_per_gpu": b_run, "draft_len": cfg.draft_len,
                       "sample": "passes right after the prompt (short KV caches), forced acceptance schedule"},
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                             "sample": f"{steps} passes of {b_run} sequence(s), short KV caches"},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="medium", choices=list(S.CONFIGS))
    ap.add_argument("--start-frac", type=float, default=0.5, help="fraction of the run already in the caches")
    ap.add_argument("--cpu-seconds", type=float, default=20.0)
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-batched", action="store_true", help="skip the batch-16 add-on of the default run")
    ap.add_argument("--timed-only", action="store_true", help="stop after the timed passes (for profiler captures)")
    ap.add_argument("--draft-len", type=int, default=-1, help="override the workload's number of drafts D (0 = plain decoding)")
    ap.add_argument("--draft-heads", default="reduced", choices=["reduced", "full"], help="draft modules: reduced heads or the full SP / HF blocks")
    ap.add_argument("--draft-levels", default="three", choices=["three", "coord"], help="coord: D coordinate heads only (the supplement's ablation)")
    ap.add_argument("--kv-heads", type=int, default=0, help="override n_kv_heads (1 = one shared KV head)")
    ap.add_argument("--full-run", action="store_true", help="decode the workload's whole length from its own prompt; report tokens/s over the run and the verify-step fraction at the start, middle and end")
    ap.add_argument("--stop-lengths", action="store_true", help="with --full-run: per-sequence stop lengths from the face-count split of the paper's data")
    ap.add_argument("--pin-accept", type=int, default=0,
                    help="teacher drafts with the true acceptance pinned to this many tokens per pass (1 .. D+1); 0 = seeded schedule")
    args = ap.parse_args()
    args.warmup = max(3, args.warmup) if args.impl == "ours" else args.warmup
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.gpus > 1 and world == 1 and "RANK" not in os.environ:
        # started plainly with --gpus N: run the N replicas as N ranks, one per GPU
        port = 29500 + os.getpid() % 2000
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        sys.exit(subprocess.run(cmd).returncode)
    if args.gpus != world:
        sys.exit(f"bench.py: --gpus {args.gpus} but WORLD_SIZE is {world}: launch one rank per GPU "
                 f"(python -m torch.distributed.run --nproc-per-node {args.gpus} ... bench.py --gpus {args.gpus})")
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
