"""ctypes binding of include/flashmesh.h: argument marshalling only.

Module-level functions carry the C names and take raw addresses (ints) for device pointers.
`FlashMesh` is a convenience wrapper that owns the torch workspace tensor and converts
torch tensors / numpy arrays to those addresses; it computes nothing itself.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

FM_MAX_FACE_HEADS = 4
FM_MAX_DRAFT = 27

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None


class FmError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {fm_strerror(code)} ({code})")


class FmConfig(C.Structure):
    _fields_ = [("d_model", C.c_int32), ("n_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("d_ff", C.c_int32), ("layers", C.c_int32 * 5), ("n_bins", C.c_int32), ("n_prefix", C.c_int32),
                ("window", C.c_int32 * 3), ("draft_len", C.c_int32), ("max_batch", C.c_int32),
                ("max_tokens", C.c_int32), ("rope_theta", C.c_float), ("norm_eps", C.c_float),
                ("allow_eos", C.c_int32), ("draft_heads", C.c_int32), ("draft_levels", C.c_int32),
                ("hf_ff", C.c_int32), ("avg_levels", C.c_int32)]


_FP = C.POINTER(C.c_float)


class FmLayerWeights(C.Structure):
    _fields_ = [(n, _FP) for n in ("g1", "Wqkv", "Wo", "g2", "W1", "W2")]


class FmSpWeights(C.Structure):
    _fields_ = [(n, _FP) for n in ("g", "A", "ga", "Wq", "Wo")]


class FmHfWeights(C.Structure):
    _fields_ = [(n, _FP) for n in ("g", "Wq", "W1", "W2")]


class FmWeights(C.Structure):
    _fields_ = [("E", _FP), ("stack", C.POINTER(FmLayerWeights) * 5),
                ("S_cv", _FP), ("S_vf", _FP), ("U_fv", _FP), ("U_vc", _FP), ("g_out", _FP), ("W_out", _FP),
                ("heads_c", C.POINTER(FmSpWeights)), ("heads_v", C.POINTER(FmSpWeights)), ("heads_f", C.POINTER(FmSpWeights)),
                ("hf_vc", C.POINTER(FmHfWeights)), ("hf_fv", C.POINTER(FmHfWeights)), ("hf_fc", C.POINTER(FmHfWeights)),
                ("label_g", _FP), ("label_W", _FP)]


class FmTeacher(C.Structure):
    _fields_ = [("truth", C.c_void_p), ("truth_stride", C.c_int32), ("keep", C.c_void_p), ("n_sched", C.c_int32)]


class FmStats(C.Structure):
    _fields_ = [("steps", C.c_int64), ("emitted", C.c_int64), ("accept_hist", C.c_int64 * (FM_MAX_DRAFT + 2)),
                ("ms", C.c_float)]


class FmProfile(C.Structure):
    _fields_ = [("gemm_ms", C.c_double), ("gemm_bytes", C.c_double), ("gemm_launches", C.c_int64),
                ("attn_ms", C.c_double), ("attn_launches", C.c_int64)]


def library_path() -> str:
    return os.path.join(_HERE, "libflashmesh.so")


def load_library():
    """Load libflashmesh.so (built in-tree by paper_2511_15618_b200.build).  Raises if absent."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = library_path()
    if not os.path.exists(path):
        raise FileNotFoundError(f"{path} is missing: run `python -m paper_2511_15618_b200.build` "
                                "(there is no fallback implementation)")
    lib = C.CDLL(path)
    vp, i32, f32p = C.c_void_p, C.c_int32, C.c_void_p
    lib.fm_workspace_bytes.restype = C.c_size_t
    lib.fm_workspace_bytes.argtypes = [C.POINTER(FmConfig)]
    lib.fm_create.restype = C.c_int
    lib.fm_create.argtypes = [C.POINTER(FmConfig), C.POINTER(FmWeights), vp, C.c_size_t, vp, C.POINTER(vp)]
    lib.fm_destroy.restype = C.c_int
    lib.fm_destroy.argtypes = [vp]
    lib.fm_prefill.restype = C.c_int
    lib.fm_prefill.argtypes = [vp, i32, vp, vp, C.POINTER(C.c_int32)]
    lib.fm_set_max_faces.restype = C.c_int
    lib.fm_set_max_faces.argtypes = [vp, C.POINTER(C.c_int32)]
    lib.fm_draft.restype = C.c_int
    lib.fm_draft.argtypes = [vp, vp, f32p, f32p]
    lib.fm_correct.restype = C.c_int
    lib.fm_correct.argtypes = [vp, vp, vp]
    lib.fm_draft_labels.restype = C.c_int
    lib.fm_draft_labels.argtypes = [vp, vp, f32p]
    lib.fm_correct_ex.restype = C.c_int
    lib.fm_correct_ex.argtypes = [vp, vp, vp, i32]
    lib.fm_verify.restype = C.c_int
    lib.fm_verify.argtypes = [vp, vp, vp, f32p, f32p]
    lib.fm_verify_static_scratch.restype = C.c_int
    lib.fm_verify_static_scratch.argtypes = [vp, vp, vp, f32p, f32p]
    lib.fm_step_host.restype = C.c_int
    lib.fm_step_host.argtypes = [vp, vp, vp, vp, vp]
    lib.fm_accept.restype = C.c_int
    lib.fm_accept.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.fm_generate.restype = C.c_int
    lib.fm_generate.argtypes = [vp, i32, vp, i32, vp, C.POINTER(FmTeacher), i32, C.c_int64, C.POINTER(FmStats)]
    lib.fm_verify_bytes.restype = C.c_double
    lib.fm_verify_bytes.argtypes = [vp, i32, C.POINTER(C.c_int32)]
    lib.fm_profile_begin.restype = C.c_int
    lib.fm_profile_begin.argtypes = [vp]
    lib.fm_profile_end.restype = C.c_int
    lib.fm_profile_end.argtypes = [vp, C.POINTER(FmProfile)]
    lib.fm_profile_class.restype = C.c_int
    lib.fm_profile_class.argtypes = [vp, i32, i32, C.POINTER(FmProfile)]
    lib.fm_attention_layout.restype = C.c_int
    lib.fm_attention_layout.argtypes = [vp, i32, C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    lib.fm_launch_count.restype = C.c_int64
    lib.fm_launch_count.argtypes = [vp]
    lib.fm_selftest_wait_timeout.restype = C.c_int
    lib.fm_selftest_wait_timeout.argtypes = [vp, C.c_int64]
    lib.fm_strerror.restype = C.c_char_p
    lib.fm_strerror.argtypes = [C.c_int]
    lib.fm_device_status.restype = C.c_int
    lib.fm_device_status.argtypes = [vp]
    _LIB = lib
    return lib


# ------------------------------------------------------------------ C-named thin functions
def fm_strerror(code: int) -> str:
    return load_library().fm_strerror(int(code)).decode()


def fm_workspace_bytes(cfg: FmConfig) -> int:
    return int(load_library().fm_workspace_bytes(C.byref(cfg)))


def fm_create(cfg: FmConfig, weights: FmWeights, dev_workspace: int, nbytes: int, stream: int):
    ctx = C.c_void_p()
    rc = load_library().fm_create(C.byref(cfg), C.byref(weights), dev_workspace, nbytes, stream, C.byref(ctx))
    return rc, ctx


def fm_destroy(ctx):
    return load_library().fm_destroy(ctx)


def _i32_array(values):
    arr = (C.c_int32 * len(values))(*[int(v) for v in values])
    return arr


def fm_prefill(ctx, batch, cond_ptr, prompt_ptr, prompt_off):
    return load_library().fm_prefill(ctx, batch, cond_ptr, prompt_ptr, _i32_array(prompt_off))


def fm_set_max_faces(ctx, max_faces):
    return load_library().fm_set_max_faces(ctx, _i32_array(max_faces))


def fm_draft(ctx, cand_ptr, draft_logits_ptr=None, draft_margin_ptr=None):
    return load_library().fm_draft(ctx, cand_ptr, draft_logits_ptr, draft_margin_ptr)


def fm_correct(ctx, cand_ptr, labels_ptr):
    return load_library().fm_correct(ctx, cand_ptr, labels_ptr)


def fm_draft_labels(ctx, labels_ptr, margin_ptr=None):
    return load_library().fm_draft_labels(ctx, labels_ptr, margin_ptr)


def fm_correct_ex(ctx, cand_ptr, labels_ptr=None, use_history=0):
    return load_library().fm_correct_ex(ctx, cand_ptr, labels_ptr, int(use_history))


def fm_verify(ctx, cand_ptr, argmax_ptr=None, logits_ptr=None, margin_ptr=None):
    return load_library().fm_verify(ctx, cand_ptr, argmax_ptr, logits_ptr, margin_ptr)


def fm_verify_static_scratch(ctx, cand_ptr, argmax_ptr=None, logits_ptr=None, margin_ptr=None):
    """fm_verify with the attention kernel's scratch in the library's own fixed array: for hosts
    that may not allocate device memory for it (see include/flashmesh.h)."""
    return load_library().fm_verify_static_scratch(ctx, cand_ptr, argmax_ptr, logits_ptr, margin_ptr)


def fm_step_host(ctx, cand_host_ptr, n_acc_host_ptr, emitted_host_ptr=None, kv_len_host_ptr=None):
    """One pass with host buffers (addresses of host memory; see include/flashmesh.h)."""
    return load_library().fm_step_host(ctx, cand_host_ptr, n_acc_host_ptr, emitted_host_ptr, kv_len_host_ptr)


def fm_accept(ctx, force_len_ptr=None, force_tok_ptr=None, n_acc_ptr=None, emitted_ptr=None, kv_len_ptr=None):
    return load_library().fm_accept(ctx, force_len_ptr, force_tok_ptr, n_acc_ptr, emitted_ptr, kv_len_ptr)


def fm_generate(ctx, max_faces, out_tok_ptr, out_stride, out_len_ptr, teacher=None, plain=0, max_steps=0, stats=None):
    t = C.byref(teacher) if teacher is not None else None
    s = C.byref(stats) if stats is not None else None
    return load_library().fm_generate(ctx, max_faces, out_tok_ptr, out_stride, out_len_ptr, t, plain, max_steps, s)


def fm_verify_bytes(ctx, batch, kv_len):
    flat = [int(v) for row in kv_len for v in row]
    return float(load_library().fm_verify_bytes(ctx, batch, _i32_array(flat)))


def fm_profile_begin(ctx):
    return load_library().fm_profile_begin(ctx)


def fm_profile_end(ctx):
    p = FmProfile()
    rc = load_library().fm_profile_end(ctx, C.byref(p))
    return rc, p


def fm_profile_class(ctx, cls, reps):
    p = FmProfile()
    rc = load_library().fm_profile_class(ctx, int(cls), int(reps), C.byref(p))
    return rc, p


def fm_attention_layout(ctx, level):
    """(slots per chunk, chunks per group, groups of the full cache) of a level's attention."""
    a, b, c = C.c_int32(), C.c_int32(), C.c_int32()
    rc = load_library().fm_attention_layout(ctx, int(level), C.byref(a), C.byref(b), C.byref(c))
    return rc, (a.value, b.value, c.value)


def fm_launch_count(ctx):
    return int(load_library().fm_launch_count(ctx))


def fm_selftest_wait_timeout(ctx, limit_cycles):
    return int(load_library().fm_selftest_wait_timeout(ctx, int(limit_cycles)))


def fm_device_status(ctx):
    return int(load_library().fm_device_status(ctx))


# ------------------------------------------------------------------ convenience wrapper
def make_config(mc, max_batch=None, max_tokens=None, draft_len=None) -> FmConfig:
    """FmConfig from an object with the fields of fm_synth.ModelConfig."""
    cfg = FmConfig()
    cfg.d_model, cfg.n_heads, cfg.n_kv_heads, cfg.head_dim, cfg.d_ff = (mc.d_model, mc.n_heads, mc.n_kv_heads,
                                                                         mc.head_dim, mc.d_ff)
    cfg.layers = (C.c_int32 * 5)(*mc.layers)
    cfg.n_bins, cfg.n_prefix = mc.n_bins, mc.n_prefix
    cfg.window = (C.c_int32 * 3)(*mc.window)
    cfg.draft_len = mc.draft_len if draft_len is None else draft_len
    cfg.max_batch = mc.max_batch if max_batch is None else max_batch
    cfg.max_tokens = mc.max_tokens if max_tokens is None else max_tokens
    cfg.rope_theta, cfg.norm_eps, cfg.allow_eos = mc.rope_theta, mc.norm_eps, mc.allow_eos
    cfg.draft_heads = 1 if getattr(mc, "draft_heads", "reduced") == "full" else 0
    cfg.draft_levels = 1 if getattr(mc, "draft_levels", "three") == "coord" else 0
    cfg.hf_ff = int(getattr(mc, "hf_ff", 0))
    cfg.avg_levels = int(getattr(mc, "avg_levels", 0))
    return cfg


def _fp(a):
    assert a.dtype == np.float32 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(_FP)


def make_weights(w: dict):
    """FmWeights pointing into the float32 numpy arrays of `w` (which must stay alive)."""
    fw = FmWeights()
    keep = []
    fw.E = _fp(w["E"])
    for s in range(5):
        arr = (FmLayerWeights * max(1, len(w["stacks"][s])))()
        for l, lw in enumerate(w["stacks"][s]):
            for name in ("g1", "Wqkv", "Wo", "g2", "W1", "W2"):
                setattr(arr[l], name, _fp(lw[name]))
        keep.append(arr)
        fw.stack[s] = C.cast(arr, C.POINTER(FmLayerWeights))
    for name in ("S_cv", "S_vf", "U_fv", "U_vc", "g_out", "W_out"):
        setattr(fw, name, _fp(w[name]))

    def block_array(kind, fields, blocks):
        arr = (kind * max(1, len(blocks)))()
        for i, blk in enumerate(blocks):
            for name in fields:
                if name in blk:
                    setattr(arr[i], name, _fp(blk[name]))
        keep.append(arr)
        return C.cast(arr, C.POINTER(kind))

    for name in ("heads_c", "heads_v", "heads_f"):
        setattr(fw, name, block_array(FmSpWeights, ("g", "A", "ga", "Wq", "Wo"), w.get(name, [])))
    for name in ("hf_vc", "hf_fv", "hf_fc"):
        setattr(fw, name, block_array(FmHfWeights, ("g", "Wq", "W1", "W2"), w.get(name, [])))
    if "label" in w:
        fw.label_g, fw.label_W = _fp(w["label"]["g"]), _fp(w["label"]["W"])
    return fw, keep


class FlashMesh:
    """Owns a context and its torch workspace; every method forwards to the C entry point of
    the same name.  Tensors returned are freshly allocated torch CUDA tensors."""

    def __init__(self, model_cfg, weights: dict, device="cuda:0", stream=None, **cfg_overrides):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("FlashMesh needs a CUDA device; there is no CPU path")
        load_library()
        self.torch = torch
        self.device = torch.device(device)
        self.mc = model_cfg
        self.cfg = make_config(model_cfg, **cfg_overrides)
        self.D = int(self.cfg.draft_len)
        self.V = int(self.cfg.n_bins) + 3
        nbytes = fm_workspace_bytes(self.cfg)
        if nbytes == 0:
            raise FmError(-1, "fm_workspace_bytes")
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
            base = (self.workspace.data_ptr() + 255) // 256 * 256
            # a stream of its own: the legacy default stream cannot be captured into a CUDA graph
            self.stream = stream if stream is not None else torch.cuda.Stream(self.device)
            fw, self._keep = make_weights(weights)
            rc, self.ctx = fm_create(self.cfg, fw, base, nbytes, self.stream.cuda_stream)
        if rc != 0:
            raise FmError(rc, "fm_create")
        self.workspace_bytes = nbytes
        self.batch = 0

    def close(self):
        if getattr(self, "ctx", None) is not None:
            fm_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc, where):
        if rc != 0:
            raise FmError(rc, where)

    def _before(self):
        """Order the context's stream after the caller's current stream (inputs are ready)."""
        self.stream.wait_stream(self.torch.cuda.current_stream(self.device))

    def _after(self, *tensors):
        """Order the caller's current stream after the context's stream (outputs are ready)."""
        cur = self.torch.cuda.current_stream(self.device)
        cur.wait_stream(self.stream)
        for t in tensors:
            if t is not None:
                t.record_stream(self.stream)

    def _dev(self, x, dtype):
        t = self.torch
        if isinstance(x, t.Tensor):
            assert x.is_cuda and x.dtype == dtype and x.is_contiguous()
            return x
        return t.as_tensor(np.ascontiguousarray(x), dtype=dtype).to(self.device)

    def _empty(self, shape, dtype):
        return self.torch.empty(shape, dtype=dtype, device=self.device)

    def _out(self, name, shape, dtype, reuse):
        """An output buffer: a fresh one, or with `reuse` the same one on every call (the library
        replays a call whose pointers repeat as one CUDA graph; the next call overwrites it)."""
        if not reuse:
            return self._empty(shape, dtype)
        key = (name, tuple(shape), dtype)
        if not hasattr(self, "_held"):
            self._held = {}
        if key not in self._held:
            self._held[key] = self._empty(shape, dtype)
        return self._held[key]

    def prefill(self, cond, prompts):
        """cond: [B,P,d] float32 (tensor or array); prompts: list of int sequences."""
        t = self.torch
        B = len(prompts)
        off = [0]
        for p in prompts:
            off.append(off[-1] + len(p))
        flat = np.concatenate([np.asarray(p, dtype=np.int32) for p in prompts] + [np.zeros(1, np.int32)])
        self._cond = self._dev(cond, t.float32)
        self._prompt = self._dev(flat, t.int32)
        self._before()
        self._check(fm_prefill(self.ctx, B, self._cond.data_ptr(), self._prompt.data_ptr(), off), "fm_prefill")
        self._after()
        self.batch = B

    def set_max_faces(self, max_faces):
        self._before()
        self._check(fm_set_max_faces(self.ctx, list(max_faces)), "fm_set_max_faces")
        self._after()

    def draft(self, want_logits=False, reuse=False):
        t = self.torch
        B, D = self.batch, self.D
        cand = self._out("cand", (B, D + 1), t.int32, reuse)
        dl = self._out("dl", (B, D, self.V), t.float32, reuse) if want_logits else None
        dm = self._empty((B, max(D, 1)), t.float32)[:, :D].contiguous() if want_logits else None
        self._before()
        self._check(fm_draft(self.ctx, cand.data_ptr(), dl.data_ptr() if dl is not None else None,
                             dm.data_ptr() if dm is not None and D > 0 else None), "fm_draft")
        self._after(cand, dl, dm)
        return cand, dl, dm

    def correct(self, cand, labels=None, use_history=False):
        """Edit the drafts of `cand` (int32 [B, D+1], device) in place with the per-point labels
        (int32 [B, D+1], device; None = the label head's of the last draft); returns `cand`."""
        self._before()
        if labels is not None and not use_history:
            self._check(fm_correct(self.ctx, cand.data_ptr(), labels.data_ptr()), "fm_correct")
        else:
            self._check(fm_correct_ex(self.ctx, cand.data_ptr(), labels.data_ptr() if labels is not None else None,
                                      1 if use_history else 0), "fm_correct_ex")
        self._after(cand, labels)
        return cand

    def draft_labels(self):
        """Labels [B, D+1] int32 and margins [B, D+1] float32 of the last draft (device tensors)."""
        t = self.torch
        lab = self._empty((self.batch, self.D + 1), t.int32)
        mg = self._empty((self.batch, self.D + 1), t.float32)
        self._before()
        self._check(fm_draft_labels(self.ctx, lab.data_ptr(), mg.data_ptr()), "fm_draft_labels")
        self._after(lab, mg)
        return lab, mg

    def verify(self, cand, want_logits=False, reuse=False):
        t = self.torch
        B, D = self.batch, self.D
        cand = self._dev(cand, t.int32)
        o = self._out("o", (B, D + 1), t.int32, reuse)
        mg = self._out("mg", (B, D + 1), t.float32, reuse)
        lg = self._out("lg", (B, D + 1, self.V), t.float32, reuse) if want_logits else None
        self._before()
        self._check(fm_verify(self.ctx, cand.data_ptr(), o.data_ptr(), lg.data_ptr() if lg is not None else None,
                              mg.data_ptr()), "fm_verify")
        self._after(cand, o, lg, mg)
        return o, lg, mg

    def accept(self, force_len=None, force_tok=None, reuse=False):
        t = self.torch
        B, D = self.batch, self.D
        fl = self._dev(force_len, t.int32) if force_len is not None else None
        ft = self._dev(force_tok, t.int32) if force_tok is not None else None
        n_acc = self._out("n_acc", (B,), t.int32, reuse)
        em = self._out("em", (B, D + 1), t.int32, reuse)
        kv = self._out("kv", (B, 3), t.int32, reuse)
        self._before()
        self._check(fm_accept(self.ctx, fl.data_ptr() if fl is not None else None,
                              ft.data_ptr() if ft is not None else None, n_acc.data_ptr(), em.data_ptr(),
                              kv.data_ptr()), "fm_accept")
        self._after(fl, ft, n_acc, em, kv)
        return n_acc, em, kv

    def step_host(self, cand_h, n_acc_h, emitted_h=None, kv_len_h=None):
        """One pass through fm_step_host; the arguments are host tensors (pinned for asynchronous
        copies), int32: cand_h [B, D+1] or None, n_acc_h [B], emitted_h [B, D+1], kv_len_h [B, 3]."""
        self._before()
        ptr = lambda x: x.data_ptr() if x is not None else None
        self._check(fm_step_host(self.ctx, ptr(cand_h), ptr(n_acc_h), ptr(emitted_h), ptr(kv_len_h)), "fm_step_host")

    def generate(self, max_faces, truth=None, keep=None, plain=False, out=None, max_steps=0, stride=None):
        """Run the decode loop; returns (tokens [B, 9*max_faces] int32, lengths [B], FmStats).
        `out` = (tokens, lengths) of an earlier call continues appending to them.  max_faces = -1
        keeps the limits of set_max_faces (give `stride`, the row length of the token buffer)."""
        t = self.torch
        B = self.batch
        stride = 9 * max_faces if stride is None else int(stride)
        out_tok = out[0] if out is not None else self.torch.full((B, max(stride, 1)), -1, dtype=t.int32, device=self.device)
        out_len = out[1] if out is not None else self._empty((B,), t.int32)
        teacher = None
        if truth is not None:
            self._truth = self._dev(truth, t.int32)
            self._keep_sched = self._dev(keep, t.int32) if keep is not None else None
            teacher = FmTeacher()
            teacher.truth = self._truth.data_ptr()
            teacher.truth_stride = int(self._truth.shape[1])
            teacher.keep = self._keep_sched.data_ptr() if self._keep_sched is not None else None
            teacher.n_sched = int(self._keep_sched.shape[0]) if self._keep_sched is not None else 0
        stats = FmStats()
        self._before()
        self._check(fm_generate(self.ctx, max_faces, out_tok.data_ptr(), stride, out_len.data_ptr(), teacher,
                                1 if plain else 0, max_steps, stats), "fm_generate")
        self._after(out_tok, out_len)
        return out_tok, out_len, stats

    def verify_bytes(self, kv_len):
        return fm_verify_bytes(self.ctx, len(kv_len), kv_len)

    def profile_begin(self):
        self._check(fm_profile_begin(self.ctx), "fm_profile_begin")

    def profile_end(self):
        rc, p = fm_profile_end(self.ctx)
        self._check(rc, "fm_profile_end")
        return p

    def profile_class(self, cls, reps=20):
        """Milliseconds and launches per verify pass of one kernel class timed alone (0 GEMM, 1 attention)."""
        self._before()
        rc, p = fm_profile_class(self.ctx, cls, reps)
        self._check(rc, "fm_profile_class")
        self._after()
        return (p.gemm_ms, p.gemm_launches, p.gemm_bytes) if cls == 0 else (p.attn_ms, p.attn_launches, 0.0)

    def launch_count(self):
        return fm_launch_count(self.ctx)

    def device_status(self):
        return fm_device_status(self.ctx)
