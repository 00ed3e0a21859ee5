"""Model / workload configurations (the five benchmark workloads plus toys).

Stack order everywhere: coord_down, vertex_down, face, vertex_up, coord_up.
Levels: 0 = coordinate, 1 = vertex (3 coordinates), 2 = face (9 coordinates).
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Tuple

STACK_LEVEL = (0, 1, 2, 1, 0)          # level of each of the five stacks
LEVEL_RATIO = (1, 3, 9)                # coordinate positions per level position


@dataclass(frozen=True)
class ModelConfig:
    name: str
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    d_ff: int
    layers: Tuple[int, int, int, int, int]
    n_bins: int
    n_prefix: int
    window: Tuple[int, int, int]        # per level, 0 = full attention
    draft_len: int                      # D
    max_batch: int
    max_tokens: int                     # capacity per sequence, coordinate positions
    rope_theta: float = 10000.0         # 0 = no positional encoding
    norm_eps: float = 1e-5
    allow_eos: int = 0
    # --- workload recipe (not part of the model) ---
    seed: int = 0
    batch: int = 1
    gen_faces: int = 32                 # faces generated after the prompt
    prompt_faces: Tuple[int, int] = (0, 0)   # inclusive range of prompt faces per sequence
    prompt_subdiv: int = 1              # icosphere subdivisions for the prompt mesh
    cond_kind: str = "gauss"            # gauss | sphere | solids
    cond_points: int = 0
    weight_std: float = 0.02
    out_std: float = 0.0                # std of the output matrix W_out; 0 => weight_std
    # --- draft modules ---
    draft_heads: str = "reduced"        # "reduced": SP = h + A rms(h), HF = the backbone's upsample matrices;
                                        # "full": SP-Block with attention, HF-Blocks after every upsample
    draft_levels: str = "three"         # "three": coordinate + point + face level; "coord": D coordinate heads only
    hf_ff: int = 0                      # hidden width of the HF-Blocks' feed-forward networks; 0 => d_model
    avg_levels: int = 0                 # 1: average the levels' distributions where several predict a position
    gain_std: float = 0.0               # 0 => RMSNorm gains exactly 1

    @property
    def vocab(self) -> int:
        return self.n_bins + 3

    @property
    def bos(self) -> int:
        return self.n_bins

    @property
    def eos(self) -> int:
        return self.n_bins + 1

    @property
    def pad(self) -> int:
        return self.n_bins + 2

    @property
    def n_coord_heads(self) -> int:
        return 2 if self.draft_levels == "three" else self.draft_len

    @property
    def hf_width(self) -> int:
        return self.hf_ff if self.hf_ff > 0 else self.d_model

    @property
    def n_face_heads(self) -> int:
        # face head e drafts the face e - 1 after the one that holds the pending token; a draft
        # can reach face (8 + D) // 9 after it, and only offsets >= 7 ever leave the next two points
        if self.draft_levels != "three":
            return 0
        return 1 if self.draft_len < 7 else (self.draft_len + 8) // 9 + 1

    def with_(self, **kw) -> "ModelConfig":
        return replace(self, **kw)


def _cap(prompt_faces_max: int, gen_faces: int, draft_len: int) -> int:
    # inputs consumed at the end = 1 + 9*(prompt+gen); the verify step writes up to D rows beyond
    return 1 + 9 * (prompt_faces_max + gen_faces) + draft_len + 1


CONFIGS = {
    # d 256, 4 heads of 64, layers 1/1/2/1/1, 128 bins, 64 Gaussian prefix tokens, D=3, 32 faces
    "tiny": ModelConfig(
        name="tiny", d_model=256, n_heads=4, n_kv_heads=4, head_dim=64, d_ff=1024,
        layers=(1, 1, 2, 1, 1), n_bins=128, n_prefix=64, window=(0, 0, 0), draft_len=3,
        max_batch=1, max_tokens=_cap(0, 32, 3), seed=0, batch=1, gen_faces=32,
        prompt_faces=(0, 0), cond_kind="gauss"),
    # d 512, 8 heads, 2/2/8/2/2, 1024 bins, sphere point cloud -> 256 prefix tokens, 8-face prompt, D=9
    "small": ModelConfig(
        name="small", d_model=512, n_heads=8, n_kv_heads=8, head_dim=64, d_ff=2048,
        layers=(2, 2, 8, 2, 2), n_bins=1024, n_prefix=256, window=(0, 0, 0), draft_len=9,
        max_batch=1, max_tokens=_cap(8, 256, 9), seed=1, batch=1, gen_faces=256,
        prompt_faces=(8, 8), prompt_subdiv=1, cond_kind="sphere", cond_points=2048),
    # d 1024, 16 heads, 4/4/16/4/4, window 8192 at the coordinate level, 512 prefix tokens, D=9
    "medium": ModelConfig(
        name="medium", d_model=1024, n_heads=16, n_kv_heads=16, head_dim=64, d_ff=4096,
        layers=(4, 4, 16, 4, 4), n_bins=1024, n_prefix=512, window=(8192, 0, 0), draft_len=9,
        max_batch=1, max_tokens=_cap(8, 4000, 9), seed=2, batch=1, gen_faces=4000,
        prompt_faces=(8, 8), prompt_subdiv=1, cond_kind="solids", cond_points=4096),
    # the medium model at batch 16, ragged prompts of 8..64 faces, per-sequence acceptance
    "batched": ModelConfig(
        name="batched", d_model=1024, n_heads=16, n_kv_heads=16, head_dim=64, d_ff=4096,
        layers=(4, 4, 16, 4, 4), n_bins=1024, n_prefix=512, window=(8192, 0, 0), draft_len=9,
        max_batch=16, max_tokens=_cap(64, 4000, 9), seed=2, batch=16, gen_faces=4000,
        prompt_faces=(8, 64), prompt_subdiv=2, cond_kind="solids", cond_points=4096),
    # d 2048, 16 heads of 128, 4/4/24/4/4, window 8192 coordinate, full vertex/face, B=4, D=12
    "large": ModelConfig(
        name="large", d_model=2048, n_heads=16, n_kv_heads=16, head_dim=128, d_ff=8192,
        layers=(4, 4, 24, 4, 4), n_bins=1024, n_prefix=512, window=(8192, 0, 0), draft_len=12,
        max_batch=4, max_tokens=_cap(8, 16000, 12), seed=4, batch=4, gen_faces=16000,
        prompt_faces=(8, 8), prompt_subdiv=1, cond_kind="solids", cond_points=4096),
}


def get_config(name: str, **overrides) -> ModelConfig:
    cfg = CONFIGS[name]
    return replace(cfg, **overrides) if overrides else cfg


def toy_config(**kw) -> ModelConfig:
    """A d=64 model small enough for brute-force checks (one layer per stack by default)."""
    base = dict(
        name="toy", d_model=64, n_heads=2, n_kv_heads=2, head_dim=32, d_ff=256,
        layers=(1, 1, 1, 1, 1), n_bins=16, n_prefix=4, window=(0, 0, 0), draft_len=3,
        max_batch=2, max_tokens=_cap(4, 8, 12), seed=7, batch=1, gen_faces=4,
        prompt_faces=(0, 0), cond_kind="gauss", weight_std=0.2, gain_std=0.1)
    base.update(kw)
    return ModelConfig(**base)
