"""Random-init weights, drawn once from the configuration's seed.

Every matrix is stored `[out, in]` row-major in float32 and holds values that
are exactly representable in bfloat16 (rounded to nearest-even after drawing),
so that neither consumer adds a weight-rounding error of its own.

Draw order (numpy `default_rng(seed)`, `standard_normal(float32) * weight_std`):
  E[V,d];
  for each stack in (coord_down, vertex_down, face, vertex_up, coord_up),
    for each layer: g1[d], Wqkv[(H+2Hkv)*dh, d], Wo[d, H*dh], g2[d], W1[d_ff,d], W2[d,d_ff];
  S_cv[d,3d], S_vf[d,3d], U_fv[3d,d], U_vc[3d,d]; g_out[d], W_out[V,d];
  draft heads: (gain[d], A[d,d]) for coordinate heads 1..Ec; vertex heads 1,2; face heads 1..Ef
  (Ec = ModelConfig.n_coord_heads, Ef = ModelConfig.n_face_heads; no vertex / face heads when
  draft_levels == "coord");
  label head of the correction stage: gain[d], W_lab[3,d];
  with draft_heads == "full", in the same head order (coordinate, vertex, face): per head the
  attention of its SP-Block ga[d], Wq[H*dh,d], Wo[d,H*dh]; then the HF-Blocks, each
  (gain[d], Wq[H*dh,d], W1[hf,H*dh], W2[d,hf]): hf_vc[0..5] (point pipeline, coordinate offsets
  3..8 from the vertex row), hf_fv[0..3Ef-1] (face pipeline, vertex level), hf_fc[0..9Ef-1] (face
  pipeline, coordinate level).
`W_out` alone is scaled by `out_std` when that is set (toy models keep sharp attention with
std-0.1 matrices but logits on the scale of the workloads').
Gains are exactly 1 when `gain_std == 0` (nothing is drawn for them then), else
1 + gain_std * N(0,1) in float32 (gains are not rounded to bfloat16).
"""
from __future__ import annotations

import numpy as np

from .configs import ModelConfig

stack_names = ("coord_down", "vertex_down", "face", "vertex_up", "coord_up")


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); result stays float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    r = (u + bias) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def make_weights(cfg: ModelConfig, seed: int | None = None) -> dict:
    rng = np.random.default_rng(cfg.seed if seed is None else seed)
    d, H, Hkv, dh, dff, V = cfg.d_model, cfg.n_heads, cfg.n_kv_heads, cfg.head_dim, cfg.d_ff, cfg.vocab

    def mat(o, i, std=None):
        w = rng.standard_normal((o, i), dtype=np.float32)
        w *= np.float32(cfg.weight_std if std is None else std)
        return round_to_bf16(w)

    def gain():
        if cfg.gain_std == 0.0:
            return np.ones(d, dtype=np.float32)
        return (1.0 + cfg.gain_std * rng.standard_normal(d, dtype=np.float32)).astype(np.float32)

    w = {"E": mat(V, d), "stacks": []}
    for s in range(5):
        layers = []
        for _ in range(cfg.layers[s]):
            layers.append({
                "g1": gain(),
                "Wqkv": mat((H + 2 * Hkv) * dh, d),
                "Wo": mat(d, H * dh),
                "g2": gain(),
                "W1": mat(dff, d),
                "W2": mat(d, dff),
            })
        w["stacks"].append(layers)
    w["S_cv"] = mat(d, 3 * d)
    w["S_vf"] = mat(d, 3 * d)
    w["U_fv"] = mat(3 * d, d)
    w["U_vc"] = mat(3 * d, d)
    w["g_out"] = gain()
    w["W_out"] = mat(V, d, cfg.out_std if cfg.out_std > 0 else None)
    three = cfg.draft_levels == "three"
    w["heads_c"] = [{"g": gain(), "A": mat(d, d)} for _ in range(cfg.n_coord_heads)]
    w["heads_v"] = [{"g": gain(), "A": mat(d, d)} for _ in range(2 if three else 0)]
    w["heads_f"] = [{"g": gain(), "A": mat(d, d)} for _ in range(cfg.n_face_heads)]
    w["label"] = {"g": gain(), "W": mat(3, d)}
    if cfg.draft_heads == "full":
        hd, hf = H * dh, cfg.hf_width
        for hs in (w["heads_c"], w["heads_v"], w["heads_f"]):
            for h in hs:
                h["ga"], h["Wq"], h["Wo"] = gain(), mat(hd, d), mat(d, hd)

        def hf_block():
            return {"g": gain(), "Wq": mat(hd, d), "W1": mat(hf, hd), "W2": mat(d, hf)}

        w["hf_vc"] = [hf_block() for _ in range(6 if three else 0)]
        w["hf_fv"] = [hf_block() for _ in range(3 * cfg.n_face_heads)]
        w["hf_fc"] = [hf_block() for _ in range(9 * cfg.n_face_heads)]
    return w
