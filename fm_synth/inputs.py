"""Seeded conditioning vectors, prompts and acceptance schedules.

These stand in for the paper's evaluation meshes (ShapeNetV2 / gObjaverse test
sets and trained weights are not available): the inputs have the same shape
and structure -- 9 quantised-coordinate tokens per face, vertices ordered
z-y-x, faces sorted, point-cloud conditioning encoded to prefix tokens -- but
are drawn from seeds.
"""
from __future__ import annotations

import itertools

import numpy as np

from .configs import ModelConfig


# ----------------------------------------------------------------------------------------
# conditioning
# ----------------------------------------------------------------------------------------
def _sphere_points(rng, n):
    p = rng.standard_normal((n, 3))
    return p / np.linalg.norm(p, axis=1, keepdims=True)


def _box_points(rng, n, centre, half):
    areas = np.array([half[1] * half[2], half[0] * half[2], half[0] * half[1]]) * 4.0
    axis = rng.choice(3, size=n, p=areas / areas.sum())
    sign = rng.choice([-1.0, 1.0], size=n)
    p = rng.uniform(-1.0, 1.0, size=(n, 3)) * half
    p[np.arange(n), axis] = sign * half[axis]
    return p + centre


def _cylinder_points(rng, n, centre, radius, half_h):
    lateral = 2.0 * np.pi * radius * 2.0 * half_h
    cap = np.pi * radius * radius
    part = rng.choice(3, size=n, p=np.array([lateral, cap, cap]) / (lateral + 2 * cap))
    ang = rng.uniform(0.0, 2.0 * np.pi, size=n)
    r = np.where(part == 0, radius, radius * np.sqrt(rng.uniform(0.0, 1.0, size=n)))
    z = np.where(part == 0, rng.uniform(-half_h, half_h, size=n),
                 np.where(part == 1, half_h, -half_h))
    return np.stack([r * np.cos(ang), r * np.sin(ang), z], axis=1) + centre


def _solids_points(rng, n):
    """Area-weighted samples on 2..5 random boxes and cylinders inside [-1,1]^3."""
    k = int(rng.integers(2, 6))
    solids, areas = [], []
    for _ in range(k):
        centre = rng.uniform(-0.5, 0.5, size=3)
        if rng.random() < 0.5:
            half = rng.uniform(0.1, 0.45, size=3)
            solids.append(("box", centre, half))
            areas.append(8.0 * (half[0] * half[1] + half[1] * half[2] + half[0] * half[2]))
        else:
            radius, half_h = rng.uniform(0.1, 0.45), rng.uniform(0.1, 0.45)
            solids.append(("cyl", centre, radius, half_h))
            areas.append(2 * np.pi * radius * (2 * half_h) + 2 * np.pi * radius ** 2)
    which = rng.choice(k, size=n, p=np.array(areas) / np.sum(areas))
    out = np.zeros((n, 3))
    for i, s in enumerate(solids):
        m = int((which == i).sum())
        if m == 0:
            continue
        pts = _box_points(rng, m, s[1], s[2]) if s[0] == "box" else _cylinder_points(rng, m, s[1], s[2], s[3])
        out[which == i] = pts
    return np.clip(out, -1.0, 1.0)


def make_condition(cfg: ModelConfig, seq: int = 0) -> np.ndarray:
    """Conditioning vectors c[P, d] (float32) for sequence `seq` of the workload."""
    rng = np.random.default_rng([cfg.seed, 1000 + seq])
    P, d = cfg.n_prefix, cfg.d_model
    if cfg.cond_kind == "gauss":
        return rng.standard_normal((P, d)).astype(np.float32)
    n = cfg.cond_points
    assert n == 8 * P, "eight consecutive points make one prefix token"
    pts = _sphere_points(rng, n) if cfg.cond_kind == "sphere" else _solids_points(rng, n)
    # harness-side linear point encoder 24 -> d, entries N(0, 1/24), drawn from the model seed only
    enc_rng = np.random.default_rng([cfg.seed, 999])
    enc = enc_rng.standard_normal((24, d)) / np.sqrt(24.0)
    return (pts.reshape(P, 24) @ enc).astype(np.float32)


# ----------------------------------------------------------------------------------------
# prompts: icosphere mesh -> quantised, sorted token stream
# ----------------------------------------------------------------------------------------
def icosphere_faces(subdiv: int) -> np.ndarray:
    """Triangles [F,3,3] of an icosahedron subdivided `subdiv` times onto the unit sphere."""
    phi = (1.0 + np.sqrt(5.0)) / 2.0
    verts = []
    for a, b in itertools.product((-1.0, 1.0), (-phi, phi)):
        verts += [(0.0, a, b), (a, b, 0.0), (b, 0.0, a)]
    verts = np.array(verts)
    verts /= np.linalg.norm(verts, axis=1, keepdims=True)
    dist = np.linalg.norm(verts[:, None] - verts[None], axis=2)
    edge = np.min(dist[dist > 1e-9])
    tris = [t for t in itertools.combinations(range(12), 3)
            if all(abs(dist[i, j] - edge) < 1e-6 for i, j in itertools.combinations(t, 2))]
    faces = verts[np.array(tris)]                      # [20,3,3]
    for _ in range(subdiv):
        a, b, c = faces[:, 0], faces[:, 1], faces[:, 2]
        ab, bc, ca = (a + b), (b + c), (c + a)
        ab /= np.linalg.norm(ab, axis=1, keepdims=True)
        bc /= np.linalg.norm(bc, axis=1, keepdims=True)
        ca /= np.linalg.norm(ca, axis=1, keepdims=True)
        faces = np.concatenate([np.stack(t, axis=1) for t in
                                ((a, ab, ca), (ab, b, bc), (ca, bc, c), (ab, bc, ca))])
    return faces


def make_prompt(cfg: ModelConfig, seq: int = 0) -> np.ndarray:
    """int32 token ids (9 per face) of the first faces of a rotated, quantised icosphere."""
    rng = np.random.default_rng([cfg.seed, 2000 + seq])
    lo, hi = cfg.prompt_faces
    n_faces = int(rng.integers(lo, hi + 1)) if hi > lo else lo
    if n_faces == 0:
        return np.zeros(0, dtype=np.int32)
    q, r = np.linalg.qr(rng.standard_normal((3, 3)))
    q = q * np.sign(np.diag(r))
    if np.linalg.det(q) < 0:
        q[:, 0] = -q[:, 0]
    faces = icosphere_faces(cfg.prompt_subdiv) @ q.T           # [F,3,(x,y,z)]
    faces = faces / np.max(np.abs(faces))                       # into [-1,1]^3
    ids = np.minimum(cfg.n_bins - 1, np.floor((faces + 1.0) / 2.0 * cfg.n_bins)).astype(np.int64)
    zyx = ids[:, :, ::-1]                                       # vertex token order (z, y, x)
    out = []
    for f in zyx:
        vs = sorted(tuple(int(t) for t in v) for v in f)        # vertices ascending by (z,y,x)
        out.append(tuple(itertools.chain.from_iterable(vs)))
    out.sort()                                                  # faces lexicographic by 9 tokens
    assert n_faces <= len(out)
    return np.array(out[:n_faces], dtype=np.int32).reshape(-1)


def fill_prompt(cfg: ModelConfig, seq: int, n_faces: int) -> list:
    """Seeded mesh tokens standing in for an already generated prefix of `n_faces` faces: the
    sorted faces of a twice-subdivided icosphere, repeated as often as needed."""
    base = make_prompt(cfg.with_(prompt_faces=(320, 320), prompt_subdiv=2), seq)
    reps = -(-n_faces * 9 // len(base))
    return [int(t) for t in np.tile(base, reps)[:9 * n_faces]]


# ----------------------------------------------------------------------------------------
# acceptance schedules and stop lengths (stand-ins for trained draft heads / real meshes)
# ----------------------------------------------------------------------------------------
def accept_schedule(seed: int, batch: int, steps: int, draft_len: int, mean_drafts: float) -> np.ndarray:
    """Accept lengths a[steps, batch] in 1..D+1 with a-1 ~ min(D, Geometric), E[a-1] = mean_drafts."""
    D = draft_len
    if D == 0:
        return np.ones((steps, batch), dtype=np.int32)
    mean_drafts = min(mean_drafts, D - 1e-6)
    lo, hi = 0.0, 1.0 - 1e-12
    for _ in range(200):                     # E[min(D,G)] = sum_{k=1..D} q^k, increasing in q
        q = 0.5 * (lo + hi)
        if sum(q ** k for k in range(1, D + 1)) < mean_drafts:
            lo = q
        else:
            hi = q
    rng = np.random.default_rng([seed, 3000])
    g = rng.geometric(1.0 - q, size=(steps, batch)) - 1
    return (1 + np.minimum(D, g)).astype(np.int32)


def stop_lengths(seed: int, batch: int, cap_faces: int) -> np.ndarray:
    """Faces per sequence from the training-set split 55% <3k, 27% 3k-6k, 18% 6k-10k, clipped."""
    rng = np.random.default_rng([seed, 4000])
    bucket = rng.choice(3, size=batch, p=[0.55, 0.27, 0.18])
    lo = np.array([100, 3000, 6000])[bucket]
    hi = np.array([3000, 6000, 10000])[bucket]
    return np.minimum(cap_faces, rng.integers(lo, hi)).astype(np.int32)
