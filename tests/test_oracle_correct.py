"""Pins of the correction-stage oracle (Sec. 3.2): a hand-worked case laid out like the section's
figure, the special cases the section names, and brute-force properties on random rows that are
computed here without the oracle's code."""
import numpy as np
import pytest

from oracle.correct import LABEL_HISTORICAL as H, LABEL_INTRA as I, LABEL_NEW as N, correct_row, draft_points

BINS = 16


def _row(main, verts):
    return [main] + [t for v in verts for t in v]


def test_points_are_the_vertices_made_of_drafts_only():
    # L = 18: the main token is mesh token 17 (last of face 1), slot 1 starts face 2
    assert draft_points(18, 19) == [1, 4, 7, 10, 13, 16]
    # L = 20: main token is mesh token 19 (coordinate 1 of vertex 0 of face 2); the first complete
    # draft vertex starts at mesh token 21 = slot 2; a vertex cut off by the end of the row is no point
    assert draft_points(20, 10) == [2, 5]
    assert draft_points(20, 4) == []
    # right after BOS (L = 1) the main token is mesh token 0: slots 1, 2 finish vertex 0
    assert draft_points(1, 10) == [3, 6]


def test_worked_example_two_displaced_vertices_snap_to_the_vertices_they_share():
    # Like the figure: a first new triangle A B C, then a triangle whose second and third vertex
    # should have been B and C but came out displaced.  F, the new vertex of the second triangle,
    # is nearer to the displaced B' than B is, but lies in the same triangle and must not be used.
    A, B, C = (5, 5, 5), (5, 9, 1), (8, 3, 3)
    F, B2, C2 = (5, 9, 4), (5, 9, 3), (8, 4, 3)
    cand = _row(7, [A, B, C, F, B2, C2])
    labels = [0] * 19
    for s, lab in zip((1, 4, 7, 10, 13, 16), (N, N, N, N, I, I)):
        labels[s] = lab
    out = correct_row(cand, labels, 18, BINS)
    # B' -> B (distance 4; A: 20, C: 49), C' -> C (distance 1), then z-y-x order inside the triangle
    assert out == _row(7, [A, B, C, B, F, C])
    assert out[0] == 7


def test_intra_batch_point_that_overlaps_another_vertex_of_the_batch_stays():
    A, B, C = (1, 1, 1), (2, 2, 2), (3, 3, 3)
    cand = _row(0, [A, B, C, (2, 2, 2), (9, 9, 9), (9, 9, 10)])
    labels = [0] * 19
    for s, lab in zip((1, 4, 7, 10, 13, 16), (N, N, N, I, N, N)):
        labels[s] = lab
    assert correct_row(cand, labels, 18, BINS) == cand


def test_no_candidate_leaves_the_point_and_special_tokens_block_a_vertex():
    # the only new point lies in the same triangle: nothing to duplicate
    cand = _row(3, [(4, 4, 4), (6, 6, 6), (5, 5, 5)])
    labels = [0, N, 0, 0, I, 0, 0, H, 0, 0]
    assert correct_row(cand, labels, 18, BINS) == _row(3, [(4, 4, 4), (5, 5, 5), (6, 6, 6)])    # only the sort acts
    # a vertex holding a non-coordinate token (>= n_bins) is neither corrected, sorted nor copied
    cand = _row(3, [(9, 9, BINS + 1), (6, 6, 6), (5, 5, 5)])
    assert correct_row(cand, labels, 18, BINS) == _row(3, [(9, 9, BINS + 1), (5, 5, 5), (6, 6, 6)])


def test_unaligned_row_keeps_main_token_and_partial_vertices():
    L = 20                                      # slots 0, 1 finish a vertex begun earlier
    cand = [11, 12, 9, 9, 9, 1, 1, 1, 13, 14]   # points at slots 2 and 5 (same face 2: mesh tokens 21..26), tail cut off
    labels = [0] * 10
    labels[2], labels[5] = N, N
    out = correct_row(cand, labels, L, BINS)
    assert out[:2] == [11, 12] and out[8:] == [13, 14]
    assert out[2:8] == [1, 1, 1, 9, 9, 9]       # both in face 2: sorted


@pytest.mark.parametrize("seed", range(40))
def test_random_rows_properties(seed):
    rng = np.random.default_rng(seed)
    D = int(rng.integers(3, 28))
    L = int(rng.integers(1, 60))
    cand = rng.integers(0, 6, size=D + 1).tolist()          # few bins: coincidences are common
    labels = rng.integers(0, 3, size=D + 1).tolist()
    out = correct_row(cand, labels, L, 6)
    starts = [s for s in range(1, D + 1) if (L - 1 + s) % 3 == 0 and s + 2 <= D]
    covered = {s + c for s in starts for c in range(3)}
    # tokens outside complete draft vertices never change (the main token among them)
    assert all(out[i] == cand[i] for i in range(D + 1) if i not in covered)
    vin = {s: tuple(cand[s:s + 3]) for s in starts}
    vout = {s: tuple(out[s:s + 3]) for s in starts}
    face = {s: (L - 1 + s) // 9 for s in starts}
    # corrections only duplicate vertices of the batch
    assert set(vout.values()) <= set(vin.values())
    for f in set(face.values()):
        ss = [s for s in starts if face[s] == f]
        got = [vout[s] for s in ss]
        assert got == sorted(got)                           # z-y-x order inside the face
        # points that are not intra-batch keep their coordinates (they are only permuted in the face)
        keep = sorted(vin[s] for s in ss if labels[s] != I)
        pool = list(got)
        for v in keep:
            assert v in pool
            pool.remove(v)
    if all(labels[s] != I for s in starts):
        assert correct_row(out, labels, L, 6) == out        # nothing left to do


@pytest.mark.parametrize("seed", range(40))
def test_single_intra_point_takes_the_nearest_earlier_new_point_of_another_face(seed):
    rng = np.random.default_rng(1000 + seed)
    L, D = 18, 27                                            # three whole draft faces, 9 points
    verts = rng.integers(0, BINS, size=(9, 3))
    k = int(rng.integers(3, 9))                              # a point of the second or third face
    labels_pt = rng.integers(0, 2, size=9)                   # historical or new
    labels_pt[k] = I
    cand = [0] + verts.reshape(-1).tolist()
    labels = [0] * (D + 1)
    for p in range(9):
        labels[1 + 3 * p] = int(labels_pt[p])
    out = correct_row(cand, labels, L, BINS)
    me = verts[k]
    overlap = any((verts[p] == me).all() for p in range(9) if p != k)
    pool = [p for p in range(k) if labels_pt[p] == N and p // 3 != k // 3]
    expect = verts.copy()
    if not overlap and pool:
        d2 = ((verts[pool] - me) ** 2).sum(axis=1)
        expect[k] = verts[pool[int(np.argmin(d2))]]          # argmin returns the first minimum
    want = []
    for f in range(3):
        want += sorted(tuple(int(t) for t in v) for v in expect[3 * f:3 * f + 3])
    assert out == [0] + [t for v in want for t in v]
