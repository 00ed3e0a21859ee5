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


# ------------------------------------------------------------------ historical points (R7)
def test_history_window_holds_the_complete_vertices_of_this_face_and_the_one_before():
    from oracle.correct import history_window
    hist = list(range(100))                              # token i has the value i: vertices are (3v, 3v+1, 3v+2)
    # L = 23: main token is t_22, coordinate 1 of vertex 7 (face 2); complete vertices before it: 0..6;
    # the window starts with the previous face (face 1 = vertices 3, 4, 5) and ends with vertex 6
    assert history_window(hist, 23, 1000) == [(9, 10, 11), (12, 13, 14), (15, 16, 17), (18, 19, 20)]
    assert history_window(hist, 1, 1000) == []           # right after BOS nothing is accepted
    assert history_window(hist, 10, 1000) == [(0, 1, 2), (3, 4, 5), (6, 7, 8)]   # main = first token of face 1
    assert history_window([5, 5, 1001, 1, 2, 3], 7, 1000) == [(1, 2, 3)]      # a vertex with a special token is skipped


def test_historical_point_snaps_to_the_nearest_accepted_vertex_hand_worked():
    # accepted: face 0 = (1,1,1) (4,4,4) (9,9,9); the main token opens face 1.  The drafted face has
    # a point labelled historical at (4,5,4): distance 1 to (4,4,4), 27+... to the others -> (4,4,4);
    # a historical point that already equals an accepted vertex stays; a new point is not touched.
    hist = [1, 1, 1, 4, 4, 4, 9, 9, 9]
    cand = [2, 2, 2, 4, 5, 4, 9, 9, 9, 7]               # main token 2, then slots 1.. : (2,2 | ...) see below
    # L = 10: slot 0 is t_9 (first coordinate of vertex 3); slots 1,2 finish that vertex; points start at slots 3 and 6
    labels = [0, 0, 0, H, 0, 0, H, 0, 0, 0]
    out = correct_row(cand, labels, 10, BINS, history=hist)
    assert out == [2, 2, 2, 4, 4, 4, 9, 9, 9, 7]
    assert correct_row(cand, labels, 10, BINS) == cand                         # no history given: not moved
    labels[3] = N
    assert correct_row(cand, labels, 10, BINS, history=hist) == cand


@pytest.mark.parametrize("seed", range(20))
def test_historical_rule_brute_force(seed):
    from oracle.correct import history_window
    rng = np.random.default_rng(100 + seed)
    L = int(rng.integers(1, 60))
    n = int(rng.integers(4, 28))
    hist = rng.integers(0, 6, size=L - 1).tolist()
    cand = rng.integers(0, 6, size=n).tolist()
    labels = rng.choice([H, N], size=n).tolist()          # no intra-batch points: only R7 and the sort act
    out = correct_row(cand, labels, L, BINS, history=hist)
    win = history_window(hist, L, BINS)
    by_face = {}
    for s in draft_points(L, n):
        before = tuple(cand[s:s + 3])
        if labels[s] == H and win and before not in win:
            dmin = min(sum((a - b) ** 2 for a, b in zip(before, c)) for c in win)
            want = next(c for c in win if sum((a - b) ** 2 for a, b in zip(before, c)) == dmin)
        else:
            want = before
        by_face.setdefault((L - 1 + s) // 9, []).append((s, want))
    for f, items in by_face.items():                      # then sorted inside the face
        slots = [s for s, _ in items]
        for s, v in zip(slots, sorted(w for _, w in items)):
            assert tuple(out[s:s + 3]) == v
    assert out[0] == cand[0]
