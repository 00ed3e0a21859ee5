"""CPU oracle of the correction stage that sits between drafting and verifying.

THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  Only the test-suite may import it.  It shares no
code with the CUDA library and is deliberately plain: Python loops over a handful of vertices.

What it follows (FlashMesh, arXiv 2511.15618, Sec. 3.2 "Correction Mechanism"):
  * every generated point carries one of three labels: historical (coincides with a vertex of an
    earlier batch), new (a novel position), intra-batch (duplicates a new point generated earlier
    in the same batch);
  * for each intra-batch point: look for an overlap with another vertex of the same batch; if
    there is none, duplicate the nearest new point outside the current triangle;
  * finally the vertices are sorted again along z-y-x;
  * only draft tokens are touched, never the main token.

The label head itself (a linear layer on point features) is part of the draft modules
(oracle/hourglass.py, OracleSeq.draft_labels); labels are inputs here.

Readings taken where the section is silent:
  R1  a "point" of a candidate row is a vertex whose three coordinate tokens (z, y, x) are all
      drafts of this pass; vertices that contain the main token or already accepted tokens, or
      that are cut off by the end of the row, are left alone.  A vertex with a token that is not a
      coordinate bin (BOS / EOS / PAD) is left alone and is nobody's candidate.
  R2  "the batch" is the set of such points of one sequence in one pass; "the current triangle"
      is the face the point belongs to.
  R3  intra-batch points are handled in sequence order, each seeing the corrections made before it.
  R4  "overlap": another point of the batch (any label) with the same three tokens.
  R5  candidates for duplication: points labelled new that come earlier in the batch (the label's
      own definition) and belong to another face; distance is squared Euclidean distance between
      the bin indices; ties go to the earliest candidate; with no candidate the point stays.
  R6  re-sorting: inside each face, the points of the batch are sorted ascending by (z, y, x)
      among the slots they occupy (accepted vertices of the same face cannot move); faces are not
      reordered.
  R7  historical points: the section defines the label (the point coincides with a vertex
      generated before this batch) and gives no operation.  Without a history they are not moved.
      With the accepted tokens given, the label is enforced the way the intra-batch rule enforces
      its own: a historical point that equals no vertex of the history window is replaced by the
      nearest vertex of the window (same distance, ties to the earliest).  The window holds the
      complete accepted vertices of the face that contains the main token and of the face before
      it (a shared vertex of a sorted mesh lies in a neighbouring face); the vertex that contains
      the main token is not complete and is not in it.  Historical points are handled first, in
      sequence order.

Pins (tests/test_oracle_correct.py): a hand-worked case built like the section's figure (two
displaced vertices snap to the vertices they should share, then the face is re-sorted); brute-force
properties on random inputs, written independently of this file (untouched main token and partial
vertices, nearest-candidate optimality, sortedness, idempotence when nothing is labelled
intra-batch, label/new points only permuted inside their face).
"""
from __future__ import annotations

LABEL_HISTORICAL = 0
LABEL_NEW = 1
LABEL_INTRA = 2


def draft_points(L: int, n_cand: int):
    """Slots (indices into the candidate row) at which a complete draft vertex starts.

    The candidate row holds the mesh tokens with indices L-1 (the main token, slot 0) to
    L-1+n_cand-1; mesh token j is coordinate j % 3 of vertex (j % 9) // 3 of face j // 9 (R1)."""
    out = []
    for s in range(1, n_cand):                   # slot 0 is the main token
        j = L - 1 + s
        if j % 3 == 0 and s + 2 < n_cand:
            out.append(s)
    return out


def history_window(history, L: int, n_bins: int):
    """Complete accepted vertices (z, y, x) of the face that holds the main token t_{L-1} and of
    the face before it, oldest first (R7).  history[i] = mesh token t_i for i < L - 1."""
    first = max(0, 3 * ((L - 1) // 9 - 1))           # first vertex of the previous face
    out = []
    for v in range(first, (L - 1) // 3):             # vertices whose three tokens precede the main token
        c = tuple(int(history[3 * v + k]) for k in range(3))
        if all(0 <= t < n_bins for t in c):
            out.append(c)
    return out


def correct_row(cand, labels, L: int, n_bins: int, history=None):
    """Corrected copy of one sequence's candidate row.

    cand: D+1 token ids (main token first); labels: D+1 ints, labels[s] is the label of the
    vertex that starts at slot s (read only at the slots `draft_points` returns); history:
    optional accepted mesh tokens t_0 .. t_{L-2} (R7)."""
    cand = [int(t) for t in cand]
    n = len(cand)
    starts = draft_points(L, n)
    pts = []                                     # [slot, face, label, usable]
    for s in starts:
        j = L - 1 + s
        ok = all(0 <= cand[s + c] < n_bins for c in range(3))
        pts.append([s, j // 9, int(labels[s]), ok])

    def coords(s):
        return (cand[s], cand[s + 1], cand[s + 2])

    # historical points against the accepted vertices (R7)
    if history is not None:
        window = history_window(history, L, n_bins)
        for s, face, lab, ok in pts:
            if lab != LABEL_HISTORICAL or not ok or not window:
                continue
            me = coords(s)
            if me in window:
                continue
            dist = [sum((a - b) * (a - b) for a, b in zip(me, c)) for c in window]
            cand[s:s + 3] = list(window[dist.index(min(dist))])

    # intra-batch points, in order (R3)
    for k, (s, face, lab, ok) in enumerate(pts):
        if lab != LABEL_INTRA or not ok:
            continue
        me = coords(s)
        if any(k2 != k and pts[k2][3] and coords(pts[k2][0]) == me for k2 in range(len(pts))):
            continue                             # overlaps another vertex of the batch (R4)
        best, best_d = -1, None
        for k2 in range(k):                      # new points generated earlier, outside this triangle (R5)
            s2, face2, lab2, ok2 = pts[k2]
            if lab2 != LABEL_NEW or not ok2 or face2 == face:
                continue
            c2 = coords(s2)
            d2 = sum((a - b) * (a - b) for a, b in zip(me, c2))
            if best_d is None or d2 < best_d:
                best, best_d = k2, d2
        if best >= 0:
            s2 = pts[best][0]
            cand[s:s + 3] = cand[s2:s2 + 3]

    # z-y-x order inside each face, among the slots the batch's points occupy (R6)
    faces = sorted({p[1] for p in pts})
    for f in faces:
        slots = [p[0] for p in pts if p[1] == f and p[3]]
        verts = sorted((coords(s) for s in slots))       # tuples compare lexicographically: z, then y, then x
        for s, v in zip(slots, verts):
            cand[s:s + 3] = list(v)
    return cand


def correct(cand_rows, label_rows, Ls, n_bins: int, histories=None):
    """All sequences of a pass: lists of rows, one L per sequence."""
    if histories is None:
        histories = [None] * len(cand_rows)
    return [correct_row(c, l, int(L), n_bins, h) for c, l, L, h in zip(cand_rows, label_rows, Ls, histories)]
