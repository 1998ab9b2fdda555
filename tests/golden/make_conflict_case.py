"""Writes tests/golden/conflict_hand.json.

A worked run of the capacity-conflict pass: the one-pass ordering of a large
queue by the risk score (paper Section 5.3, last sentence), with the decode KV
capacity of Eq. 3-4 as the resource that placements compete for.  The rule, in
words: visit the calls by decreasing priority (Eq. 2 value), lower call index
first among equal priorities; a call takes the first of its K listed candidates
whose decode instance still has at least m(c) free KV tokens; that removes m(c)
tokens from the instance and adds the call's prefill time to the queue of the
candidate's prefill instance (one binary32 addition per placement, in visiting
order); a call none of whose candidates has room stays unplaced.

The paper prints no numeric example, so the eight-call case below was worked
out by hand; the narration is the hand calculation, the constants under HAND
are its results.  The script re-evaluates the case in exact rational
arithmetic (python fractions, with an explicit round-to-nearest-even step for
every binary32 addition) and refuses to write the file unless that evaluation
and the hand results agree.  It calls neither the oracle nor the CUDA library.

Cluster slice: 2 prefill instances, 3 decode instances, K = 3 candidates per
call, pair index j = p * 3 + d.
  free KV tokens   d0 1000, d1 650, d2 300
  prefill queues   p0 1.0 s, p1 0.5 s

Calls (index: priority, demand m, candidates as (p, d), prefill time of each candidate):
  0: 2.5,   200, (0,2) (1,0) (1,1),   0.25   0.125  0.125
  1: 4.0,   300, (0,0) (0,1) none,    2^-24 + 2^-26,  0.5,  -
  2: 2.0,   500, (0,1) (0,0) (1,2),   0.5    0.5    0.5
  3: 5.0,   700, (0,0) (1,1) (0,2),   2^-24  0.25   0.25
  4: 1.0,   400, (1,1) none none,     2^-3 + 2^-25,  -,  -
  5: 4.0,   300, (1,0) (1,2) (0,1),   0.5    0.25   0.5
  6: +inf,    1, none none none       (no decode instance can ever hold it: Eq. 4)
  7: 0.25,  100, (0,1) (1,1) none,    0.5    0.5    -

Hand calculation, in visiting order 6, 3, 1, 5, 0, 2, 4, 7:
  6  priority +inf comes first; it lists no candidate: unplaced.
  3  d0 has 1000 >= 700: takes (0,0) = pair 0.  d0 -> 300.
     p0: 1 + 2^-24 lies exactly half way between 1 and 1 + 2^-23: ties go to the even
     mantissa, p0 stays 1.
  1  and 5 tie at 4.0: the lower index, 1, goes first.  d0 has 300 >= 300 (equality
     fits): takes (0,0) = pair 0.  d0 -> 0.
     p0: 1 + 2^-24 + 2^-26 is above the half-way point: p0 -> 1 + 2^-23.
     (Had call 1 gone before call 3, p0 would be 1 + 2^-23 after call 1 and
     1 + 2^-23 + 2^-24 -> tie -> even -> 1 + 2^-22 after call 3: the order of the
     additions is part of the result.)
  5  first candidate d0 has 0 < 300: full.  Second candidate d2 has 300 >= 300: takes
     (1,2) = pair 5.  d2 -> 0.  p1: 0.5 + 0.25 = 0.75.
     (Had call 5 gone before call 1, it would hold d0 and call 1 would move to d1.)
  0  d2 has 0, d0 has 0, third candidate d1 has 650 >= 200: takes (1,1) = pair 4.
     d1 -> 450.  p1: 0.75 + 0.125 = 0.875.
  2  d1 has 450 < 500, d0 has 0, d2 has 0: unplaced.
  4  d1 has 450 >= 400: takes (1,1) = pair 4.  d1 -> 50.
     p1: 0.875 + 2^-3 + 2^-25 = 1 + 2^-25, a quarter of the spacing 2^-23 above 1: p1 -> 1.
  7  d1 has 50 < 100 (twice): unplaced.
"""
import json
import os
from fractions import Fraction as Fr

K, P, D = 3, 2, 3
FREE = [1000, 650, 300]
QP = [Fr(1), Fr(1, 2)]
INF = "inf"
NONE = None
# priority, demand, candidates (p, d) or None, prefill time per candidate
CALLS = [
    (Fr(5, 2), 200, [(0, 2), (1, 0), (1, 1)], [Fr(1, 4), Fr(1, 8), Fr(1, 8)]),
    (Fr(4), 300, [(0, 0), (0, 1), NONE], [Fr(1, 2**24) + Fr(1, 2**26), Fr(1, 2), Fr(0)]),
    (Fr(2), 500, [(0, 1), (0, 0), (1, 2)], [Fr(1, 2), Fr(1, 2), Fr(1, 2)]),
    (Fr(5), 700, [(0, 0), (1, 1), (0, 2)], [Fr(1, 2**24), Fr(1, 4), Fr(1, 4)]),
    (Fr(1), 400, [(1, 1), NONE, NONE], [Fr(1, 8) + Fr(1, 2**25), Fr(0), Fr(0)]),
    (Fr(4), 300, [(1, 0), (1, 2), (0, 1)], [Fr(1, 2), Fr(1, 4), Fr(1, 2)]),
    (INF, 1, [NONE, NONE, NONE], [Fr(0), Fr(0), Fr(0)]),
    (Fr(1, 4), 100, [(0, 1), (1, 1), NONE], [Fr(1, 2), Fr(1, 2), Fr(0)]),
]

# results of the hand calculation in the docstring
HAND_ORDER = [6, 3, 1, 5, 0, 2, 4, 7]
HAND_ASSIGN = [4, 0, -1, 0, 4, 5, -1, -1]
HAND_FREE = [0, 50, 0]
HAND_QP = [Fr(1) + Fr(1, 2**23), Fr(1)]


def round_f32(x: Fr) -> Fr:
    """x >= 0 rounded to the nearest binary32 value, ties to the even mantissa (normal range only)."""
    if x == 0:
        return x
    e = 0
    while Fr(2) ** (e + 1) <= x:
        e += 1
    while Fr(2) ** e > x:
        e -= 1
    assert -126 <= e <= 127
    ulp = Fr(2) ** (e - 23)
    q, r = divmod(x, ulp)                 # q = integer mantissa in [2^23, 2^24)
    if r > ulp / 2 or (r == ulp / 2 and q % 2 == 1):
        q += 1
    return q * ulp


def is_f32(x: Fr) -> bool:
    return round_f32(x) == x


def evaluate():
    free, qP = list(FREE), list(QP)
    key = lambda c: (0 if CALLS[c][0] == INF else 1, -(CALLS[c][0] if CALLS[c][0] != INF else 0), c)
    order = sorted(range(len(CALLS)), key=key)
    assign = [-1] * len(CALLS)
    for c in order:
        _, m, cands, tpre = CALLS[c]
        for k in range(K):
            if cands[k] is None:
                continue
            p, d = cands[k]
            if free[d] >= m:
                free[d] -= m
                qP[p] = round_f32(qP[p] + tpre[k])
                assign[c] = p * D + d
                break
    return order, assign, free, qP


def main():
    order, assign, free, qP = evaluate()
    assert order == HAND_ORDER and assign == HAND_ASSIGN and free == HAND_FREE and qP == HAND_QP, \
        (order, assign, free, qP)
    for prio, m, cands, tpre in CALLS:                       # every input is a binary32 value
        assert prio == INF or is_f32(prio)
        assert all(is_f32(t) for t in tpre)
    # the two remarks of the narration about other orders, evaluated as well
    swapped = round_f32(round_f32(QP[0] + CALLS[1][3][0]) + CALLS[3][3][0])
    assert swapped == Fr(1) + Fr(1, 2**22) and swapped != HAND_QP[0]
    out = {
        "source": "hand-worked case of the one-pass capacity rule (Section 5.3 last sentence, Eq. 3-4); "
                  "written by tests/golden/make_conflict_case.py",
        "K": K, "P": P, "D": D,
        "free": FREE,
        "qP": [float(q) for q in QP],
        "prio": [INF if c[0] == INF else float(c[0]) for c in CALLS],
        "m": [c[1] for c in CALLS],
        "pair": [[-1 if pd is None else pd[0] * D + pd[1] for pd in c[2]] for c in CALLS],
        "tpre": [[float(t) for t in c[3]] for c in CALLS],       # exact: all are binary32 values
        "expect": {"order": HAND_ORDER, "assign": HAND_ASSIGN, "free": HAND_FREE,
                   "qP_hex": [float(q).hex() for q in HAND_QP]},
    }
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "conflict_hand.json")
    with open(path, "w") as f:
        json.dump(out, f, indent=1)
    print("wrote", path)


if __name__ == "__main__":
    main()
