"""Writes tests/golden/decode_hand.json.

A worked run of the decode-stage scheduler (paper Section 5.4, "Adaptive greedy
decode assignment"): repeatedly take the waiting call with the largest ratio
R = (elapsed + Delta_D) / H (Eq. 2), where Delta_D is its earliest projected
decode finish over its legal decode instances; a locked call may only use its
instance; the earliest capacity-feasible start on an instance is the first time
t >= ready at which the instance has m(c) = L_in + L_out (Eq. 3) tokens free for
the whole decode (Cap(d) of Eq. 4 minus the tokens of the intervals that overlap);
the chosen interval is added to the simulated state.  The paper prints no
numeric example, so the run is evaluated here in exact rational arithmetic from
the definition (candidate starts = the ready time and the ends of intervals;
usage checked at the start and at every interval start inside the window); it
calls neither the oracle nor the CUDA library.  Every decision wins by a
relative margin of 1e-4.

One GPU class per decode instance: D0 = {1000 TFLOP/s, 1 TB/s}, 3000 tokens;
D1 = {250 TFLOP/s, 0.5 TB/s}, 2500 tokens.  Model phi = 2e9, omega = 1e9,
kappa = 1e5.  Running now: on D0 1200 tokens until 0.030 s and 900 tokens until
0.012 s; on D1 800 tokens until 0.050 s.
"""
import json
import os
from fractions import Fraction as Fr

TYPES = [(1000, Fr(1)), (250, Fr(1, 2))]
MODEL = (2 * 10**9, 10**9, 10**5)
TYPE_D = [0, 1]
CAP = [3000, 2500]
RUNNING = [[(Fr(30, 1000), 1200), (Fr(12, 1000), 900)], [(Fr(50, 1000), 800)]]
# (prompt, output, lock, ready, elapsed, H)
CALLS = [(1000, 100, -1, Fr(0), Fr(1, 2), Fr(2)),
         (600, 50, 1, Fr(5, 1000), Fr(1, 10), Fr(1, 2)),
         (1500, 200, -1, Fr(0), Fr(0), Fr(1)),
         (300, 20, -1, Fr(2, 1000), Fr(3, 10), Fr(1)),
         (900, 60, 0, Fr(0), Fr(1), Fr(4)),
         (2600, 300, -1, Fr(0), Fr(1), Fr(1))]
MARGIN = Fr(1, 10**4)


def tdec(n, o, g):
    phi, omega, kappa = (Fr(x) for x in MODEL)
    B = Fr(TYPES[g][1]) * 10**12
    return Fr(o) * (omega + kappa * (Fr(n) + Fr(o - 1) / 2)) / B


def usage(iv, t):
    return sum(m for s, e, m in iv if s <= t < e)


def earliest(iv, cap, m, tau, ready):
    cands = sorted({ready} | {e for s, e, _ in iv if e > ready})
    for c in cands:
        checks = [c] + [s for s, e, _ in iv if c < s < c + tau]
        if all(usage(iv, t) + m <= cap for t in checks):
            return c
    raise AssertionError("no feasible start")


def clear(best, others):
    return all(abs(x - best) > MARGIN * abs(best) for x in others)


def project(iv, c):
    """(instance, start, finish) with the earliest finish over the legal instances, None if there is none."""
    n, o, lock, ready, el, H = CALLS[c]
    opts = {}
    for d in range(2):
        if (lock >= 0 and lock != d) or n + o > CAP[d]:
            continue
        tau = tdec(n, o, TYPE_D[d])
        s = earliest(iv[d], CAP[d], n + o, tau, ready)
        opts[d] = (s + tau, s)
    if not opts:
        return None
    d = min(opts, key=lambda k: (opts[k][0], k))
    assert clear(opts[d][0], [v[0] for k, v in opts.items() if k != d]), ("instance margin", c)
    return d, opts[d][1], opts[d][0]


def one_pass():
    """The fallback ordering (Section 5.4 with Section 5.3, last sentence): ranked once by the ratio projected
    against the running intervals alone, then placed in that order against the growing state."""
    iv = [[(Fr(0), e, m) for e, m in RUNNING[d]] for d in range(2)]
    score = {}
    for c in range(len(CALLS)):
        pr = project(iv, c)
        if pr is not None:
            score[c] = (CALLS[c][4] + pr[2]) / CALLS[c][5]
    visit = sorted(score, key=lambda c: (-score[c], c))
    for a, b in zip(visit, visit[1:]):
        assert score[a] - score[b] > MARGIN * score[a], ("score margin", a, b)
    inst = [-1] * len(CALLS); start = [None] * len(CALLS); ratio = [None] * len(CALLS)
    for c in visit:
        d, s, f = project(iv, c)
        iv[d].append((s, f, CALLS[c][0] + CALLS[c][1]))
        inst[c], start[c], ratio[c] = d, s, score[c]
    return dict(order=visit, inst=inst, start=[None if s is None else float(s) for s in start],
                ratio=[None if r is None else float(r) for r in ratio])


def main():
    iv = [[(Fr(0), e, m) for e, m in RUNNING[d]] for d in range(2)]
    waiting = list(range(len(CALLS)))
    inst = [-1] * len(CALLS); start = [None] * len(CALLS); ratio = [None] * len(CALLS)
    order, trace = [], []
    while waiting:
        proj = {}
        for c in waiting:
            n, o, lock, ready, el, H = CALLS[c]
            m = n + o
            opts = {}
            for d in range(2):
                if (lock >= 0 and lock != d) or m > CAP[d]:
                    continue
                tau = tdec(n, o, TYPE_D[d])
                s = earliest(iv[d], CAP[d], m, tau, ready)
                opts[d] = (s + tau, s)
            if not opts:
                continue
            d = min(opts, key=lambda k: (opts[k][0], k))
            assert clear(opts[d][0], [v[0] for k, v in opts.items() if k != d]), ("instance margin", c)
            proj[c] = (d, opts[d][1], opts[d][0], (el + opts[d][0]) / H)
        if not proj:
            break
        cs = max(proj, key=lambda c: (proj[c][3], -c))
        assert clear(proj[cs][3], [v[3] for c, v in proj.items() if c != cs]), ("call margin", cs)
        d, s, f, R = proj[cs]
        n, o = CALLS[cs][0], CALLS[cs][1]
        iv[d].append((s, f, n + o))
        inst[cs], start[cs], ratio[cs] = d, s, R
        order.append(cs)
        waiting.remove(cs)
        trace.append(dict(call=cs, inst=d, start=float(s), finish=float(f), ratio=float(R)))
    out = dict(
        source="exact rational evaluation of the decode-stage greedy of Section 5.4 ('Adaptive greedy decode "
               "assignment'): ratio by Eq. 2, demand by Eq. 3, capacity by Eq. 4 over token-capacity intervals",
        inputs=dict(gpu_types=[[float(a), float(b)] for a, b in TYPES], model=[float(x) for x in MODEL],
                    typeD=TYPE_D, capD=CAP,
                    running=[[dict(end=float(e), tokens=m) for e, m in RUNNING[d]] for d in range(2)],
                    calls=[dict(prompt_tokens=n, output_tokens=o, lock=lock, ready=float(r), elapsed=float(el),
                                H=float(H)) for n, o, lock, r, el, H in CALLS]),
        expected=dict(order=order, inst=inst, start=[None if s is None else float(s) for s in start],
                      ratio=[None if r is None else float(r) for r in ratio], trace=trace),
        expected_one_pass=one_pass())
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "decode_hand.json")
    with open(path, "w") as f:
        json.dump(out, f, indent=1)
    print("wrote", path)
    for t in trace:
        print(t)
    print("one pass:", out["expected_one_pass"])
    print("unplaced:", [c for c in range(len(CALLS)) if inst[c] < 0])


if __name__ == "__main__":
    main()
