"""Writes tests/golden/greedy_hand.json.

A worked run of the recomputing greedy planner (paper Algorithm 1, the
while-loop over the queue snapshot; Section 5.3 "Adaptive greedy prefill
assignment"): until the queue is empty, project every waiting call's best
feasible pair against the simulated state, take the call with the largest
ratio R = (elapsed + Delta) / H (Eq. 2), record its pair, add its prefill time
to the chosen prefill queue, take its KV tokens (Eq. 3) from the chosen decode
instance, remove it.  The paper prints no numeric example, so the run below is
evaluated in exact rational arithmetic with python fractions; it calls neither
the oracle nor the CUDA library.  Every decision (the pair of a call, the call
of an iteration) is required either to win by a relative margin of 1e-4 or to
tie exactly through the same clamped admission time (then the lower index
wins on both sides), so binary32 rounding cannot change the expected integers.

Cluster: classes {1000 TFLOP/s, 1 TB/s} and {250 TFLOP/s, 0.5 TB/s};
prefill P0 (class 0, queue 0.010 s), P1 (class 1, idle);
decode D0 (class 0, admits at 0.020 s, 4000 tokens free), D1 (class 1, admits
at once, 2400 tokens free); both hold 4096 tokens in total;
links 100 / 50 / 25 / 200 GB/s; model phi = 2e9, omega = 1e9, kappa = 1e5.
"""
import json
import os
from fractions import Fraction as Fr

TYPES = [(1000, Fr(1)), (250, Fr(1, 2))]
MODEL = (2 * 10**9, 10**9, 10**5)
TYPE_P, TYPE_D = [0, 1], [0, 1]
QP = [Fr(1, 100), Fr(0)]
QD = [Fr(2, 100), Fr(0)]
CAP = [4096, 4096]
FREE = [4000, 2400]
BW = [[100, 50], [25, 200]]
# (prompt tokens, output tokens, elapsed seconds of the workflow, horizon H of the workflow)
CALLS = [(1000, 100, Fr(1, 2), Fr(2)), (400, 50, Fr(1, 10), Fr(1, 2)), (1200, 200, Fr(0), Fr(1)),
         (300, 20, Fr(3, 10), Fr(1)), (900, 60, Fr(1), Fr(4)), (2000, 500, Fr(1), Fr(1))]
MARGIN = Fr(1, 10**4)


def terms(n, o):
    phi, omega, kappa = (Fr(x) for x in MODEL)
    out = []
    for tflops, tbps in TYPES:
        F, B = Fr(tflops) * 10**12, Fr(tbps) * 10**12
        tpre = max(Fr(n) * phi / F, (omega + Fr(n) * kappa) / B)
        tdec = Fr(o) * (omega + kappa * (Fr(n) + Fr(o - 1) / 2)) / B
        out.append((tpre, tdec))
    return out


def clear(best, others):
    """every other value either ties exactly (both sides clamp to the same admission time, so the
    binary32 values tie as well and the index rule decides) or is off by the relative margin"""
    return all(x == best or abs(x - best) > MARGIN * abs(best) for x in others)


def main():
    qP, free = list(QP), list(FREE)
    waiting = list(range(len(CALLS)))
    assign = [-1] * len(CALLS)
    ratio = [None] * len(CALLS)
    order, trace = [], []
    while waiting:
        proj = {}
        for c in waiting:
            n, o, el, H = CALLS[c]
            t = terms(n, o)
            fins = {}
            for p in range(2):
                for d in range(2):
                    if n + o > CAP[d] or n + o > free[d]:
                        continue
                    ready = qP[p] + t[TYPE_P[p]][0] + Fr(n) * MODEL[2] / (Fr(BW[p][d]) * 10**9)
                    fins[p * 2 + d] = max(ready, QD[d]) + t[TYPE_D[d]][1]
            if not fins:
                continue
            j = min(fins, key=lambda k: (fins[k], k))
            assert clear(fins[j], [v for k, v in fins.items() if k != j]), ("pair margin", c)
            proj[c] = (j, (el + fins[j]) / H)
        if not proj:
            break
        cstar = max(proj, key=lambda c: (proj[c][1], -c))
        assert clear(proj[cstar][1], [v[1] for c, v in proj.items() if c != cstar]), ("call margin", cstar)
        j, R = proj[cstar]
        p, d = divmod(j, 2)
        n, o, _, _ = CALLS[cstar]
        qP[p] += terms(n, o)[TYPE_P[p]][0]
        free[d] -= n + o
        assign[cstar], ratio[cstar] = j, R
        order.append(cstar)
        waiting.remove(cstar)
        trace.append(dict(call=cstar, pair=j, ratio=float(R), qP=[float(x) for x in qP], free=list(free)))
    out = dict(
        source="exact rational evaluation of the recomputing greedy loop of Algorithm 1 (Section 5.3, "
               "'Adaptive greedy prefill assignment'), ratio by Eq. 2, demand by Eq. 3, feasibility by Eq. 4 "
               "and by the free KV tokens of the simulated state",
        inputs=dict(gpu_types=[[float(a), float(b)] for a, b in TYPES], model=[float(x) for x in MODEL],
                    typeP=TYPE_P, typeD=TYPE_D, qP=[float(x) for x in QP], qD=[float(x) for x in QD],
                    capD=CAP, freeD=FREE, link_gbps=BW,
                    calls=[dict(prompt_tokens=n, output_tokens=o, elapsed=float(el), H=float(H))
                           for n, o, el, H in CALLS]),
        expected=dict(order=order, assign=assign, ratio=[None if r is None else float(r) for r in ratio],
                      qP=[float(x) for x in qP], freeD=free, trace=trace))
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "greedy_hand.json")
    with open(path, "w") as f:
        json.dump(out, f, indent=1)
    print("wrote", path)
    for t in trace:
        print(t)
    print("unplaced:", [c for c in range(len(CALLS)) if assign[c] < 0])


if __name__ == "__main__":
    main()
