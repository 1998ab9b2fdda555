"""Writes tests/golden/latency_closed_forms.json.

The paper prints no worked numeric example of its latency model, so the
fixtures are closed-form evaluations, in exact rational arithmetic, of the
single-call cases below (prefill roofline, KV transfer, decode, queueing as
read from Section 4.2 "Scheduler internals" / "Heterogeneous resource
modelling" and Section 5.3, feasibility by Eq. 3-4, scores by Eq. 2).  This
script uses python fractions only: it calls neither the oracle nor the CUDA
library, so the numbers are independent of both.

Case "hand" is chosen so that every term can be checked with pencil and paper:
  class 1000 TFLOP/s, 1 TB/s; model phi = 2e9 flop/token, omega = 1e9 B,
  kappa = 1e5 B/token; call n = 1000, o = 11
  kvB = 1e8 B;  compute 1000*2e9/1e15 = 0.002 s;  memory (1e9+1e8)/1e12 = 0.0011 s
  prefill = 0.002 s;  context = 1000 + 0.5*10 = 1005 tokens
  bytes/step = 1e9 + 1e5*1005 = 1.1005e9;  decode = 11*1.1005e9/1e12 = 0.0121055 s
  link 100 GB/s -> transfer 0.001 s;  qP = 0.25 -> ready 0.253;  qD = 0.1 < ready
  finish = 0.253 + 0.0121055 = 0.2651055 s
"""
import json
import os
from fractions import Fraction as Fr


def terms(types, model, n, o):
    phi, omega, kappa = (Fr(x) for x in model[:3])
    psi = Fr(model[3]) if len(model) > 3 else Fr(0)      # attention FLOPs per pair of prompt tokens (variant)
    out = []
    for tflops, tbps in types:
        F, B = Fr(tflops) * 10**12, Fr(tbps) * 10**12
        pf = (Fr(n) * phi + Fr(n) * Fr(n) * psi) / F
        pm = (omega + Fr(n) * kappa) / B
        tdec = Fr(o) * (omega + kappa * (Fr(n) + Fr(o - 1) / 2)) / B
        out.append(dict(pf=pf, pm=pm, tpre=max(pf, pm), tdec=tdec))
    return out


def case(name, types, model, n, o, typeP, typeD, qP, qD, capD, bw, elapsed, tail, H, alpha, note):
    t = terms(types, model, n, o)
    kvB = Fr(n) * Fr(model[2])
    fin = []
    for p in range(len(typeP)):
        for d in range(len(typeD)):
            ready = Fr(qP[p]) + t[typeP[p]]["tpre"] + kvB / (Fr(bw[p][d]) * 10**9)
            start = max(ready, Fr(qD[d]))
            fin.append(start + t[typeD[d]]["tdec"] if n + o <= capD[d] else None)
    feas = [f for f in fin if f is not None]
    best = min(feas) if feas else None
    assign = fin.index(best) if feas else -1
    exp = dict(kvB=float(kvB), m=float(n + o),
               tpre=[float(x["tpre"]) for x in t], tdec=[float(x["tdec"]) for x in t],
               pf=[float(x["pf"]) for x in t], pm=[float(x["pm"]) for x in t],
               fin=[None if f is None else float(f) for f in fin], assign=assign)
    if feas:
        comp = Fr(elapsed) + best + Fr(tail)
        exp.update(delta=float(best), completion=float(comp), ratio=float(comp / Fr(H)),
                   ratio_eq2=float((Fr(elapsed) + best) / Fr(H)),
                   slack=float(Fr(alpha) * Fr(H) - comp))
    return dict(name=name, note=note,
                inputs=dict(gpu_types=[[float(a), float(b)] for a, b in types], model=[float(x) for x in model[:3]],
                            attn_flops_per_token2=float(model[3]) if len(model) > 3 else 0.0,
                            prompt_tokens=n, output_tokens=o, typeP=typeP, typeD=typeD,
                            qP=[float(x) for x in qP], qD=[float(x) for x in qD], capD=capD, link_gbps=bw,
                            elapsed=float(elapsed), tail=float(tail), H=float(H), alpha=float(alpha)),
                expected=exp)


def main():
    T3 = [(990, Fr(8)), (312, Fr(2)), (181, Fr(9, 10))]
    cases = [
        case("hand", [(1000, Fr(1))], (2 * 10**9, 10**9, 10**5), 1000, 11, [0], [0],
             [Fr(1, 4)], [Fr(1, 10)], [10**6], [[100]], 0, 0, 1, Fr(3, 2),
             "single class, single pair, every term checkable by hand (see module docstring)"),
        case("hetero_tie", T3, (16 * 10**9, 16 * 10**9, 131072), 1024, 128, [0, 1], [0, 2],
             [Fr(1, 2), 0], [1, 0], [10**6, 10**6], [[100, 50], [400, 25]], 2, 3, 10, Fr(3, 2),
             "three classes, asymmetric link matrix; pairs 0 and 2 both wait for decode instance 0 "
             "and tie exactly, so the lower pair index wins; compute-bound prefill on every class"),
        case("memory_bound_prefill", T3, (14 * 10**10, 14 * 10**10, 327680), 16, 1, [0, 1, 2], [0],
             [0, 0, 0], [0], [10**6], [[200], [200], [200]], 0, 0, 1, Fr(3, 2),
             "short prompt on a large model: the memory term of the prefill roofline wins; with one "
             "output token the decode time equals that memory term"),
        case("capacity_mask", [(1000, Fr(1))], (2 * 10**9, 10**9, 10**5), 1000, 11, [0], [0, 0],
             [0], [0, 5], [1010, 1011], [[100, 100]], 1, 0, 2, Fr(3, 2),
             "demand 1011 tokens: instance 0 (capacity 1010) is infeasible by Eq. 4, instance 1 "
             "(capacity 1011, equality allowed) is taken although it admits five seconds later"),
        case("quadratic_prefill", [(1000, Fr(1))], (2 * 10**9, 10**9, 10**5, 4 * 10**5), 8000, 11, [0], [0],
             [0], [0], [10**6], [[100]], 0, 0, 1, Fr(3, 2),
             "prefill variant with a quadratic attention term: 8000 tokens, 4e5 FLOPs per token pair: "
             "compute = (8000*2e9 + 8000^2*4e5)/1e15 = 0.016 + 0.0256 = 0.0416 s, above the memory term 0.0018 s"),
        case("all_infeasible", [(1000, Fr(1))], (2 * 10**9, 10**9, 10**5), 1000, 11, [0], [0],
             [0], [0], [100], [[100]], 0, 0, 1, Fr(3, 2),
             "no decode instance can hold the call: assignment -1"),
    ]
    out = dict(source="closed-form evaluation in exact rational arithmetic of single-call cases; "
                      "latency reading of Section 4.2/5.3, feasibility Eq. 3-4, scores Eq. 2",
               cases=cases)
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "latency_closed_forms.json")
    with open(path, "w") as f:
        json.dump(out, f, indent=1)
    print("wrote", path)


if __name__ == "__main__":
    main()
