"""Seeded input generator for the five evaluation configurations.

Everything here is input data: GPU-type tables, instance pools, link-bandwidth
matrices, queue loads, KV capacities, workflow DAG forests in successor-CSR
form, per-node call annotations (model, prompt length, output length) and the
batch of ready calls.  No quantity that the scheduler computes (latencies,
critical paths, scores) is produced or used here.

The public traces the paper evaluates on (conversational chains, function
calling chains, tree-search fan-outs, Section 7.1 "Workloads") are not
available offline; the shapes below stand in for them: chains, fan-out/join
stages and random layered DAGs with log-normal token lengths.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np

CALL_DTYPE = np.dtype([("node", "<u4"), ("model", "<u4"),
                       ("prompt_tokens", "<f4"), ("output_tokens", "<f4")])

CONFIG_NAMES = ("tiny", "medium", "large", "cp_stress", "sweep")

# peak dense TFLOP/s, HBM TB/s.  The first three are the values the Tiny
# configuration fixes; the remaining five only extend the list so that six and
# eight distinct classes exist.
_GPU_TYPES = np.array([[990.0, 8.0], [312.0, 2.0], [181.0, 0.9],
                       [1979.0, 3.35], [989.0, 4.8], [125.0, 0.3],
                       [2250.0, 8.0], [60.0, 0.9]], dtype=np.float32)

# flops per token, weight bytes, KV bytes per token
_MODEL_8B = (1.6e10, 1.6e10, 131072.0)     # 32 layers x 8 KV heads x 128 x 2 (K,V) x bf16
_MODEL_70B = (1.4e11, 1.4e11, 327680.0)    # 80 layers x 8 KV heads x 128 x 2 x bf16

_CAP_TOKENS = np.array([262144.0, 524288.0, 1048576.0], dtype=np.float32)


@dataclass
class Workload:
    name: str
    seed: int
    gpu_types: np.ndarray          # (G, 2) f32
    P: int
    D: int
    inst_type: np.ndarray          # (P+D,) u32, prefill instances first
    load_s: np.ndarray             # (P+D,) f32 seconds until the instance can take new work
    kv_cap: np.ndarray             # (P+D,) f32 tokens (0 for prefill instances)
    kv_free: np.ndarray            # (P+D,) f32 tokens
    link_gbps: np.ndarray          # (P+D, P+D) f32
    models: np.ndarray             # (M, 3) f32
    row_ptr: np.ndarray            # (N+1,) u32 successor CSR
    col: np.ndarray                # (E,) u32
    node_wf: np.ndarray            # (N,) u32
    n_workflows: int
    node_calls: np.ndarray         # (N,) CALL_DTYPE, annotation of every node
    elapsed: np.ndarray            # (W,) f32 seconds since workflow arrival
    ready_nodes: np.ndarray        # (C,) u32 nodes in the ready batch
    chunk: int                     # calls per scheduler invocation
    topk: int = 0
    commit: bool = False
    alpha: float = 1.5
    node_cost: Optional[np.ndarray] = None   # (N,) f32 when the config fixes node costs
    depth: Optional[np.ndarray] = None       # (W,) number of layers drawn per workflow
    notes: dict = field(default_factory=dict)

    @property
    def n_nodes(self) -> int:
        return int(self.node_wf.shape[0])

    @property
    def n_edges(self) -> int:
        return int(self.col.shape[0])

    @property
    def calls(self) -> np.ndarray:
        return np.ascontiguousarray(self.node_calls[self.ready_nodes])

    @property
    def n_candidates(self) -> int:
        return int(self.ready_nodes.shape[0]) * self.P * self.D


# --------------------------------------------------------------------------
# forests
# --------------------------------------------------------------------------

MODE_RANDOM, MODE_STAGES, MODE_CHAIN = 0, 1, 2


def _layered_forest(rng, n_w, depth_w, mode_w, fan_in_max, extra_mean):
    """Build a forest of layered DAGs.

    Every workflow w has n_w[w] nodes spread over depth_w[w] non-empty layers.
    Nodes are numbered workflow by workflow and, inside a workflow, layer by
    layer, so the numbering is a topological order.  Edges run from earlier
    layers to later ones:
      MODE_CHAIN  - one node per layer, each linked to its predecessor;
      MODE_STAGES - alternating single hub / fan-out layers, every node linked
                    to all nodes of the previous layer (fan-out then join);
      MODE_RANDOM - one parent in the previous layer (children dealt round-robin
                    over that layer) plus a geometric number of extra parents
                    anywhere earlier in the same workflow, at most fan_in_max.
    Returns successor CSR (row_ptr, col), node_wf and the per-node max parent
    (-1 for sources).
    """
    n_w = np.asarray(n_w, dtype=np.int64)
    depth_w = np.minimum(np.asarray(depth_w, dtype=np.int64), n_w)
    depth_w = np.maximum(depth_w, 1)
    W = n_w.shape[0]
    N = int(n_w.sum())
    wf_start = np.zeros(W + 1, dtype=np.int64)
    np.cumsum(n_w, out=wf_start[1:])
    wf = np.repeat(np.arange(W, dtype=np.int64), n_w)
    local = np.arange(N, dtype=np.int64) - wf_start[wf]
    depth = depth_w[wf]
    mode = np.asarray(mode_w, dtype=np.int64)[wf]

    u = rng.random(N)
    lay_rand = np.minimum((u * depth).astype(np.int64), depth - 1)
    # fan-out layers are the odd ones; a workflow with a single layer keeps layer 0
    n_odd = depth // 2
    lay_odd = np.where(n_odd > 0, 2 * np.minimum((u * n_odd).astype(np.int64),
                                                 np.maximum(n_odd - 1, 0)) + 1, 0)
    extra_layer = np.where(mode == MODE_STAGES, lay_odd, lay_rand)
    layer = np.where(local < depth, local, extra_layer)

    order = np.lexsort((layer, wf))          # stable: by workflow, then by layer
    layer = layer[order]
    mode = mode[order]
    # (wf, local) are unchanged by a permutation inside each workflow
    idx = np.arange(N, dtype=np.int64)
    key = wf * (int(depth_w.max()) + 1) + layer
    new_group = np.ones(N, dtype=bool)
    new_group[1:] = key[1:] != key[:-1]
    group_id = np.cumsum(new_group) - 1
    group_start = idx[new_group]
    layer_start = group_start[group_id]
    prev_start = np.where(layer > 0, group_start[np.maximum(group_id - 1, 0)], layer_start)
    prev_width = layer_start - prev_start    # 0 for layer-0 nodes
    rank = idx - layer_start
    w_start = wf_start[wf]

    has_parent = layer > 0
    extra = np.minimum(np.floor(rng.exponential(extra_mean, N)).astype(np.int64),
                       fan_in_max - 1) if extra_mean > 0 else np.zeros(N, dtype=np.int64)
    cnt = np.where(mode == MODE_STAGES, np.minimum(prev_width, fan_in_max),
                   np.where(mode == MODE_CHAIN, 1, 1 + extra))
    cnt = np.where(has_parent, cnt, 0)
    E0 = int(cnt.sum())
    child = np.repeat(idx, cnt)
    e_start = np.zeros(N + 1, dtype=np.int64)
    np.cumsum(cnt, out=e_start[1:])
    k = np.arange(E0, dtype=np.int64) - e_start[child]
    shift = rng.integers(0, 1 << 30, size=int(group_id[-1]) + 1 if N else 0)[group_id]
    primary = prev_start + (rank + shift) % np.maximum(prev_width, 1)
    ue = rng.random(E0)
    span = (layer_start - w_start)[child]
    anywhere = w_start[child] + np.minimum((ue * span).astype(np.int64), np.maximum(span - 1, 0))
    dense = prev_start[child] + k
    parent = np.where(mode[child] == MODE_STAGES, dense,
                      np.where(k == 0, primary[child], anywhere))
    pair = np.unique(parent * N + child)     # drop duplicate edges, sort by (parent, child)
    parent = pair // N
    child = pair % N
    assert np.all(parent < child)
    row_ptr = np.zeros(N + 1, dtype=np.int64)
    np.add.at(row_ptr, parent + 1, 1)
    np.cumsum(row_ptr, out=row_ptr)
    maxpar = np.full(N, -1, dtype=np.int64)
    np.maximum.at(maxpar, child, parent)
    return (row_ptr.astype(np.uint32), child.astype(np.uint32), wf.astype(np.uint32),
            maxpar, wf_start, layer)


def _workflow_shapes(rng, W, n_lo, n_hi, mix):
    """Draw node count, layer count and connection mode per workflow."""
    n_w = rng.integers(n_lo, n_hi + 1, size=W)
    mode_w = rng.choice(np.array([MODE_RANDOM, MODE_STAGES, MODE_CHAIN]), size=W, p=np.asarray(mix))
    fan = rng.integers(2, 9, size=W)                       # fan-out 2..8 of a stage
    stages = np.maximum(1, n_w // (fan + 1))
    depth_stage = np.minimum(n_w, 2 * stages + 1)
    # random DAGs: widths of about 1..3 per layer
    depth_rand = np.maximum(1, np.minimum(n_w, np.ceil(n_w / rng.uniform(1.2, 3.0, size=W)).astype(np.int64)))
    depth_w = np.where(mode_w == MODE_CHAIN, n_w, np.where(mode_w == MODE_STAGES, depth_stage, depth_rand))
    return n_w, depth_w, mode_w


def _cp_stress_shapes(rng, W, N_total, max_depth):
    """Heavy-tailed workflow sizes summing to N_total exactly; depth up to max_depth."""
    raw = rng.lognormal(3.2, 1.1, size=W)
    n_w = np.clip(np.round(raw * (N_total / raw.sum())), 1, 4096).astype(np.int64)
    # land on the exact total by nudging randomly chosen workflows one node at a time
    diff = int(N_total - n_w.sum())
    while diff != 0:
        step = 1 if diff > 0 else -1
        cand = np.flatnonzero((n_w + step >= 1) & (n_w + step <= 4096))
        pick = rng.choice(cand, size=min(abs(diff), cand.shape[0]), replace=False)
        n_w[pick] += step
        diff = int(N_total - n_w.sum())
    depth_w = 1 + (rng.random(W) * np.minimum(n_w, max_depth)).astype(np.int64)
    depth_w = np.minimum(depth_w, np.minimum(n_w, max_depth))
    big = int(np.argmax(n_w))
    depth_w[big] = min(int(n_w[big]), max_depth)           # the deepest case is always present
    mode_w = np.full(W, MODE_RANDOM, dtype=np.int64)
    return n_w, depth_w, mode_w


def _pick_ready(rng, C, n_w, wf_start, node_wf, maxpar):
    """Choose exactly C not-yet-complete nodes, runnable ones first.

    A random topological prefix of every workflow is complete.  A node is
    runnable when it is outside the prefix and all its parents are inside.
    Runnable nodes are taken first (in random order); if there are fewer than C
    the batch is topped up with the nodes that follow the frontier most closely.
    """
    W = n_w.shape[0]
    N = node_wf.shape[0]
    wf = node_wf.astype(np.int64)
    q = np.minimum((rng.random(W) * n_w).astype(np.int64), n_w - 1)   # prefix length < n_w
    if C > N:
        raise ValueError("not enough nodes for the requested batch")
    while int(q.sum()) > N - C:                             # keep at least C nodes pending
        q = (q * 9) // 10
    local = np.arange(N, dtype=np.int64) - wf_start[wf]
    pending = local >= q[wf]
    runnable = pending & (maxpar < (wf_start[wf] + q[wf]))
    dist = np.where(runnable, 0, 1 + local - q[wf]).astype(np.float64)
    keyv = np.where(pending, dist + rng.random(N) * 0.5, np.inf)
    chosen = np.argpartition(keyv, C - 1)[:C]
    chosen = chosen[rng.permutation(C)]                     # arbitrary arrival order
    return chosen.astype(np.uint32), int(runnable.sum())


def _lognormal_tokens(rng, size, mu, sigma, cap):
    x = np.round(rng.lognormal(mu, sigma, size=size))
    return np.clip(x, 1.0, float(cap)).astype(np.float32)


_SPECS = {
    # name: G, P, D, C, W, n_lo, n_hi, shape mix (random, stages, chain), prompt (mu, sigma, cap), models, seed
    "tiny":      dict(G=3, P=2, D=2, C=64, W=8, n=(8, 12), mix=(1.0, 0.0, 0.0),
                      prompt=(7.0, 1.0, 32768), models=(_MODEL_8B,), seed=0, chunk=64),
    "medium":    dict(G=6, P=16, D=16, C=4096, W=512, n=(8, 64), mix=(0.2, 0.5, 0.3),
                      prompt=(7.0, 1.0, 32768), models=(_MODEL_8B,), seed=1, chunk=4096),
    "large":     dict(G=8, P=64, D=64, C=65536, W=8192, n=(8, 128), mix=(0.2, 0.5, 0.3),
                      prompt=(8.0, 1.2, 131072), models=(_MODEL_8B, _MODEL_70B), seed=2, chunk=65536),
    "cp_stress": dict(G=8, P=32, D=32, C=50000, W=16384, n=None, mix=None,
                      prompt=(7.0, 1.0, 32768), models=(_MODEL_8B,), seed=3, chunk=50000),
    "sweep":     dict(G=8, P=128, D=128, C=262144, W=32768, n=(8, 24), mix=(0.2, 0.6, 0.2),
                      prompt=(7.0, 1.0, 32768), models=(_MODEL_8B, _MODEL_70B), seed=4, chunk=16384),
}


def make_workload(name: str, seed: Optional[int] = None, scale: float = 1.0) -> Workload:
    """Build one of the five configurations.

    `scale` < 1 shrinks the call and workflow counts (cluster size unchanged) so
    that a slow checker can run the same kind of input in seconds.
    """
    spec = dict(_SPECS[name])
    seed = spec["seed"] if seed is None else int(seed)
    rng = np.random.default_rng([seed, CONFIG_NAMES.index(name)])
    G, P, D = spec["G"], spec["P"], spec["D"]
    C = max(1, int(round(spec["C"] * scale)))
    W = max(1, int(round(spec["W"] * scale)))
    chunk = min(spec["chunk"], C)

    gpu_types = _GPU_TYPES[:G].copy()
    I = P + D
    inst_type = (np.arange(I) % G).astype(np.uint32)        # every pool mixes all classes
    inst_type[P:] = (np.arange(D) % G).astype(np.uint32)
    load_s = rng.uniform(0.0, 2.0, size=I).astype(np.float32)
    kv_cap = np.zeros(I, dtype=np.float32)
    kv_cap[P:] = _CAP_TOKENS[np.arange(D) % 3]
    kv_free = kv_cap.copy()
    if name == "sweep":
        kv_free[P:] = np.floor(rng.uniform(1.5e5, 6.0e5, size=D)).astype(np.float32)
        kv_free[P:] = np.minimum(kv_free[P:], kv_cap[P:])
    link = rng.uniform(25.0, 400.0, size=(I, I)).astype(np.float32)
    models = np.array(spec["models"], dtype=np.float32)

    node_cost = None
    if name == "cp_stress":
        n_total = max(W, int(round(1_000_000 * scale)))
        n_w, depth_w, mode_w = _cp_stress_shapes(rng, W, n_total, 256)
        fan_in_max, extra_mean = 16, 1.5
    else:
        n_w, depth_w, mode_w = _workflow_shapes(rng, W, spec["n"][0], spec["n"][1], spec["mix"])
        fan_in_max, extra_mean = 8, 0.4
    row_ptr, col, node_wf, maxpar, wf_start, _ = _layered_forest(
        rng, n_w, depth_w, mode_w, fan_in_max, extra_mean)
    N = node_wf.shape[0]
    if name == "cp_stress":
        node_cost = rng.lognormal(0.0, 1.0, size=N).astype(np.float32)

    mu, sigma, cap = spec["prompt"]
    node_calls = np.zeros(N, dtype=CALL_DTYPE)
    node_calls["node"] = np.arange(N, dtype=np.uint32)
    node_calls["model"] = rng.integers(0, models.shape[0], size=N).astype(np.uint32)
    node_calls["prompt_tokens"] = _lognormal_tokens(rng, N, mu, sigma, cap)
    node_calls["output_tokens"] = _lognormal_tokens(rng, N, 5.0, 1.0, 32768)

    # seconds since arrival: up to two seconds per layer of the workflow
    elapsed = (rng.random(W) * 2.0 * depth_w).astype(np.float32)
    ready, n_runnable = _pick_ready(rng, C, n_w, wf_start, node_wf, maxpar)

    return Workload(
        name=name, seed=seed, gpu_types=gpu_types, P=P, D=D, inst_type=inst_type,
        load_s=load_s, kv_cap=kv_cap, kv_free=kv_free, link_gbps=link, models=models,
        row_ptr=row_ptr, col=col, node_wf=node_wf, n_workflows=W, node_calls=node_calls,
        elapsed=elapsed, ready_nodes=ready, chunk=chunk,
        topk=4 if name == "sweep" else 0, commit=(name == "sweep"),
        node_cost=node_cost, depth=depth_w.astype(np.int64),
        notes={"runnable_in_batch": min(n_runnable, C), "scale": scale})


def sub_forest(wl: Workload, workflows: np.ndarray):
    """Extract the given workflows as a stand-alone forest.

    Returns (row_ptr, col, node_wf_local, node_ids) where node_ids maps the new
    node numbers back to the original ones and node_wf_local numbers the kept
    workflows 0..k-1 in the order given.  Only valid for forests whose nodes are
    numbered workflow by workflow, which is what this module produces.
    """
    workflows = np.asarray(workflows, dtype=np.int64)
    wf = wl.node_wf.astype(np.int64)
    starts = np.searchsorted(wf, workflows, side="left")
    ends = np.searchsorted(wf, workflows, side="right")
    node_ids = np.concatenate([np.arange(s, e, dtype=np.int64) for s, e in zip(starts, ends)]) \
        if workflows.size else np.zeros(0, dtype=np.int64)
    new_of_old = np.full(wl.n_nodes, -1, dtype=np.int64)
    new_of_old[node_ids] = np.arange(node_ids.shape[0])
    rp = wl.row_ptr.astype(np.int64)
    deg = rp[node_ids + 1] - rp[node_ids]
    row_ptr = np.zeros(node_ids.shape[0] + 1, dtype=np.int64)
    np.cumsum(deg, out=row_ptr[1:])
    src = np.repeat(rp[node_ids], deg) + (np.arange(int(deg.sum())) - np.repeat(row_ptr[:-1], deg))
    col = new_of_old[wl.col[src].astype(np.int64)]
    assert np.all(col >= 0)
    local_wf = np.repeat(np.arange(workflows.shape[0]), ends - starts)
    return (row_ptr.astype(np.uint32), col.astype(np.uint32), local_wf.astype(np.uint32), node_ids)


def make_decode_queue(wl: Workload, n_calls: int, seed: int = 0, running_per_instance: int = 4,
                      load: float = 0.6, locked: float = 0.3):
    """Seeded decode-side snapshot for the decode-stage scheduler (Section 5.4), drawn for the decode
    pool of `wl`: the first n_calls ready calls as the decode queue, a lock for a share of them, the time
    their KV cache is on the decode side, and per decode instance a few calls decoding now that together
    hold about `load` of the instance's KV capacity until some time within the next two seconds.
    Returns (calls, lock i32, ready_s f32, run_ptr u32[D+1], run_end f32, run_tok f32)."""
    rng = np.random.default_rng([seed, 17, n_calls])
    D = wl.D
    calls = wl.calls[:n_calls].copy()
    lock = np.where(rng.random(n_calls) < locked, rng.integers(0, D, n_calls), -1).astype(np.int32)
    ready = np.where(rng.random(n_calls) < 0.5, 0.0, rng.uniform(0.0, 0.5, n_calls)).astype(np.float32)
    cap = wl.kv_cap[wl.P:]
    ptr, end, tok = [0], [], []
    for d in range(D):
        share = rng.dirichlet(np.ones(running_per_instance)) * load * cap[d]
        for s in share:
            end.append(rng.uniform(0.05, 2.0)); tok.append(np.floor(s))
        ptr.append(len(end))
    return (calls, lock, ready, np.array(ptr, np.uint32), np.array(end, np.float32), np.array(tok, np.float32))
