"""Shared plumbing of the GPU parity tests: run the same seeded workload through
the CPU oracle and through the CUDA library (via its C ABI binding) and compare."""
import numpy as np

from oracle import hx_oracle as ho

REL_TOL = 1e-5      # bar on binary32 costs: relative difference GPU vs oracle


def oracle_cluster(wl):
    return ho.Cluster.from_workload(wl)


def gpu_cluster(wl):
    import paper_2605_16637_b200 as hx
    return hx.Cluster.from_workload(wl)


def gpu_node_costs(gc, calls):
    """Unloaded best latency of every given call (stand-alone service time)."""
    import paper_2605_16637_b200 as hx
    gc.set_options(score_mode=hx.HX_MODE_COMPLETION, flags=hx.HX_FLAG_UNLOADED | hx.HX_FLAG_NO_DAG)
    _, cost = gc.schedule_batch(calls)
    return cost.cpu().numpy()


def oracle_node_costs(orc, oc, calls):
    return orc.schedule(oc, calls, flags=ho.FLAG_UNLOADED | ho.FLAG_NO_DAG)[2]


def rel_err(got, want):
    got = np.asarray(got, np.float64); want = np.asarray(want, np.float64)
    same_inf = np.isinf(got) & np.isinf(want) & (np.sign(got) == np.sign(want))
    denom = np.where(np.abs(want) > 0, np.abs(want), 1.0)
    with np.errstate(invalid="ignore"):
        err = np.abs(got - want) / denom
    return np.where(same_inf, 0.0, err)


def assert_costs_close(got, want, what=""):
    err = rel_err(got, want)
    assert not np.isnan(err).any(), what
    assert err.max(initial=0.0) <= REL_TOL, "%s: max rel err %.3g" % (what, err.max())


def assert_assign_matches(orc, oc, calls, got_assign, want_assign, flags=0, what=""):
    """Identical pairs, except where the oracle's own cost gap between its best pair and
    the pair the GPU chose is below the tolerance.  Returns the number of excused calls."""
    got_assign = np.asarray(got_assign); want_assign = np.asarray(want_assign)
    bad = np.flatnonzero(got_assign != want_assign)
    if bad.size == 0:
        return 0
    fin = orc.fin_all(oc, calls[bad], flags=flags).reshape(bad.size, -1)
    for i, c in enumerate(bad):
        g, w = got_assign[c], want_assign[c]
        assert g >= 0 and w >= 0, "%s: call %d feasibility differs (%d vs %d)" % (what, c, g, w)
        gap = abs(float(fin[i, g]) - float(fin[i, w])) / float(fin[i, w])
        assert gap < REL_TOL, "%s: call %d got pair %d (%.9g), oracle %d (%.9g)" % (
            what, c, g, fin[i, g], w, fin[i, w])
    return int(bad.size)
