"""Recursion under a non-idempotent oplus (sum / logsumexp) on derivation DAGs, CUDA path against the CPU oracle.
Tuple sets exact; path counts exact while below 2^24 (integers in fp32); weighted sums 1e-5 relative (each round's sums are
taken in fp64 and rounded to fp32, as in the oracle's delta form); logsumexp tags 1e-4 absolute."""
import math

import numpy as np
import pytest

import oracle
from paper_2609_27203_b200 import synth, workloads as W
from tests import helpers as H

pytestmark = pytest.mark.gpu


def both(program, mode="seminaive", **kw):
    from paper_2609_27203_b200 import xlog
    kw.setdefault("arena_bytes", 1 << 28)
    kw.setdefault("flags", xlog.FLAG_CHECK_INVARIANTS)
    ctx, gids, _ = xlog.load_program(program, **kw)
    receipt = ctx.fixpoint()
    o, oids, _ = oracle.load_program(program)
    stats = o.run(mode)
    return ctx, gids, o, oids, receipt, stats


def dag_edges(n, m, seed):
    a, b = synth.uniform_digraph(n, m, seed)
    s, d = np.minimum(a, b), np.maximum(a, b)                 # u < v only: acyclic
    key = np.unique(s.astype(np.int64) * n + d)
    return (key // n).astype(np.int32), (key % n).astype(np.int32)


def test_complete_dag_path_counts_are_powers_of_two():
    n = 20
    s, d = np.triu_indices(n, 1)
    prog = W.closure_program(s, d, None, W.SUMPROD, name="complete_dag")
    ctx, gids, o, oids, receipt, stats = both(prog)
    cols, tags = ctx.read(gids["path"])
    assert tags.tolist() == [float(2 ** (j - i - 1)) for i, j in zip(cols[0], cols[1])]
    rep = H.compare_relations((cols, tags), o.read(oids["path"]), what="complete dag")
    assert rep["bit_unequal"] == 0 and receipt["derived_tuples"] == stats["derived_tuples"] == n * (n - 1) // 2
    assert receipt["iterations"] == stats["iterations"] == n
    # evaluated again: recomputed from the facts, not added a second time
    again = ctx.fixpoint()
    assert np.array_equal(ctx.read(gids["path"])[1], tags) and again["derived_tuples"] == receipt["derived_tuples"]
    ctx.close()


def test_grid_dag_single_source_counts_are_binomials():
    R, C = 9, 12
    s, d = [], []
    for r in range(R):
        for c in range(C):
            if c + 1 < C:
                s.append(r * C + c); d.append(r * C + c + 1)
            if r + 1 < R:
                s.append(r * C + c); d.append((r + 1) * C + c)
    prog = W.sssp_program(np.array(s), np.array(d), np.ones(len(s), np.float32), source=0, semiring=W.SUMPROD, name="grid")
    prog.facts["dist"] = ([np.array([0], np.int32)], np.ones(1, np.float32))
    ctx, gids, o, oids, _, _ = both(prog)
    cols, tags = ctx.read(gids["dist"])
    assert cols[0].tolist() == list(range(R * C))
    assert tags.tolist() == [float(math.comb(r + c, r)) for r in range(R) for c in range(C)]
    assert H.compare_relations((cols, tags), o.read(oids["dist"]), what="grid")["bit_unequal"] == 0
    ctx.close()


@pytest.mark.parametrize("n,m,seed", [(40, 160, 1), (400, 1300, 2), (3000, 7000, 3)])
def test_random_dag_counts_weights_and_log_space(n, m, seed):
    s, d = dag_edges(n, m, seed)
    # counts: exact (the oracle's delta form rounds at the same places; checked below 2^24)
    ctx, gids, o, oids, receipt, stats = both(W.closure_program(s, d, None, W.SUMPROD, name="dag_counts"))
    got, want = ctx.read(gids["path"]), o.read(oids["path"])
    assert want[1].max() < 2 ** 24
    assert H.compare_relations(got, want, what="dag counts")["bit_unequal"] == 0
    assert receipt["derived_tuples"] == stats["derived_tuples"]
    ctx.close()
    # weighted sums of path products
    w = (0.25 + synth.uniform01(seed, 3, 0, len(s))).astype(np.float32)
    ctx, gids, o, oids, _, _ = both(W.closure_program(s, d, w, W.SUMPROD, name="dag_weighted"))
    H.compare_relations(ctx.read(gids["path"]), o.read(oids["path"]), rel_tol=1e-5, what="dag weighted")
    ctx.close()
    # log space
    ctx, gids, o, oids, _, _ = both(W.closure_program(s, d, np.log(w.astype(np.float64)).astype(np.float32), W.LOGSUMEXP, name="dag_lse"))
    H.compare_relations(ctx.read(gids["path"]), o.read(oids["path"]), abs_tol=1e-4, what="dag logsumexp")
    ctx.close()


def test_rmat_derived_dag_against_the_naive_oracle_and_numpy():
    # an R-MAT graph with every edge turned to point from the smaller to the larger id; single-source path counts
    p5 = W.config5(scale=9, n_sources=1)
    (a, b), _ = p5.facts["edge"]
    n = 1 << 9
    key = np.unique(np.minimum(a, b).astype(np.int64) * n + np.maximum(a, b))
    s, d = (key // n).astype(np.int32), (key % n).astype(np.int32)
    w = (0.05 + 0.2 * synth.uniform01(9, 3, 0, len(s))).astype(np.float32)
    prog = W.sssp_program(s, d, w, source=0, semiring=W.SUMPROD, name="rmat_dag")
    prog.facts["dist"] = ([np.array([0], np.int32)], np.ones(1, np.float32))
    ctx, gids, o, oids, _, _ = both(prog, mode="naive")
    got = ctx.read(gids["dist"])
    H.compare_relations(got, o.read(oids["dist"]), rel_tol=1e-5, what="rmat dag vs naive oracle")
    Wm = np.zeros((n, n))
    Wm[s, d] = w
    x = np.zeros(n); x[0] = 1.0
    total, cur = x.copy(), x
    for _ in range(n):
        cur = cur @ Wm
        total += cur
    nz = np.flatnonzero(total)
    assert got[0][0].tolist() == nz.tolist() and np.allclose(got[1], total[nz], rtol=1e-5)
    ctx.close()


def test_mutually_recursive_sum_relations():
    # even(y) :- odd(x), e(x,y).  odd(y) :- even(x), e(x,y).  even(0) = 1: walks of even / odd length from node 0
    n = 60
    s, d = dag_edges(n, 240, 7)
    prog = W.Program("parity", {"e": (2, W.SUMPROD), "even": (1, W.SUMPROD), "odd": (1, W.SUMPROD)},
                     [W.Rule("even", (W.V(1),), (W.Atom("odd", (W.Var(0),)), W.Atom("e", (W.Var(0), W.Var(1))))),
                      W.Rule("odd", (W.V(1),), (W.Atom("even", (W.Var(0),)), W.Atom("e", (W.Var(0), W.Var(1)))))],
                     {"e": ([s, d], None), "even": ([np.array([0], np.int32)], np.ones(1, np.float32))}, ("even", "odd"))
    ctx, gids, o, oids, _, _ = both(prog)
    A = np.zeros((n, n), np.int64)
    A[s, d] = 1
    x = np.zeros(n, np.int64); x[0] = 1
    ev, od, cur = x.copy(), np.zeros(n, np.int64), x
    for k in range(1, n + 1):
        cur = cur @ A
        if k % 2:
            od += cur
        else:
            ev += cur
    for name, ref in (("even", ev), ("odd", od)):
        cols, tags = ctx.read(gids[name])
        assert cols[0].tolist() == np.flatnonzero(ref).tolist() and tags.tolist() == ref[ref > 0].astype(np.float32).tolist()
        assert H.compare_relations((cols, tags), o.read(oids[name]), what=name)["bit_unequal"] == 0
    ctx.close()


@pytest.mark.parametrize("sr", [W.SUMPROD, W.LOGSUMEXP])
def test_cycle_ends_at_the_iteration_cap(sr):
    from paper_2609_27203_b200 import xlog
    ctx, ids, _ = xlog.load_program(W.closure_program([0, 1, 2, 5], [1, 2, 0, 0], None, sr), arena_bytes=1 << 26, max_iterations=40)
    with pytest.raises(xlog.XlogError) as e:
        ctx.fixpoint()
    assert e.value.status == "CONVERGENCE_FAILURE"
    with pytest.raises(xlog.XlogError) as e:
        ctx.read(ids["path"])
    assert e.value.status == "INVALID_STATE"
    ctx.reset_idb()
    assert ctx.size(ids["path"]) == 0
    ctx.close()
