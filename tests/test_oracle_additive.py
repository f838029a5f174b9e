"""Pins for recursion under a non-idempotent oplus (sum / logsumexp) on derivation DAGs: the tag of a tuple is the
oplus over ALL of its derivations.  Expected values are closed forms (powers of two on the complete DAG, binomials on a
grid, Catalan numbers for the non-linear rule) and numpy int64 / float64 matrix powers, never the oracle's own output."""
import math

import numpy as np
import pytest

import oracle
from paper_2609_27203_b200 import synth, workloads as W

MODES = ["naive", "seminaive"]


def paths_program(src, dst, tag, sr, name="paths"):
    """paths(x,y) :- edge(x,y).  paths(x,z) :- paths(x,y), edge(y,z)."""
    return W.closure_program(src, dst, tag, sr, name=name)


def run(program, mode, **kw):
    o, ids, _ = oracle.load_program(program)
    st = o.run(mode, **kw)
    return o, ids, st


def walk_sums(n, src, dst, w):
    """sum over k >= 1 of W^k in float64 (the graph must be acyclic: W is nilpotent)."""
    Wm = np.zeros((n, n))
    Wm[src, dst] = w
    total, P = np.zeros((n, n)), Wm.copy()
    for _ in range(n):
        total += P
        P = P @ Wm
    assert not P.any()
    return total


@pytest.mark.parametrize("mode", MODES)
def test_complete_dag_has_two_to_the_gap_minus_one_paths(mode):
    n = 14
    s, d = np.triu_indices(n, 1)
    o, ids, st = run(paths_program(s, d, None, W.SUMPROD), mode)
    cols, tags = o.read(ids["path"])
    assert len(tags) == n * (n - 1) // 2
    assert tags.tolist() == [float(2 ** (j - i - 1)) for i, j in zip(cols[0], cols[1])]
    # the longest path has n - 1 edges: the delta form needs n - 1 productive rounds and one that derives nothing,
    # the naive form one more round to see that nothing changed
    assert st["iterations"] == n


@pytest.mark.parametrize("mode", MODES)
def test_grid_dag_counts_are_binomials_from_a_single_source(mode):
    # cnt(y) :- cnt(x), edge(x,y) with cnt(origin) = 1: monotone lattice paths, C(r + c, r) of them to cell (r, c)
    R, C = 7, 9
    idx = lambda r, c: r * C + c
    s, d = [], []
    for r in range(R):
        for c in range(C):
            if c + 1 < C:
                s.append(idx(r, c)); d.append(idx(r, c + 1))
            if r + 1 < R:
                s.append(idx(r, c)); d.append(idx(r + 1, c))
    prog = W.sssp_program(np.array(s), np.array(d), np.ones(len(s), np.float32), source=0, semiring=W.SUMPROD)
    prog.facts["dist"] = ([np.array([0], np.int32)], np.ones(1, np.float32))
    o, ids, _ = run(prog, mode)
    cols, tags = o.read(ids["dist"])
    assert cols[0].tolist() == list(range(R * C))
    assert tags.tolist() == [float(math.comb(r + c, r)) for r in range(R) for c in range(C)]


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("seed", [1, 2])
def test_random_dag_counts_equal_the_sum_of_adjacency_powers(mode, seed):
    n = 40
    a, b = synth.uniform_digraph(n, 160, seed)
    s, d = np.minimum(a, b), np.maximum(a, b)                 # edges u < v only: acyclic
    key = np.unique(s.astype(np.int64) * n + d)
    s, d = (key // n).astype(np.int32), (key % n).astype(np.int32)
    A = np.zeros((n, n), np.int64)
    A[s, d] = 1
    total, P = np.zeros((n, n), np.int64), A.copy()
    while P.any():
        total += P
        P = P @ A
    assert total.max() < 2 ** 24                                # exact in fp32
    o, ids, _ = run(paths_program(s, d, None, W.SUMPROD), mode)
    cols, tags = o.read(ids["path"])
    xs, zs = np.nonzero(total)
    assert cols[0].tolist() == xs.tolist() and cols[1].tolist() == zs.tolist()
    assert tags.tolist() == total[xs, zs].astype(np.float32).tolist()


@pytest.mark.parametrize("mode", MODES)
def test_weighted_path_sums_and_log_space(mode):
    n = 30
    a, b = synth.uniform_digraph(n, 110, 5)
    s, d = np.minimum(a, b), np.maximum(a, b)
    key = np.unique(s.astype(np.int64) * n + d)
    s, d = (key // n).astype(np.int32), (key % n).astype(np.int32)
    w = (0.25 + synth.uniform01(5, 3, 0, len(s))).astype(np.float32)
    ref = walk_sums(n, s, d, w.astype(np.float64))
    xs, zs = np.nonzero(ref)
    o, ids, _ = run(paths_program(s, d, w, W.SUMPROD), mode)
    cols, tags = o.read(ids["path"])
    assert cols[0].tolist() == xs.tolist() and cols[1].tolist() == zs.tolist()
    assert np.allclose(tags, ref[xs, zs], rtol=2e-6, atol=0)
    # the same sums in log space: tags log w, oplus = logaddexp, otimes = +
    o, ids, _ = run(paths_program(s, d, np.log(w.astype(np.float64)).astype(np.float32), W.LOGSUMEXP), mode)
    cols, tags = o.read(ids["path"])
    assert cols[0].tolist() == xs.tolist() and cols[1].tolist() == zs.tolist()
    assert np.all(np.abs(tags - np.log(ref[xs, zs])) < 1e-5)
    # zero log-weights: logsumexp counts, ln(number of paths)
    o, ids, _ = run(paths_program(s, d, np.zeros(len(s), np.float32), W.LOGSUMEXP), mode)
    cnt = walk_sums(n, s, d, np.ones(len(s)))
    assert np.all(np.abs(o.read(ids["path"])[1] - np.log(cnt[xs, zs])) < 1e-5)


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("sr", [W.SUMPROD, W.LOGSUMEXP])
def test_a_cycle_never_converges(mode, sr):
    with pytest.raises(oracle.OracleError) as e:
        run(paths_program([0, 1, 2, 5], [1, 2, 0, 0], None, sr), mode, max_iterations=40)
    assert e.value.status == "CONVERGENCE_FAILURE"


def test_non_linear_rule_counts_bracketings_in_naive_mode_only():
    # p(x,y) :- e(x,y).  p(x,z) :- p(x,y), p(y,z): a path of L edges has Catalan(L - 1) derivation trees
    L = 7
    prog = W.Program("brackets", {"e": (2, W.SUMPROD), "p": (2, W.SUMPROD)},
                     [W.Rule("p", (W.V(0), W.V(1)), (W.Atom("e", (W.Var(0), W.Var(1))),)),
                      W.Rule("p", (W.V(0), W.V(2)), (W.Atom("p", (W.Var(0), W.Var(1))), W.Atom("p", (W.Var(1), W.Var(2)))))],
                     {"e": ([np.arange(L, dtype=np.int32), np.arange(1, L + 1, dtype=np.int32)], None)})
    o, ids, _ = run(prog, "naive")
    cols, tags = o.read(ids["p"])
    catalan = lambda k: math.comb(2 * k, k) // (k + 1)
    assert tags.tolist() == [float(catalan(j - i - 1)) for i, j in zip(cols[0], cols[1])]
    with pytest.raises(oracle.OracleError) as e:
        run(prog, "seminaive")
    assert e.value.status == "UNSUPPORTED"


def test_rerunning_recomputes_instead_of_adding_again():
    n = 8
    s, d = np.triu_indices(n, 1)
    o, ids, _ = oracle.load_program(paths_program(s, d, None, W.SUMPROD))
    o.run("seminaive")
    first = o.read(ids["path"])[1].copy()
    o.run("seminaive")
    assert np.array_equal(first, o.read(ids["path"])[1])
    o.run("naive")
    assert np.array_equal(first, o.read(ids["path"])[1])
