"""Pins for the CPU oracle's recursive (max-plus / min-plus) evaluation.

Every expected value here comes from a worked example, a closed form or an
independent textbook routine in tests/helpers.py, never from the oracle itself.
"""
import numpy as np
import pytest

import oracle
from paper_2609_27203_b200 import synth, workloads as W
from tests import helpers as H

MODES = ("naive", "seminaive")


def run(program, mode, **kw):
    o, ids, rules = oracle.load_program(program)
    stats = o.run(mode, **kw)
    return o, ids, stats


def f32_fold(ws):
    t = np.float32(ws[0])
    for w in ws[1:]:
        t = np.float32(t + np.float32(w))
    return t


@pytest.mark.parametrize("mode", MODES)
def test_listing1_chain_golden(mode):
    g = H.read_golden("listing1_chain_maxplus.txt")
    e, c = g["edges"], g["closure"]
    o, ids, stats = run(W.closure_program(e[:, 0], e[:, 1], e[:, 2]), mode)
    cols, tags = o.read(ids["path"])
    H.compare_relations((cols, tags), ([c[:, 0], c[:, 1]], c[:, 2]), what="listing 1")
    assert stats["derived_tuples"] == 6
    # the query ?- reach(1, N)
    assert sorted(int(y) for x, y in zip(*cols) if x == 1) == [2, 3, 4]


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("n", [2, 5, 33])
def test_chain_closed_form(mode, n):
    w = synth.log_prob_tags(n - 1, 7)
    o, ids, _ = run(W.closure_program(np.arange(n - 1), np.arange(1, n), w), mode)
    cols, tags = o.read(ids["path"])
    assert len(tags) == n * (n - 1) // 2
    got = H.relation_dict(cols, tags)
    for i in range(n):
        for j in range(i + 1, n):
            assert got[(i, j)].tobytes() == f32_fold(w[i:j]).tobytes()


@pytest.mark.parametrize("mode", MODES)
def test_complete_dag_unit_weights_maxplus(mode):
    # i -> j for i < j, weight +1: the best (longest) path i..j visits every node between,
    # so tag(i,j) = j - i, reached only after j-i-1 successive improvements of the same tuple.
    n = 12
    s, d = np.triu_indices(n, 1)
    o, ids, stats = run(W.closure_program(s, d, np.ones(len(s), np.float32)), mode)
    cols, tags = o.read(ids["path"])
    assert len(tags) == len(s)                                   # closure == edge set
    assert np.array_equal(tags, (cols[1] - cols[0]).astype(np.float32))


@pytest.mark.parametrize("mode", MODES)
def test_directed_cycle_has_n_squared_tuples(mode):
    n = 9
    o, ids, _ = run(W.closure_program(np.arange(n), (np.arange(n) + 1) % n, -np.ones(n, np.float32)), mode)
    cols, tags = o.read(ids["path"])
    assert len(tags) == n * n
    got = H.relation_dict(cols, tags)
    for x in range(n):
        for y in range(n):
            assert got[(x, y)] == -float(((y - x - 1) % n) + 1)


@pytest.mark.parametrize("mode", MODES)
def test_cycle3_golden(mode):
    g = H.read_golden("cycle3_maxplus.txt")
    e, c = g["edges"], g["closure"]
    o, ids, _ = run(W.closure_program(e[:, 0], e[:, 1], e[:, 2]), mode)
    H.compare_relations(o.read(ids["path"]), ([c[:, 0], c[:, 1]], c[:, 2]), what="3-cycle")


def test_diamond_golden_and_delta_sequence():
    g = H.read_golden("diamond_sssp_minplus.txt")
    e, dist = g["edges"], g["dist"]
    for mode in MODES:
        o, ids, _ = run(W.sssp_program(e[:, 0], e[:, 1], e[:, 2], 0), mode)
        H.compare_relations(o.read(ids["dist"]), ([dist[:, 0]], dist[:, 1]), what="diamond")
    assert o.delta_trace() == [int(x) for x in g["delta"][0]]


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_tuple_set_equals_bfs_reachability(seed):
    n, m = 40, 90
    s, d = synth.uniform_digraph(n, m, seed)
    want = H.reachable_pairs(n, s, d)
    for mode in MODES:
        o, ids, _ = run(W.closure_program(s, d, synth.log_prob_tags(m, seed)), mode)
        cols, _t = o.read(ids["path"])
        assert set(zip(cols[0].tolist(), cols[1].tolist())) == want


@pytest.mark.parametrize("semiring,maximize", [(W.MAXPLUS, True), (W.MINPLUS, False)])
def test_floyd_warshall_fp64(semiring, maximize):
    n, m = 48, 200
    s, d = synth.uniform_digraph(n, m, 11)
    w = synth.log_prob_tags(m, 11) if maximize else (1 + 9 * synth.uniform01(11, 9, 0, m)).astype(np.float32)
    D = H.floyd_warshall(n, s, d, w.astype(np.float64), maximize)
    for mode in MODES:
        o, ids, _ = run(W.closure_program(s, d, w, semiring), mode)
        cols, tags = o.read(ids["path"])
        assert len(tags) == int(np.isfinite(D).sum())
        ref = D[cols[0], cols[1]]
        assert np.all(np.abs(tags - ref) <= 1e-5 * np.abs(ref))


@pytest.mark.parametrize("maximize", [True, False])
def test_brute_force_paths_tiny(maximize):
    n, m = 6, 14
    s, d = synth.uniform_digraph(n, m, 5)
    w = synth.log_prob_tags(m, 5) if maximize else (1 + 9 * synth.uniform01(5, 9, 0, m)).astype(np.float32)
    want = H.best_simple_paths_f32(n, s, d, w, maximize)
    for mode in MODES:
        o, ids, _ = run(W.closure_program(s, d, w, W.MAXPLUS if maximize else W.MINPLUS), mode)
        got = H.relation_dict(*o.read(ids["path"]))
        assert set(got) == set(want)
        for k in want:
            assert got[k].tobytes() == np.float32(want[k]).tobytes(), k


@pytest.mark.parametrize("scale", [6, 10])
def test_sssp_bit_equals_dijkstra_fp32(scale):
    p = W.config2(scale=scale)
    (s, d), w = p.facts["edge"]
    n = 1 << scale
    off, dd, ww = H.csr(n, s, d, w)
    ref = H.dijkstra_f32(n, off, dd, ww, 0)
    for mode in MODES:
        o, ids, stats = run(p, mode)
        cols, tags = o.read(ids["dist"])
        reach = np.flatnonzero(np.isfinite(ref))
        assert np.array_equal(cols[0], reach)
        assert tags.tobytes() == ref[reach].tobytes()
        assert stats["derived_tuples"] == len(reach) - 1


def test_multi_source_reach_bit_equals_dijkstra_fp32():
    p = W.config5(scale=9, n_sources=6)
    (s, d), w = p.facts["edge"]
    n = 1 << 9
    off, dd, ww = H.csr(n, s, d, w)
    srcs = p.facts["src"][0][0]
    want_keys, want_tags = [], []
    for sidx in srcs:
        ref = H.dijkstra_f32(n, off, dd, ww, int(sidx))
        for y in np.flatnonzero(np.isfinite(ref)):
            want_keys.append((int(sidx), int(y)))
            want_tags.append(ref[y])
    for mode in MODES:
        o, ids, _ = run(p, mode)
        cols, tags = o.read(ids["reach"])
        assert list(zip(cols[0].tolist(), cols[1].tolist())) == want_keys
        assert tags.tobytes() == np.asarray(want_tags, np.float32).tobytes()


def test_naive_equals_seminaive_on_random_graphs():
    for seed, (n, m) in enumerate([(30, 60), (60, 200), (100, 150)]):
        s, d = synth.uniform_digraph(n, m, 100 + seed)
        t = synth.log_prob_tags(m, 100 + seed)
        a, ia, _ = run(W.closure_program(s, d, t), "naive")
        b, ib, _ = run(W.closure_program(s, d, t), "seminaive")
        rep = H.compare_relations(a.read(ia["path"]), b.read(ib["path"]))
        assert rep["bit_unequal"] == 0


def test_naive_equals_seminaive_on_random_programs():
    # the two evaluation orders share only the rule enumeration: non-linear and mutual recursion, negation over a finished
    # stratum, loaded facts in derived relations, the cyclic joins, aggregates (same tuples; max/min tags bit-equal)
    from tests.random_programs import random_program
    for seed in range(60):
        p = random_program(seed)
        a, ia, _ = run(p, "naive")
        b, ib, _ = run(p, "seminaive")
        for name in p.outputs:
            rep = H.compare_relations(a.read(ia[name]), b.read(ib[name]), abs_tol=1e-6, what=f"{p.name}:{name}")
            if p.relations[name][1] in (W.MAXPLUS, W.MINPLUS):
                assert rep["bit_unequal"] == 0


def test_fixpoint_is_idempotent_and_stable_under_one_more_round():
    p = W.config1(n_nodes=60, n_edges=180)
    o, ids, _ = run(p, "seminaive")
    first = o.read(ids["path"])
    for mode in MODES:                      # running again from the fixpoint derives nothing
        stats = o.run(mode)
        again = o.read(ids["path"])
        assert H.compare_relations(again, first)["bit_unequal"] == 0
    assert o.delta_trace() == [0]


def test_duplicate_facts_combine_with_oplus():
    o = oracle.Oracle()
    r = o.relation(2, "minplus")
    o.load(r, [np.array([3, 1, 3, 1]), np.array([4, 2, 4, 2])], np.array([5.0, 2.0, 3.0, 9.0], np.float32))
    cols, tags = o.read(r)
    assert cols[0].tolist() == [1, 3] and cols[1].tolist() == [2, 4] and tags.tolist() == [2.0, 3.0]
    r2 = o.relation(1, "logsumexp")
    o.load(r2, [np.array([7, 7])], np.array([0.0, 0.0], np.float32))
    assert abs(o.read(r2)[1][0] - np.log(2.0)) < 1e-7


def test_typed_failures():
    # iteration cap on a chain: needs n-1 rounds
    p = W.closure_program(np.arange(9), np.arange(1, 10), -np.ones(9, np.float32))
    for mode in MODES:
        o, ids, _r = oracle.load_program(p)
        with pytest.raises(oracle.OracleError) as e:
            o.run(mode, max_iterations=3)
        assert e.value.status == "CONVERGENCE_FAILURE"
    # a recursive component that mixes max/min relations with logsumexp relations is rejected
    mixed = W.Program("mixed", {"e": (1, W.MAXPLUS), "a": (1, W.MAXPLUS), "b": (1, W.LOGSUMEXP)},
                      [W.Rule("a", (W.V(0),), (W.Atom("e", (W.Var(0),)),)), W.Rule("a", (W.V(0),), (W.Atom("b", (W.Var(0),)),)),
                       W.Rule("b", (W.V(0),), (W.Atom("a", (W.Var(0),)),))], {"e": ([np.array([1, 2], np.int32)], None)})
    o, ids, _r = oracle.load_program(mixed)
    with pytest.raises(oracle.OracleError) as e:
        o.run("naive")
    assert e.value.status == "UNSUPPORTED"
    # NaN tag and negative key are rejected at load
    o = oracle.Oracle()
    r = o.relation(1, "maxplus")
    with pytest.raises(oracle.OracleError):
        o.load(r, [np.array([1])], np.array([np.nan], np.float32))
    with pytest.raises(oracle.OracleError):
        o.load(r, [np.array([-1])], None)
    # head expression leaving [0, 2^31) is an error, never a wrap
    prog = W.Program("ovf", {"a": (1, W.MAXPLUS), "b": (1, W.MAXPLUS)},
                     [W.Rule("b", (W.Affine(0, ((0, 2),)),), (W.Atom("a", (W.Var(0),)),))],
                     {"a": ([np.array([1 << 30], np.int32)], None)})
    o, ids, _r = oracle.load_program(prog)
    with pytest.raises(oracle.OracleError) as e:
        o.run("naive")
    assert e.value.status == "CAPACITY_EXCEEDED"
