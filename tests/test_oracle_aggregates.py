"""Pins for the CPU oracle's non-recursive aggregates: count, logsumexp, sum, and the
gradient of a logsumexp rule.  Expected values come from worked examples, closed forms,
brute force and library routines (numpy / torch on CPU), never from the oracle."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2609_27203_b200 import synth, workloads as W
from tests import helpers as H


def run(program, mode="naive"):
    o, ids, rules = oracle.load_program(program)
    o.run(mode)
    return o, ids, rules


def degree_program(src, dst):
    return W.Program("degree", {"edge": (2, W.SUMPROD), "degree": (2, W.SUMPROD)},
                     [W.Rule("degree", (W.V(0),), (W.Atom("edge", (W.Var(0), W.Var(1))),), emit_count=True)],
                     {"edge": ([np.asarray(src, np.int32), np.asarray(dst, np.int32)], None)})


def test_listing7_degree_golden():
    g = H.read_golden("listing7_degree_count.txt")
    o, ids, _ = run(degree_program(g["edges"][:, 0], g["edges"][:, 1]))
    cols, tags = o.read(ids["degree"])
    assert cols[0].tolist() == g["degree"][:, 0].tolist()
    assert cols[1].tolist() == g["degree"][:, 1].tolist()
    assert tags.tolist() == [3.0, 1.0]          # sum of unit tags == count


def test_k3_triangle_golden():
    g = H.read_golden("k3_triangle_lse.txt")
    e, t = g["edges"], g["tri_agg"]
    o, ids, _ = run(W.triangle_program(e[:, 0], e[:, 1], e[:, 2]))
    cols, tags = o.read(ids["tri_agg"])
    assert cols[0].tolist() == [0, 1, 2] and cols[1].tolist() == [2, 2, 2]
    assert np.allclose(tags, t[:, 2], atol=1e-6)
    assert np.allclose(tags, math.log(math.exp(0.875) + math.exp(-1.75)), atol=1e-6)


@pytest.mark.parametrize("n", [3, 4, 7])
def test_complete_digraph_triangle_counts(n):
    s, d = np.nonzero(~np.eye(n, dtype=bool))
    o, ids, _ = run(W.triangle_program(s, d, np.zeros(len(s), np.float32)))
    cols, tags = o.read(ids["tri_agg"])
    assert cols[0].tolist() == list(range(n))
    assert cols[1].tolist() == [(n - 1) * (n - 2)] * n
    # all weights zero: logsumexp is exactly ln(count)
    assert np.allclose(tags, math.log((n - 1) * (n - 2)), atol=1e-6)


@pytest.mark.parametrize("scale", [5, 7])
def test_triangles_trace_and_brute_force(scale):
    p = W.config3(scale=scale)
    (s, d), w = p.facts["e"]
    n = 1 << scale
    A = np.zeros((n, n), np.int64)
    A[s, d] = 1
    Wm = np.full((n, n), np.nan)
    Wm[s, d] = w.astype(np.float64)
    o, ids, _ = run(p)
    cols, tags = o.read(ids["tri_agg"])
    assert int(cols[1].sum()) == int(np.trace(A @ A @ A))
    assert int(cols[1].sum()) % 3 == 0
    # O(n^3) brute force per x
    cnt = np.zeros(n, np.int64)
    terms = [[] for _ in range(n)]
    for x in range(n):
        for y in np.flatnonzero(A[x]):
            for z in np.flatnonzero(A[y]):
                if A[z, x]:
                    cnt[x] += 1
                    terms[x].append((Wm[x, y] + Wm[y, z]) + Wm[z, x])
    xs = np.flatnonzero(cnt)
    assert cols[0].tolist() == xs.tolist()
    assert cols[1].tolist() == cnt[xs].tolist()
    ref = np.array([torch.logsumexp(torch.tensor(terms[x], dtype=torch.float64), 0).item() for x in xs])
    assert np.all(np.abs(tags - ref) < 1e-5)


def test_single_term_group_passes_through_bit_exactly():
    # one directed 3-cycle: each x has exactly one term, (w1+w2)+w3 in rotated order
    w = np.array([0.1, 0.2, 0.7], np.float32)
    o, ids, _ = run(W.triangle_program([0, 1, 2], [1, 2, 0], w))
    cols, tags = o.read(ids["tri_agg"])
    assert cols[1].tolist() == [1, 1, 1]
    for x in range(3):
        t = (float(w[x]) + float(w[(x + 1) % 3])) + float(w[(x + 2) % 3])
        assert tags[x] == np.float32(t)


def test_sum_semiring_counts_paths():
    # SUMPROD with unit tags counts two-step walks: p2(x,z) :- e(x,y), e(y,z)
    s, d = synth.uniform_digraph(20, 80, 3)
    prog = W.Program("p2", {"e": (2, W.SUMPROD), "p2": (2, W.SUMPROD)},
                     [W.Rule("p2", (W.V(0), W.V(2)), (W.Atom("e", (W.Var(0), W.Var(1))), W.Atom("e", (W.Var(1), W.Var(2)))))],
                     {"e": ([s, d], None)})
    o, ids, _ = run(prog)
    cols, tags = o.read(ids["p2"])
    A = np.zeros((20, 20), np.int64)
    A[s, d] = 1
    A2 = A @ A
    xs, zs = np.nonzero(A2)
    assert cols[0].tolist() == xs.tolist() and cols[1].tolist() == zs.tolist()
    assert tags.tolist() == A2[xs, zs].astype(np.float32).tolist()


# ---- the digit-sum program (forward) ----------------------------------------------------

def conv_reference(lt):
    """log of the discrete convolution of the two softmax vectors of each pair, fp64."""
    P = np.exp(lt.astype(np.float64))
    B = lt.shape[0] // 2
    out = np.zeros((B, 19))
    for p in range(B):
        out[p] = np.convolve(P[2 * p], P[2 * p + 1])
    return np.log(out)


@pytest.mark.parametrize("B", [1, 16, 200])
def test_digit_sum_forward_is_log_convolution(B):
    lt = synth.digit_log_tags(2 * B, 44)
    o, ids, _ = run(W.digits_program(lt))
    cols, tags = o.read(ids["sum"])
    assert len(tags) == 19 * B
    assert np.array_equal(cols[0], np.repeat(np.arange(B), 19)) and np.array_equal(cols[1], np.tile(np.arange(19), B))
    ref = conv_reference(lt).reshape(-1)
    assert np.all(np.abs(tags - ref) < 1e-5)
    # the nineteen sums of one pair are exhaustive and exclusive: probabilities add to one
    tot = torch.logsumexp(torch.tensor(tags.reshape(B, 19), dtype=torch.float64), 1).numpy()
    assert np.all(np.abs(tot) < 1e-5)


def test_digit_sum_near_one_hot_puts_mass_at_a_plus_b():
    lt = np.full((2, 10), -40.0, np.float32)
    lt[0, 3] = 0.0
    lt[1, 8] = 0.0
    o, ids, _ = run(W.digits_program(lt))
    cols, tags = o.read(ids["sum"])
    assert int(cols[1][np.argmax(tags)]) == 11 and abs(tags.max()) < 1e-6


def test_uniform_digits_golden_forward_and_gradient():
    g = H.read_golden("uniform_digits_lse.txt")
    B = 3
    lt = np.full((2 * B, 10), -math.log(10.0), np.float32)
    o, ids, rules = run(W.digits_program(lt))
    cols, tags = o.read(ids["sum"])
    for s_, v in g["out"]:
        s_ = int(s_)
        for s2 in (s_, 18 - s_):
            assert np.all(np.abs(tags[cols[1] == s2] - v) < 2e-6)
            assert abs(v - math.log((min(s2, 18 - s2) + 1) / 100.0)) < 1e-6
    grads = o.backward(rules[0], np.ones(len(tags), np.float32))
    total = (grads[0] + grads[1]).reshape(2 * B, 10)       # both atoms read `digit`
    for a, v in g["grad"]:
        assert np.all(np.abs(total[:, int(a)] - v) < 2e-6)
    assert np.allclose(total.sum(axis=1), 19.0, atol=1e-5)


# ---- gradient -------------------------------------------------------------------------

def test_backward_matches_torch_autograd_and_finite_differences():
    B = 5
    lt = synth.digit_log_tags(2 * B, 45)
    prog = W.digits_program(lt)
    o, ids, rules = run(prog)
    cols, tags = o.read(ids["sum"])
    g = synth.head_gradient(len(tags), 45)
    grads = o.backward(rules[0], g)
    total = (grads[0] + grads[1]).reshape(2 * B, 10).astype(np.float64)

    x = torch.tensor(lt.astype(np.float64), requires_grad=True)
    a = x[0::2].unsqueeze(2)                # [B,10,1]
    b = x[1::2].unsqueeze(1)                # [B,1,10]
    joint = a + b
    outs = []
    for s in range(19):
        idx = [(i, s - i) for i in range(10) if 0 <= s - i <= 9]
        outs.append(torch.logsumexp(torch.stack([joint[:, i, j] for i, j in idx], 1), 1))
    out = torch.stack(outs, 1)              # [B,19]
    assert np.allclose(out.detach().numpy().reshape(-1), tags, atol=1e-5)
    (out.reshape(-1) * torch.tensor(g.astype(np.float64))).sum().backward()
    assert np.all(np.abs(total - x.grad.numpy()) <= 1e-5 + 1e-4 * np.abs(x.grad.numpy()))

    # central finite differences on a few inputs, evaluating the loss through the fp64 convolution
    def loss(l):
        return float((conv_reference(l).reshape(-1) * g.astype(np.float64)).sum())
    base = lt.astype(np.float64)
    for (i, dgt) in [(0, 0), (3, 7), (9, 9)]:
        h = 1e-5
        up, dn = base.copy(), base.copy()
        up[i, dgt] += h
        dn[i, dgt] -= h
        fd = (loss(up) - loss(dn)) / (2 * h)
        assert abs(fd - total[i, dgt]) < 1e-4 * max(1.0, abs(fd))


def test_backward_softmax_weights_sum_to_one_per_head_row():
    # with g = e_h (one head row), the weights of all bindings of that row sum to 1,
    # so the gradient summed over the first atom's rows is exactly 1.
    B = 4
    lt = synth.digit_log_tags(2 * B, 46)
    o, ids, rules = run(W.digits_program(lt))
    n = o.size(ids["sum"])
    for h in (0, 9, 18, 19 * 3 + 5):
        g = np.zeros(n, np.float32)
        g[h] = 1.0
        grads = o.backward(rules[0], g)
        assert abs(float(grads[0].astype(np.float64).sum()) - 1.0) < 1e-5
        assert abs(float(grads[1].astype(np.float64).sum()) - 1.0) < 1e-5


def test_facts_of_a_derived_relation_are_one_more_contribution():
    # q(x) has a loaded fact and a derived contribution; logsumexp combines both
    prog = W.Program("mix", {"a": (1, W.LOGSUMEXP), "q": (1, W.LOGSUMEXP)},
                     [W.Rule("q", (W.V(0),), (W.Atom("a", (W.Var(0),)),))],
                     {"a": ([np.array([1, 2], np.int32)], np.array([0.0, -1.0], np.float32)),
                      "q": ([np.array([2, 5], np.int32)], np.array([-1.0, -3.0], np.float32))})
    o, ids, _ = run(prog)
    cols, tags = o.read(ids["q"])
    assert cols[0].tolist() == [1, 2, 5]
    assert np.allclose(tags, [0.0, -1.0 + math.log(2.0), -3.0], atol=1e-6)
    o.run("naive")                                  # evaluating again recomputes the same relation
    assert np.allclose(o.read(ids["q"])[1], tags, atol=0)


# ---- stratified negation ------------------------------------------------------------------

def test_negation_is_set_difference_and_wildcards_mean_exists():
    a = np.array([1, 2, 3, 5, 8, 13], np.int32)
    b = np.array([2, 3, 4, 13, 21], np.int32)
    prog = W.Program("diff", {"a": (1, W.MINPLUS), "b": (1, W.MINPLUS), "only_a": (1, W.MINPLUS)},
                     [W.Rule("only_a", (W.V(0),), (W.Atom("a", (W.Var(0),)), W.Atom("b", (W.Var(0),), negated=True)))],
                     {"a": ([a], np.arange(6, dtype=np.float32)), "b": ([b], None)}, ("only_a",))
    o, ids, _ = run(prog)
    cols, tags = o.read(ids["only_a"])
    keep = np.setdiff1d(a, b)
    assert cols[0].tolist() == keep.tolist()
    assert tags.tolist() == [float(np.flatnonzero(a == v)[0]) for v in keep]      # the negated atom adds nothing to the tag
    # paper Listing 7: the constraint  :- edge(X,_), not degree(X,_)  has no violation
    g = H.read_golden("listing7_degree_count.txt")
    e0, e1 = g["edges"][:, 0].astype(np.int32), g["edges"][:, 1].astype(np.int32)
    prog = W.Program("l7", {"edge": (2, W.SUMPROD), "degree": (2, W.SUMPROD), "viol": (1, W.SUMPROD)},
                     [W.Rule("degree", (W.V(0),), (W.Atom("edge", (W.Var(0), W.Var(1))),), emit_count=True),
                      W.Rule("viol", (W.V(0),), (W.Atom("edge", (W.Var(0), W.Var(1))), W.Atom("degree", (W.Var(0), W.Var(2)), negated=True)))],
                     {"edge": ([e0, e1], None)}, ("viol",))
    o, ids, _ = run(prog)
    assert o.size(ids["viol"]) == 0
    # and with a node that has an in-edge only, `sink(y) :- edge(x,y), not edge(y,_)` lists the sinks
    prog = W.Program("sinks", {"edge": (2, W.MAXPLUS), "sink": (1, W.MAXPLUS)},
                     [W.Rule("sink", (W.V(1),), (W.Atom("edge", (W.Var(0), W.Var(1))), W.Atom("edge", (W.Var(1), W.Var(2)), negated=True)))],
                     {"edge": ([e0, e1], None)}, ("sink",))
    o, ids, _ = run(prog)
    assert o.read(ids["sink"])[0][0].tolist() == sorted(set(e1.tolist()) - set(e0.tolist()))


def test_negation_over_a_recursive_lower_stratum():
    # unreached(x) :- node(x), not dist(x): everything the BFS from node 0 does not reach
    s, d = synth.uniform_digraph(80, 110, 17)
    w = np.ones(len(s), np.float32)
    prog = W.sssp_program(s, d, w, 0)
    prog.relations["node"] = (1, W.MINPLUS)
    prog.relations["unreached"] = (1, W.MINPLUS)
    prog.facts["node"] = ([np.arange(80, dtype=np.int32)], None)
    prog.rules.append(W.Rule("unreached", (W.V(0),), (W.Atom("node", (W.Var(0),)), W.Atom("dist", (W.Var(0),), negated=True))))
    for mode in ("naive", "seminaive"):
        o, ids, _ = run(prog, mode)
        reached = {0} | {y for (x, y) in H.reachable_pairs(80, s, d) if x == 0}
        assert o.read(ids["unreached"])[0][0].tolist() == sorted(set(range(80)) - reached)
    # negation through recursion is not stratified
    bad = W.Program("bad", {"e": (1, W.MINPLUS), "p": (1, W.MINPLUS)},
                    [W.Rule("p", (W.V(0),), (W.Atom("e", (W.Var(0),)), W.Atom("p", (W.Var(0),), negated=True)))],
                    {"e": ([np.array([1], np.int32)], None)})
    o, ids, _ = oracle.load_program(bad)
    with pytest.raises(oracle.OracleError) as e:
        o.run("naive")
    assert e.value.status == "UNSUPPORTED"


def test_triangle_join_over_three_relations_against_brute_force_and_a_matrix_product():
    # tri(x,y,z) :- r(x,y), s(y,z), t(z,x): the row set by three nested Python loops, the tag (w_xy + w_yz) + w_zx in
    # fp32, and the row count by the dense product sum((R @ S) * T^T), on the hot-domain recipe at a small size
    prog = W.hot_domain_triangle(n_rows=400, domain=24)
    o, ids, _ = oracle.load_program(prog)
    o.run("naive")
    cols, tags = o.read(ids["tri"])
    rel = {}
    for name in ("r", "s", "t"):
        (a, b), w = prog.facts[name]
        rel[name] = {(int(x), int(y)): np.float32(v) for x, y, v in zip(a, b, w)}
    want = {}
    for (x, y), wxy in rel["r"].items():
        for (y2, z), wyz in rel["s"].items():
            if y2 == y and (z, x) in rel["t"]:
                want[(x, y, z)] = np.float32(np.float32(wxy + wyz) + rel["t"][(z, x)])
    got = {(int(a), int(b), int(c)): t for a, b, c, t in zip(cols[0], cols[1], cols[2], tags)}
    assert got.keys() == want.keys() and len(want) > 20
    assert all(got[k] == want[k] for k in want)
    M = []
    for name in ("r", "s", "t"):
        m = np.zeros((24, 24))
        for (x, y) in rel[name]:
            m[x, y] = 1
        M.append(m)
    assert len(want) == int(round(((M[0] @ M[1]) * M[2].T).sum()))
    # rows come back in ascending (x, y, z)
    assert sorted(got.keys()) == list(zip(cols[0].tolist(), cols[1].tolist(), cols[2].tolist()))


def four_cycle_fixture(n_rows, domain, semiring):
    return W.uniform_four_cycle(n_rows, domain, semiring)


def test_four_cycle_join_against_brute_force_and_matrix_products():
    # c4(x,y,z,w) :- r(x,y), s(y,z), t(z,w), u(w,x) (the four-cycle template of "Worst-case-optimal joins"): the row set by
    # four nested Python loops, the tag ((w_xy + w_yz) + w_zw) + w_wx in fp32, the row count by trace(R S T U) of the
    # 0/1 matrices and, under sum-product, the sum of all tags by the trace of the weighted product
    d = 14
    prog = four_cycle_fixture(90, d, W.MAXPLUS)
    o, ids, _ = oracle.load_program(prog)
    o.run("naive")
    cols, tags = o.read(ids["c4"])
    rel, adj = {}, {}
    for name in ("r", "s", "t", "u"):
        (a, b), w = prog.facts[name]
        rel[name] = {(int(x), int(y)): np.float32(v) for x, y, v in zip(a, b, w)}
        m = np.zeros((d, d))
        for (x, y) in rel[name]:
            m[x, y] = 1
        adj[name] = m
    want = {}
    for (x, y), w1 in rel["r"].items():
        for (y2, z), w2 in rel["s"].items():
            if y2 != y:
                continue
            for (z2, w), w3 in rel["t"].items():
                if z2 == z and (w, x) in rel["u"]:
                    want[(x, y, z, w)] = np.float32(np.float32(np.float32(w1 + w2) + w3) + rel["u"][(w, x)])
    got = {(int(a), int(b), int(c), int(e)): t for a, b, c, e, t in zip(*cols, tags)}
    assert got.keys() == want.keys() and len(want) > 50
    assert all(got[k] == want[k] for k in want)
    assert len(want) == int(round(np.trace(adj["r"] @ adj["s"] @ adj["t"] @ adj["u"])))
    assert sorted(got.keys()) == list(zip(*(c.tolist() for c in cols)))       # ascending (x, y, z, w)

    sp = four_cycle_fixture(90, d, W.SUMPROD)
    wm = {}
    for name in ("r", "s", "t", "u"):
        (a, b), _ = sp.facts[name]
        wv = (0.5 + 0.1 * (np.arange(len(a)) % 7)).astype(np.float32)          # weights of order one
        sp.facts[name] = ([a, b], wv)
        m = np.zeros((d, d))
        m[a, b] = wv.astype(np.float64)
        wm[name] = m
    o2, ids2, _ = oracle.load_program(sp)
    o2.run("naive")
    _, t2 = o2.read(ids2["c4"])
    assert len(t2) == len(want)
    assert abs(float(t2.astype(np.float64).sum()) - np.trace(wm["r"] @ wm["s"] @ wm["t"] @ wm["u"])) < 1e-4 * len(t2)


def test_four_cycles_of_one_relation_are_the_closed_walks_of_length_four():
    # over a single 0/1 relation the rows of c4 are the closed walks x -> y -> z -> w -> x: trace(A^4); on the directed
    # ring of n nodes with both directions there are n * 6 of them (2 choices per step, returning after four steps)
    n = 9
    a = np.concatenate([np.arange(n), np.arange(n)]).astype(np.int32)
    b = np.concatenate([(np.arange(n) + 1) % n, (np.arange(n) - 1) % n]).astype(np.int32)
    e = (a, b, np.zeros(2 * n, np.float32))
    o, ids, _ = oracle.load_program(W.four_cycle_program(e, e, e, e))
    o.run("naive")
    assert o.size(ids["c4"]) == 6 * n
    A = np.zeros((n, n))
    A[a, b] = 1
    assert o.size(ids["c4"]) == int(round(np.trace(np.linalg.matrix_power(A, 4))))
