"""Pins for the oracle's atom patterns (constants, repeated variables, constants behind a bound prefix) and for
the sum-product arm of its gradient.  Every expected value is computed here with numpy / torch on dense arrays,
never by the oracle: a dropped constant test, a wrong column index or a transposed operand fails one of them."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_27203_b200 import synth, workloads as W


def run(program, mode="naive"):
    o, ids, rules = oracle.load_program(program)
    o.run(mode)
    return o, ids, rules


def graph(n, m, seed):
    s, d = synth.uniform_digraph(n, m, seed)
    w = (synth.randint(seed, 9, 0, m, 17).astype(np.float32) - 8.0) / 4.0          # exactly representable tags
    return s.astype(np.int32), d.astype(np.int32), w


def dense(n, s, d, w, fill):
    M = np.full((n, n), fill, np.float64)
    M[s, d] = w
    return M


@pytest.mark.parametrize("sr,fill,red", [(W.MAXPLUS, -np.inf, np.max), (W.MINPLUS, np.inf, np.min)])
def test_constant_in_the_first_column_selects_that_row_block(sr, fill, red):
    # h(y) :- e(c, y)
    n, c = 23, 7
    s, d, w = graph(n, 160, 41)
    prog = W.Program("const0", {"e": (2, sr), "h": (1, sr)}, [W.Rule("h", (W.V(0),), (W.Atom("e", (W.Const(c), W.Var(0))),))],
                     {"e": ([s, d], w)})
    o, ids, _ = run(prog)
    cols, tags = o.read(ids["h"])
    sel = s == c
    order = np.argsort(d[sel])
    assert sel.sum() > 2
    assert cols[0].tolist() == d[sel][order].tolist()
    assert tags.tolist() == w[sel][order].tolist()


def test_constant_in_the_second_column_with_the_first_unbound():
    # h(x) :- e(x, c): no leading column is fixed, so the constant is tested row by row
    n, c = 19, 4
    s, d, w = graph(n, 150, 42)
    prog = W.Program("const1", {"e": (2, W.MINPLUS), "h": (1, W.MINPLUS)}, [W.Rule("h", (W.V(0),), (W.Atom("e", (W.Var(0), W.Const(c))),))],
                     {"e": ([s, d], w)})
    o, ids, _ = run(prog)
    cols, tags = o.read(ids["h"])
    sel = d == c
    order = np.argsort(s[sel])
    assert sel.sum() > 2
    assert cols[0].tolist() == s[sel][order].tolist() and tags.tolist() == w[sel][order].tolist()


def test_repeated_variable_inside_one_atom_selects_the_diagonal():
    # loop(x) :- e(x, x)
    n = 12
    s = np.array([0, 1, 1, 3, 3, 5, 7, 7, 9, 11], np.int32)
    d = np.array([0, 2, 1, 3, 4, 6, 7, 8, 0, 11], np.int32)
    w = np.arange(10, dtype=np.float32) * 0.5 - 1.0
    prog = W.Program("loops", {"e": (2, W.MAXPLUS), "loop": (1, W.MAXPLUS)}, [W.Rule("loop", (W.V(0),), (W.Atom("e", (W.Var(0), W.Var(0))),))],
                     {"e": ([s, d], w)})
    o, ids, _ = run(prog)
    cols, tags = o.read(ids["loop"])
    diag = s == d
    assert cols[0].tolist() == s[diag].tolist() == [0, 1, 3, 7, 11]
    assert tags.tolist() == w[diag].tolist()
    assert n > cols[0].max()


def test_two_atom_rule_with_a_constant_in_the_second_atom():
    # h(x) :- e(x, y), f(y, c), min-plus: h(x) = min over y of e(x,y) + f(y,c)
    n, c = 17, 5
    s, d, w = graph(n, 120, 43)
    s2, d2, w2 = graph(n, 110, 44)
    prog = W.Program("const2", {"e": (2, W.MINPLUS), "f": (2, W.MINPLUS), "h": (1, W.MINPLUS)},
                     [W.Rule("h", (W.V(0),), (W.Atom("e", (W.Var(0), W.Var(1))), W.Atom("f", (W.Var(1), W.Const(c)))))],
                     {"e": ([s, d], w), "f": ([s2, d2], w2)})
    o, ids, _ = run(prog)
    cols, tags = o.read(ids["h"])
    E, F = dense(n, s, d, w, np.inf), dense(n, s2, d2, w2, np.inf)
    ref = (E + F[:, c][None, :]).min(axis=1)                  # all tags are multiples of 1/4: the sums are exact
    xs = np.flatnonzero(np.isfinite(ref))
    assert len(xs) > 3
    assert cols[0].tolist() == xs.tolist()
    assert tags.tolist() == ref[xs].astype(np.float32).tolist()


def test_constant_behind_a_bound_prefix_and_a_free_column():
    # h(x, z) :- e(x, y), t(y, z, c): y is bound (a prefix of t), z is free, the third column is a constant
    n, c = 11, 2
    s, d, w = graph(n, 60, 45)
    ta = synth.randint(46, 1, 0, 200, n).astype(np.int32)
    tb = synth.randint(46, 2, 0, 200, n).astype(np.int32)
    tc = synth.randint(46, 3, 0, 200, 4).astype(np.int32)
    key = (ta.astype(np.int64) * n + tb) * 4 + tc
    _, first = np.unique(key, return_index=True)
    ta, tb, tc = ta[first], tb[first], tc[first]
    tw = (synth.randint(46, 4, 0, len(ta), 9).astype(np.float32) - 4.0) / 2.0
    prog = W.Program("const3", {"e": (2, W.MAXPLUS), "t": (3, W.MAXPLUS), "h": (2, W.MAXPLUS)},
                     [W.Rule("h", (W.V(0), W.V(2)), (W.Atom("e", (W.Var(0), W.Var(1))), W.Atom("t", (W.Var(1), W.Var(2), W.Const(c)))))],
                     {"e": ([s, d], w), "t": ([ta, tb, tc], tw)})
    o, ids, _ = run(prog)
    cols, tags = o.read(ids["h"])
    E = dense(n, s, d, w, -np.inf)
    T = np.full((n, n), -np.inf)
    keep = tc == c
    T[ta[keep], tb[keep]] = tw[keep]
    ref = (E[:, :, None] + T[None, :, :]).max(axis=1)         # [x, z]
    xs, zs = np.nonzero(np.isfinite(ref))
    assert len(xs) > 5
    assert cols[0].tolist() == xs.tolist() and cols[1].tolist() == zs.tolist()
    assert tags.tolist() == ref[xs, zs].astype(np.float32).tolist()


def test_naive_and_seminaive_agree_with_numpy_on_a_recursion_that_starts_from_a_constant():
    # r(y) :- e(c, y).  r(z) :- r(y), e(y, z): nodes reachable from c in >= 1 step, by boolean matrix powers
    n, c = 30, 3
    s, d, _ = graph(n, 70, 47)
    prog = W.Program("const_reach", {"e": (2, W.MAXPLUS), "r": (1, W.MAXPLUS)},
                     [W.Rule("r", (W.V(0),), (W.Atom("e", (W.Const(c), W.Var(0))),)),
                      W.Rule("r", (W.V(1),), (W.Atom("r", (W.Var(0),)), W.Atom("e", (W.Var(0), W.Var(1)))))],
                     {"e": ([s, d], None)})
    A = np.zeros((n, n), bool)
    A[s, d] = True
    reach = A[c].copy()
    for _ in range(n):
        reach = reach | (reach[:, None] & A).any(axis=0)
    for mode in ("naive", "seminaive"):
        o, ids, _ = run(prog, mode)
        cols, tags = o.read(ids["r"])
        assert cols[0].tolist() == np.flatnonzero(reach).tolist()
        assert np.all(tags == 0.0)


# ---- gradient of a sum-product rule ------------------------------------------------------------------

def test_sumprod_backward_matches_torch_autograd_on_two_step_walks():
    # p2(x, z) :- e(x, y), e(y, z) under (+, *): out = A @ A entrywise on its support; loss = sum g * out
    n = 9
    s, d = synth.uniform_digraph(n, 30, 51)
    w = (0.5 + synth.uniform01(51, 3, 0, len(s))).astype(np.float32)
    prog = W.Program("p2", {"e": (2, W.SUMPROD), "p2": (2, W.SUMPROD)},
                     [W.Rule("p2", (W.V(0), W.V(2)), (W.Atom("e", (W.Var(0), W.Var(1))), W.Atom("e", (W.Var(1), W.Var(2)))))],
                     {"e": ([s, d], w)})
    o, ids, rules = run(prog)
    hc, ht = o.read(ids["p2"])
    ec, _ = o.read(ids["e"])
    g = synth.normal(51, 4, len(ht)).astype(np.float32)
    got = o.backward(rules[0], g)
    # autograd on the dense product; tags ordered as the oracle stores e (sorted by (src, dst))
    order = np.lexsort((d, s))
    assert np.array_equal(ec[0], s[order]) and np.array_equal(ec[1], d[order])
    t = torch.tensor(w[order].astype(np.float64), requires_grad=True)
    A = torch.zeros(n, n, dtype=torch.float64).index_put((torch.tensor(s[order].astype(np.int64)), torch.tensor(d[order].astype(np.int64))), t)
    out = A @ A
    assert np.allclose(out.detach().numpy()[hc[0], hc[1]], ht, rtol=1e-6)
    G = torch.zeros(n, n, dtype=torch.float64)
    G[torch.tensor(hc[0].astype(np.int64)), torch.tensor(hc[1].astype(np.int64))] = torch.tensor(g.astype(np.float64))
    (out * G).sum().backward()
    ref = t.grad.numpy()
    assert np.allclose(got[0].astype(np.float64) + got[1].astype(np.float64), ref, rtol=1e-6, atol=1e-6)
    # the two atoms separately: d/d(first-atom tag of (x,y)) = sum_z G[x,z] A[y,z];  second atom (y,z): sum_x G[x,z] A[x,y]
    An, Gn = A.detach().numpy(), G.numpy()
    first = (Gn @ An.T)[s[order], d[order]]
    second = (An.T @ Gn)[s[order], d[order]]
    assert np.allclose(got[0], first, rtol=1e-6, atol=1e-6) and np.allclose(got[1], second, rtol=1e-6, atol=1e-6)
    assert not np.allclose(first, second)                     # a transposed operand would be caught


def test_sumprod_backward_of_a_one_atom_rule_is_the_upstream_gradient_per_group():
    # deg(x) :- e(x, y) under (+, *): out(x) = sum_y w(x,y), so d loss / d w(x,y) = g[x]
    s = np.array([0, 0, 0, 2, 2, 5], np.int32)
    d = np.array([1, 2, 3, 0, 4, 5], np.int32)
    w = np.array([0.5, 1.5, 2.0, 3.0, 0.25, 4.0], np.float32)
    prog = W.Program("deg", {"e": (2, W.SUMPROD), "deg": (1, W.SUMPROD)}, [W.Rule("deg", (W.V(0),), (W.Atom("e", (W.Var(0), W.Var(1))),))],
                     {"e": ([s, d], w)})
    o, ids, rules = run(prog)
    cols, tags = o.read(ids["deg"])
    assert cols[0].tolist() == [0, 2, 5] and tags.tolist() == [4.0, 3.25, 4.0]
    g = np.array([2.0, -1.0, 0.5], np.float32)
    got = o.backward(rules[0], g)
    assert got[0].tolist() == [2.0, 2.0, 2.0, -1.0, -1.0, 0.5]
