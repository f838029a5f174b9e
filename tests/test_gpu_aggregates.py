"""Parity of the non-recursive aggregate rules (count, logsumexp, sum) and of the logsumexp-rule
gradient with the CPU oracle.  Tolerances: counts and tuple sets exact; logsumexp tags 1e-4 absolute;
gradients |d| <= 1e-5 + 1e-4 |ref| (fp32 exp and accumulation over at most 19 terms per row)."""
import math

import numpy as np
import pytest

import oracle
from paper_2609_27203_b200 import synth, workloads as W
from tests import helpers as H

pytestmark = pytest.mark.gpu
LSE_ABS = 1e-4


def both(program, **kw):
    from paper_2609_27203_b200 import xlog
    kw.setdefault("arena_bytes", 1 << 28)
    kw.setdefault("flags", xlog.FLAG_CHECK_INVARIANTS)
    ctx, gids, grules = xlog.load_program(program, **kw)
    receipt = ctx.fixpoint()
    o, oids, orules = oracle.load_program(program)
    o.run("naive")
    return ctx, gids, grules, o, oids, orules, receipt


def test_golden_listing7_degree_and_k3_triangle():
    g = H.read_golden("listing7_degree_count.txt")
    prog = W.Program("degree", {"edge": (2, W.SUMPROD), "degree": (2, W.SUMPROD)},
                     [W.Rule("degree", (W.V(0),), (W.Atom("edge", (W.Var(0), W.Var(1))),), emit_count=True)],
                     {"edge": ([g["edges"][:, 0].astype(np.int32), g["edges"][:, 1].astype(np.int32)], None)}, ("degree",))
    ctx, gids, _, o, oids, _, _ = both(prog)
    cols, tags = ctx.read(gids["degree"])
    assert cols[0].tolist() == [1, 2] and cols[1].tolist() == [3, 1] and tags.tolist() == [3.0, 1.0]
    ctx.close()
    g = H.read_golden("k3_triangle_lse.txt")
    e, t = g["edges"], g["tri_agg"]
    ctx, gids, _, o, oids, _, _ = both(W.triangle_program(e[:, 0], e[:, 1], e[:, 2]))
    cols, tags = ctx.read(gids["tri_agg"])
    assert cols[0].tolist() == [0, 1, 2] and cols[1].tolist() == [2, 2, 2]
    assert np.allclose(tags, t[:, 2], atol=2e-6)
    ctx.close()


@pytest.mark.parametrize("scale", [6, 10, 13])
def test_triangle_aggregate_ladder(scale):
    prog = W.config3(scale=scale)
    ctx, gids, _, o, oids, _, _ = both(prog)
    rep = H.compare_relations(ctx.read(gids["tri_agg"]), o.read(oids["tri_agg"]), abs_tol=LSE_ABS, what=prog.name)
    assert rep["rows"] > 0
    assert int(ctx.read(gids["tri_agg"])[0][1].sum()) % 3 == 0
    ctx.close()


def test_triangle_aggregate_bitmap_and_search_ways_agree():
    # a graph with hubs: a dense core (every ordered pair among the first 96 nodes) plus R-MAT 12 edges, so that the core
    # nodes' in-lists are marked in the shared-memory bitmap while the rest is searched; both ways against the oracle,
    # counts equal to the bit, and the run with the bitmap way must really have launched its kernel
    from paper_2609_27203_b200 import xlog
    base = W.config3(scale=12)
    (s, d), w = base.facts["e"]
    core = 96
    cs, cd = np.meshgrid(np.arange(core, dtype=np.int32), np.arange(core, dtype=np.int32), indexing="ij")
    keep = cs != cd
    s2 = np.concatenate([s, cs[keep]]); d2 = np.concatenate([d, cd[keep]])
    key, first = np.unique(s2.astype(np.int64) << 32 | d2, return_index=True)
    s2, d2 = s2[first], d2[first]
    w2 = synth.normal(12, 5, len(s2)).astype(np.float32)
    prog = W.triangle_program(s2, d2, w2, name="triangles_core96_rmat12")
    o, oids, _ = oracle.load_program(prog)
    o.run("seminaive")
    want = o.read(oids["tri_agg"])
    got = {}
    for flags in (xlog.FLAG_PROFILE, xlog.FLAG_PROFILE | xlog.FLAG_NO_TRIANGLE_BITMAP):
        ctx, ids, _ = xlog.load_program(prog, arena_bytes=1 << 28, flags=flags)
        ctx.fixpoint()
        got[flags] = ctx.read(ids["tri_agg"])
        H.compare_relations(got[flags], want, abs_tol=LSE_ABS, what="tri_agg")
        ran = "k_tri_bitmap" in ctx.profile()
        assert ran == (not flags & xlog.FLAG_NO_TRIANGLE_BITMAP)
        ctx.close()
    a, b = got[xlog.FLAG_PROFILE], got[xlog.FLAG_PROFILE | xlog.FLAG_NO_TRIANGLE_BITMAP]
    assert all(np.array_equal(x, y) for x, y in zip(a[0], b[0]))               # keys and counts
    assert np.allclose(a[1], b[1], rtol=0, atol=LSE_ABS)
    # run to run, the bitmap way repeats itself bit for bit
    ctx, ids, _ = xlog.load_program(prog, arena_bytes=1 << 28)
    ctx.fixpoint()
    again = ctx.read(ids["tri_agg"])
    ctx.close()
    assert np.array_equal(again[1].view(np.int32), a[1].view(np.int32))


@pytest.mark.parametrize("scale", [6, 10, 13])
def test_materialised_triangles_match_oracle_and_the_fused_aggregate(scale):
    # count -> scan -> materialise over the sorted columns; rows come out sorted by (x,y,z)
    prog3 = W.config3(scale=scale)
    (s, d), w = prog3.facts["e"]
    prog = W.triangle_rows_program(s, d, w)
    ctx, gids, _, o, oids, _, receipt = both(prog)
    rows = ctx.read(gids["tri"])
    rep = H.compare_relations(rows, o.read(oids["tri"]), rel_tol=1e-6, abs_tol=1e-6, what=prog.name)
    assert rep["rows"] == receipt["derived_tuples"] and rep["rows"] % 3 == 0
    ctx.close()
    # identical row sets on both paths: per-x row counts of the materialised join == counts of the fused aggregate
    ctx2, g2, _, _, _, _, _ = both(prog3)
    ac, _at = ctx2.read(g2["tri_agg"])
    xs, cnt = np.unique(rows[0][0], return_counts=True)
    assert np.array_equal(xs, ac[0]) and np.array_equal(cnt, ac[1])
    ctx2.close()


def dense_count(prog, n):
    """Triangles of r, s, t by a dense matrix product: sum over (x,y,z) of R[x,y] S[y,z] T[z,x]."""
    M = []
    for name in ("r", "s", "t"):
        (a, b), _ = prog.facts[name]
        m = np.zeros((n, n), np.float64)
        m[a, b] = 1
        M.append(m)
    return int(round(((M[0] @ M[1]) * M[2].T).sum()))


def test_triangle_join_over_three_relations_both_plans_match_the_oracle():
    from paper_2609_27203_b200 import xlog
    prog = W.hot_domain_triangle(n_rows=3000, domain=70)
    o, oids, _ = oracle.load_program(prog)
    o.run("naive")
    want = o.read(oids["tri"])
    assert len(want[1]) == dense_count(prog, 70) > 0
    for flags, plan in [(xlog.FLAG_FORCE_WCOJ, xlog.PLAN_WCOJ), (xlog.FLAG_FORCE_CHAIN, xlog.PLAN_CHAIN), (0, xlog.PLAN_WCOJ)]:
        ctx, gids, _ = xlog.load_program(prog, arena_bytes=1 << 28, flags=xlog.FLAG_CHECK_INVARIANTS | flags)
        r = ctx.fixpoint()
        assert r["triangle_plan"] == plan
        rep = H.compare_relations(ctx.read(gids["tri"]), want, what=f"{prog.name} plan {plan}")
        assert rep["bit_unequal"] == 0            # both plans fold (w_xy + w_yz) + w_zx in that order, like the oracle
        ctx.close()
    # columns whose maxima differ between the relations: rows of r that t can never close must not trip the key range
    (ra, rb), rw = prog.facts["r"]
    prog.facts["r"] = ([np.concatenate([ra, [900, 901]]).astype(np.int32), np.concatenate([rb, [5, 6]]).astype(np.int32)],
                       np.concatenate([rw, [-0.1, -0.2]]).astype(np.float32))
    o, oids, _ = oracle.load_program(prog)
    o.run("naive")
    for flags in (xlog.FLAG_FORCE_WCOJ, xlog.FLAG_FORCE_CHAIN):
        ctx, gids, _ = xlog.load_program(prog, arena_bytes=1 << 28, flags=xlog.FLAG_CHECK_INVARIANTS | flags)
        ctx.fixpoint()
        assert H.compare_relations(ctx.read(gids["tri"]), o.read(oids["tri"]), what="ragged maxima")["bit_unequal"] == 0
        ctx.close()


def test_skew_test_picks_the_plan_and_both_plans_give_identical_rows_on_the_hot_domain_fixture():
    # three relations of 65,536 rows over a hot domain: about 4.19 M triples out of 10.6 M two-paths
    from paper_2609_27203_b200 import xlog
    prog = W.hot_domain_triangle()
    n_tri = dense_count(prog, prog.info["domain"])
    assert 3_900_000 < n_tri < 4_500_000
    got = {}
    for flags in (0, xlog.FLAG_FORCE_WCOJ, xlog.FLAG_FORCE_CHAIN):
        ctx, gids, _ = xlog.load_program(prog, arena_bytes=1 << 30, flags=flags)
        r = ctx.fixpoint()
        got[flags] = (ctx.read(gids["tri"]), r)
        ctx.close()
    assert got[0][1]["triangle_plan"] == xlog.PLAN_WCOJ                      # skewed: the intermediate is 160x the inputs
    assert got[xlog.FLAG_FORCE_CHAIN][1]["candidates"] > 2 * n_tri           # the chain really materialised the two-paths
    base_cols, base_tags = got[xlog.FLAG_FORCE_WCOJ][0]
    assert len(base_tags) == n_tri
    key = (base_cols[0].astype(np.int64) << 40) | (base_cols[1].astype(np.int64) << 20) | base_cols[2]
    assert np.all(np.diff(key) > 0)
    for flags in (0, xlog.FLAG_FORCE_CHAIN):
        cols, tags = got[flags][0]
        assert all(np.array_equal(a, b) for a, b in zip(cols, base_cols)) and np.array_equal(tags.view(np.int32), base_tags.view(np.int32))
    # uniform and empty inputs take the binary-join chain
    sparse = W.hot_domain_triangle(n_rows=65536, domain=60000)
    ctx, gids, _ = xlog.load_program(sparse, arena_bytes=1 << 30)
    r = ctx.fixpoint()
    assert r["triangle_plan"] == xlog.PLAN_CHAIN
    ctx2, g2, _ = xlog.load_program(sparse, arena_bytes=1 << 30, flags=xlog.FLAG_FORCE_WCOJ)
    r2 = ctx2.fixpoint()
    assert r2["derived_tuples"] == r["derived_tuples"]
    a, b = ctx.read(gids["tri"]), ctx2.read(g2["tri"])
    assert all(np.array_equal(x, y) for x, y in zip(a[0], b[0])) and np.array_equal(a[1].view(np.int32), b[1].view(np.int32))
    ctx.close(); ctx2.close()
    empty = W.triangle_join_program(*[(np.zeros(0, np.int32), np.zeros(0, np.int32), np.zeros(0, np.float32))] * 3)
    ctx, gids, _ = xlog.load_program(empty, arena_bytes=1 << 24)
    r = ctx.fixpoint()
    assert r["triangle_plan"] == xlog.PLAN_CHAIN and r["derived_tuples"] == 0
    ctx.close()


def test_triangle_degenerate_graphs():
    # no triangle at all; one 3-cycle (single-term groups pass through bit-exactly); complete digraph; a hub
    for s, d, w in [([0, 1], [1, 2], [0.5, 0.25]),
                    ([0, 1, 2], [1, 2, 0], [0.1, 0.2, 0.7])]:
        prog = W.triangle_program(s, d, np.asarray(w, np.float32))
        ctx, gids, _, o, oids, _, _ = both(prog)
        rep = H.compare_relations(ctx.read(gids["tri_agg"]), o.read(oids["tri_agg"]), abs_tol=0, what="tiny")
        assert rep["bit_unequal"] == 0
        ctx.close()
    n = 40
    s, d = np.nonzero(~np.eye(n, dtype=bool))
    ctx, gids, _, o, oids, _, _ = both(W.triangle_program(s, d, np.zeros(len(s), np.float32)))
    cols, tags = ctx.read(gids["tri_agg"])
    assert cols[1].tolist() == [(n - 1) * (n - 2)] * n
    assert np.allclose(tags, math.log((n - 1) * (n - 2)), atol=1e-5)     # all-zero weights: LSE == ln(count)
    ctx.close()
    # hub: node 0 linked both ways with everyone, plus a ring among the others -> one group holds most terms
    m = 3000
    others = np.arange(1, m)
    s = np.concatenate([np.zeros(m - 1, np.int64), others, others])
    d = np.concatenate([others, np.zeros(m - 1, np.int64), np.roll(others, -1)])
    w = synth.normal(8, 1, len(s)).astype(np.float32)
    ctx, gids, _, o, oids, _, _ = both(W.triangle_program(s, d, w))
    H.compare_relations(ctx.read(gids["tri_agg"]), o.read(oids["tri_agg"]), abs_tol=LSE_ABS, what="hub")
    ctx.close()


@pytest.mark.parametrize("B", [1, 16, 1024])
def test_digit_sum_forward_and_backward(B):
    import torch
    prog = W.config4(n_pairs=B)
    ctx, gids, grules, o, oids, orules, receipt = both(prog)
    got = ctx.read(gids["sum"])
    want = o.read(oids["sum"])
    H.compare_relations(got, want, abs_tol=LSE_ABS, what=prog.name)
    assert len(got[1]) == 19 * B and receipt["candidates"] == 100 * B
    g = synth.head_gradient(19 * B, 77)
    og = o.backward(orules[0], g)
    ref = (og[0].astype(np.float64) + og[1].astype(np.float64))
    gg = ctx.backward(grules[0], torch.from_numpy(g).cuda())
    assert gg[0].data_ptr() == gg[1].data_ptr()                           # both atoms read `digit`: one buffer, the sum
    out = gg[0].cpu().numpy().astype(np.float64)
    assert np.all(np.abs(out - ref) <= 1e-5 + 1e-4 * np.abs(ref))
    # separate buffers per atom give the two parts
    parts = ctx.backward(grules[0], torch.from_numpy(g).cuda(), same_buffer_for_same_relation=False)
    for j in range(2):
        r = og[j].astype(np.float64)
        assert np.all(np.abs(parts[j].cpu().numpy() - r) <= 1e-5 + 1e-4 * np.abs(r))
    # one-hot upstream gradient: the weights of one head row's bindings sum to one
    e = np.zeros(19 * B, np.float32)
    e[min(9, 19 * B - 1)] = 1.0
    parts = ctx.backward(grules[0], torch.from_numpy(e).cuda(), same_buffer_for_same_relation=False)
    assert abs(float(parts[0].sum().item()) - 1.0) < 1e-5 and abs(float(parts[1].sum().item()) - 1.0) < 1e-5
    ctx.close()


def test_uniform_digits_golden():
    import torch
    g = H.read_golden("uniform_digits_lse.txt")
    B = 5
    lt = np.full((2 * B, 10), -math.log(10.0), np.float32)
    from paper_2609_27203_b200 import xlog
    ctx, ids, rules = xlog.load_program(W.digits_program(lt), arena_bytes=1 << 26)
    ctx.fixpoint()
    cols, tags = ctx.read(ids["sum"])
    for s_, v in g["out"]:
        for s2 in (int(s_), 18 - int(s_)):
            assert np.all(np.abs(tags[cols[1] == s2] - v) < 5e-6)
    grad = ctx.backward(rules[0], torch.ones(len(tags), device="cuda"))[0].cpu().numpy().reshape(2 * B, 10)
    for a, v in g["grad"]:
        assert np.all(np.abs(grad[:, int(a)] - v) < 1e-5)
    ctx.close()


def test_sum_semiring_two_step_walk_counts_and_facts_of_a_derived_relation():
    s, d = synth.uniform_digraph(60, 400, 3)
    prog = W.Program("p2", {"e": (2, W.SUMPROD), "p2": (2, W.SUMPROD)},
                     [W.Rule("p2", (W.V(0), W.V(2)), (W.Atom("e", (W.Var(0), W.Var(1))), W.Atom("e", (W.Var(1), W.Var(2)))))],
                     {"e": ([s, d], None)}, ("p2",))
    ctx, gids, _, o, oids, _, _ = both(prog)
    rep = H.compare_relations(ctx.read(gids["p2"]), o.read(oids["p2"]), what="p2")
    assert rep["bit_unequal"] == 0
    ctx.close()
    prog = W.Program("mix", {"a": (1, W.LOGSUMEXP), "q": (1, W.LOGSUMEXP)},
                     [W.Rule("q", (W.V(0),), (W.Atom("a", (W.Var(0),)),))],
                     {"a": ([np.array([1, 2], np.int32)], np.array([0.0, -1.0], np.float32)),
                      "q": ([np.array([2, 5], np.int32)], np.array([-1.0, -3.0], np.float32))}, ("q",))
    ctx, gids, _, o, oids, _, _ = both(prog)
    H.compare_relations(ctx.read(gids["q"]), o.read(oids["q"]), abs_tol=1e-6, what="mix")
    ctx.fixpoint()                                   # recomputed, not accumulated twice
    H.compare_relations(ctx.read(gids["q"]), o.read(oids["q"]), abs_tol=1e-6, what="mix again")
    ctx.close()


@pytest.mark.parametrize("n,m", [(9, 30), (300, 6000)])
def test_sumprod_backward_matches_the_oracle(n, m):
    # p2(x,z) :- e(x,y), e(y,z) under (+, *):  d loss / d tag = g[h] * (the other atom's tag), summed over the bindings
    import torch
    s, d = synth.uniform_digraph(n, m, 51)
    w = (0.5 + synth.uniform01(51, 3, 0, m)).astype(np.float32)
    prog = W.Program("p2", {"e": (2, W.SUMPROD), "p2": (2, W.SUMPROD)},
                     [W.Rule("p2", (W.V(0), W.V(2)), (W.Atom("e", (W.Var(0), W.Var(1))), W.Atom("e", (W.Var(1), W.Var(2)))))],
                     {"e": ([s, d], w)}, ("p2",))
    ctx, gids, grules, o, oids, orules, _ = both(prog)
    rep = H.compare_relations(ctx.read(gids["p2"]), o.read(oids["p2"]), rel_tol=1e-5, abs_tol=1e-6, what="p2 tags")
    g = synth.head_gradient(rep["rows"], 52)
    og = o.backward(orules[0], g)
    parts = ctx.backward(grules[0], torch.from_numpy(g).cuda(), same_buffer_for_same_relation=False)
    for j in range(2):
        ref = og[j].astype(np.float64)
        assert np.all(np.abs(parts[j].cpu().numpy() - ref) <= 1e-5 + 1e-4 * np.abs(ref)), f"atom {j}"
    both_atoms = ctx.backward(grules[0], torch.from_numpy(g).cuda())[0].cpu().numpy()
    ref = og[0].astype(np.float64) + og[1].astype(np.float64)
    assert np.all(np.abs(both_atoms - ref) <= 2e-5 + 1e-4 * np.abs(ref))
    ctx.close()
    # one-atom rule: deg(x) :- e(x,y); every row of e receives the upstream gradient of its group
    prog = W.Program("deg", {"e": (2, W.SUMPROD), "deg": (1, W.SUMPROD)}, [W.Rule("deg", (W.V(0),), (W.Atom("e", (W.Var(0), W.Var(1))),))],
                     {"e": ([s, d], w)}, ("deg",))
    ctx, gids, grules, o, oids, orules, _ = both(prog)
    xs = ctx.read(gids["deg"])[0][0]
    g = synth.head_gradient(len(xs), 53)
    got = ctx.backward(grules[0], torch.from_numpy(g).cuda())[0].cpu().numpy()
    assert np.array_equal(got, o.backward(orules[0], g)[0])
    assert np.array_equal(got, g[np.searchsorted(xs, np.sort(s))])
    ctx.close()


def test_backward_requires_a_forward_and_a_supported_head():
    import torch
    from paper_2609_27203_b200 import xlog
    prog = W.config4(n_pairs=2)
    ctx, ids, rules = xlog.load_program(prog, arena_bytes=1 << 26)
    with pytest.raises(xlog.XlogError) as e:
        ctx.backward(rules[0], torch.ones(38, device="cuda"))
    assert e.value.status == "INVALID_STATE"
    ctx.close()
    ctx, ids, rules = xlog.load_program(W.config1(20, 40), arena_bytes=1 << 26)
    ctx.fixpoint()
    with pytest.raises(xlog.XlogError) as e:
        ctx.backward(rules[0], torch.ones(ctx.size(ids["path"]), device="cuda"))
    assert e.value.status == "UNSUPPORTED"
    ctx.close()


def test_stratified_negation_matches_oracle():
    # set difference with tags kept; wildcard in the negated atom; two fixed columns; negation over a recursive lower stratum
    a = np.sort(synth.randint(5, 1, 0, 3000, 5000).astype(np.int32))
    b = np.sort(synth.randint(5, 2, 0, 3000, 5000).astype(np.int32))
    prog = W.Program("diff", {"a": (1, W.MINPLUS), "b": (1, W.MINPLUS), "only_a": (1, W.MINPLUS)},
                     [W.Rule("only_a", (W.V(0),), (W.Atom("a", (W.Var(0),)), W.Atom("b", (W.Var(0),), negated=True)))],
                     {"a": ([a], synth.normal(5, 3, 3000).astype(np.float32)), "b": ([b], None)}, ("only_a",))
    ctx, gids, _, o, oids, _, _ = both(prog)
    rep = H.compare_relations(ctx.read(gids["only_a"]), o.read(oids["only_a"]), what="only_a")
    assert rep["bit_unequal"] == 0 and set(ctx.read(gids["only_a"])[0][0].tolist()) == set(a.tolist()) - set(b.tolist())
    ctx.close()
    s, d = synth.uniform_digraph(300, 900, 23)
    w = synth.log_prob_tags(900, 23)
    prog = W.Program("neg2", {"edge": (2, W.MAXPLUS), "sink": (1, W.MAXPLUS), "oneway": (2, W.MAXPLUS)},
                     [W.Rule("sink", (W.V(1),), (W.Atom("edge", (W.Var(0), W.Var(1))), W.Atom("edge", (W.Var(1), W.Var(2)), negated=True))),
                      W.Rule("oneway", (W.V(0), W.V(1)), (W.Atom("edge", (W.Var(0), W.Var(1))), W.Atom("edge", (W.Var(1), W.Var(0)), negated=True)))],
                     {"edge": ([s, d], w)}, ("sink", "oneway"))
    ctx, gids, _, o, oids, _, _ = both(prog)
    for name in ("sink", "oneway"):
        assert H.compare_relations(ctx.read(gids[name]), o.read(oids[name]), what=name)["bit_unequal"] == 0
    ctx.close()
    prog = W.config2(scale=10)
    n = 1 << 10
    prog.relations["node"] = (1, W.MINPLUS)
    prog.relations["unreached"] = (1, W.MINPLUS)
    prog.facts["node"] = ([np.arange(n, dtype=np.int32)], None)
    prog.rules.append(W.Rule("unreached", (W.V(0),), (W.Atom("node", (W.Var(0),)), W.Atom("dist", (W.Var(0),), negated=True))))
    prog.outputs = ("dist", "unreached")
    ctx, gids, _, o, oids, _, _ = both(prog)
    for name in prog.outputs:
        assert H.compare_relations(ctx.read(gids[name]), o.read(oids[name]), what=name)["bit_unequal"] == 0
    assert ctx.size(gids["dist"]) + ctx.size(gids["unreached"]) == n
    ctx.close()
    # negation through recursion is rejected
    from paper_2609_27203_b200 import xlog
    bad = W.Program("bad", {"e": (1, W.MINPLUS), "p": (1, W.MINPLUS)},
                    [W.Rule("p", (W.V(0),), (W.Atom("e", (W.Var(0),)), W.Atom("p", (W.Var(0),), negated=True)))],
                    {"e": ([np.array([1], np.int32)], None)})
    c2, _, _ = xlog.load_program(bad, arena_bytes=1 << 24)
    with pytest.raises(xlog.XlogError) as e:
        c2.fixpoint()
    assert e.value.status == "UNSUPPORTED"
    c2.close()


def check_four_cycle(prog, what, expect_plan=None, **kw):
    """Both plans of the four-cycle join (multiway step / binary-join chain) and the skew test's own choice against the
    oracle: identical rows and tags on every path (the paper's gate for its WCOJ comparison)."""
    from paper_2609_27203_b200 import xlog
    o, oids, _ = oracle.load_program(prog)
    o.run("naive")
    want = o.read(oids["c4"])
    chosen = None
    for flags, plan in ((xlog.FLAG_FORCE_WCOJ, xlog.PLAN_WCOJ), (xlog.FLAG_FORCE_CHAIN, xlog.PLAN_CHAIN), (0, None)):
        ctx, gids, _ = xlog.load_program(prog, **dict(dict(arena_bytes=1 << 30), **kw, flags=xlog.FLAG_CHECK_INVARIANTS | flags))
        receipt = ctx.fixpoint()
        rep = H.compare_relations(ctx.read(gids["c4"]), want, what=f"{what}, flags {flags}")
        assert rep["bit_unequal"] == 0            # ((w_xy (x) w_yz) (x) w_zw) (x) w_wx in fp32 on every path
        assert receipt["derived_tuples"] == len(want[1])
        if plan is not None:
            assert receipt["triangle_plan"] == plan
        else:
            chosen = receipt["triangle_plan"]
        ctx.close()
    assert chosen in (xlog.PLAN_WCOJ, xlog.PLAN_CHAIN)
    if expect_plan is not None:
        assert chosen == expect_plan, (what, chosen)
    return len(want[1])


def test_four_cycle_join_matches_the_oracle():
    # dense small domain (every two-path has two long lists: the warp-cooperative walk), sparse (short lists: a thread
    # per two-path), sum-product tags, and a skewed graph used four times (hub two-paths next to empty ones)
    from paper_2609_27203_b200 import xlog
    # 3000 rows over 70 values: 43 partners per value, 5.5 M three-paths against 3000 input rows -> the multiway step;
    # 20000 rows over 2500 values: 8 partners per value, hence 8^2 three-paths per input row -> still the multiway step;
    # 20000 rows over 12000 values: fewer than two partners per value -> the chain
    assert check_four_cycle(W.uniform_four_cycle(3000, 70), "dense", xlog.PLAN_WCOJ) > 100000
    assert check_four_cycle(W.uniform_four_cycle(20000, 2500), "sparse", xlog.PLAN_WCOJ) > 0
    assert check_four_cycle(W.uniform_four_cycle(20000, 12000), "very sparse", xlog.PLAN_CHAIN) >= 0
    sp = W.uniform_four_cycle(2500, 90, W.SUMPROD)
    for name in ("r", "s", "t", "u"):
        (a, b), _ = sp.facts[name]
        sp.facts[name] = ([a, b], (0.5 + 0.125 * (np.arange(len(a)) % 9)).astype(np.float32))
    assert check_four_cycle(sp, "sum-product") > 10000
    s, d, _ = synth.rmat_graph(9, 6, synth.SEED_BASE + 71, "n01")
    e = (s, d, synth.log_prob_tags(len(s), synth.SEED_BASE + 72))
    assert check_four_cycle(W.four_cycle_program(e, e, e, e, name="four_cycle_rmat9"), "rmat") > 10000


def test_four_cycle_edge_cases():
    from paper_2609_27203_b200 import xlog
    # a relation that closes nothing; an empty relation; 64-bit head keys (four 16-bit columns); ragged column maxima
    e = (np.array([0, 1, 2, 3], np.int32), np.array([1, 2, 3, 0], np.int32), np.array([0.5, 0.25, 0.125, 1.0], np.float32))
    assert check_four_cycle(W.four_cycle_program(e, e, e, e), "one ring") == 4
    none = (np.array([7], np.int32), np.array([8], np.int32), np.array([0.0], np.float32))
    assert check_four_cycle(W.four_cycle_program(e, e, e, none), "u closes nothing") == 0
    empty = (np.zeros(0, np.int32), np.zeros(0, np.int32), np.zeros(0, np.float32))
    assert check_four_cycle(W.four_cycle_program(e, e, empty, e), "empty t") == 0
    wide = W.uniform_four_cycle(3000, 70)
    for name in ("r", "s", "t", "u"):
        (a, b), w = wide.facts[name]
        wide.facts[name] = ([(a * 900 + 11).astype(np.int32), (b * 900 + 11).astype(np.int32)], w)
    assert check_four_cycle(wide, "64-bit keys") > 100000
    rag = W.uniform_four_cycle(3000, 70)
    (a, b), w = rag.facts["r"]
    rag.facts["r"] = ([np.concatenate([a, [900, 3]]).astype(np.int32), np.concatenate([b, [5, 901]]).astype(np.int32)],
                      np.concatenate([w, [-0.1, -0.2]]).astype(np.float32))
    assert check_four_cycle(rag, "ragged maxima") > 100000
    # anything else with four atoms is refused
    bad = W.uniform_four_cycle(10, 5)
    bad.rules[0] = W.Rule("c4", (W.V(0), W.V(1), W.V(2), W.V(3)),
                          (W.Atom("r", (W.Var(0), W.Var(1))), W.Atom("s", (W.Var(1), W.Var(2))), W.Atom("t", (W.Var(2), W.Var(3))), W.Atom("u", (W.Var(0), W.Var(3)))))
    with pytest.raises(xlog.XlogError) as ei:
        xlog.load_program(bad, arena_bytes=1 << 26)
    assert ei.value.status == "UNSUPPORTED"


def test_backward_of_a_rule_whose_head_is_empty():
    # a and b share no join value: the head is empty, its gradient has no rows (a NULL pointer is accepted), and both
    # atom gradients come back zero
    import torch
    a = ([np.array([0, 1], np.int32), np.array([5, 6], np.int32)], np.array([0.1, 0.2], np.float32))
    b = ([np.array([7, 8], np.int32), np.array([1, 2], np.int32)], np.array([0.3, 0.4], np.float32))
    prog = W.Program("empty_head", {"a": (2, W.LOGSUMEXP), "b": (2, W.LOGSUMEXP), "s": (2, W.LOGSUMEXP)},
                     [W.Rule("s", (W.V(0), W.V(2)), (W.Atom("a", (W.Var(0), W.Var(1))), W.Atom("b", (W.Var(1), W.Var(2)))))],
                     {"a": a, "b": b}, ("s",))
    ctx, gids, grules, o, oids, orules, _ = both(prog)
    assert ctx.size(gids["s"]) == 0 == o.size(oids["s"])
    parts = ctx.backward(grules[0], torch.zeros(0, device="cuda"), same_buffer_for_same_relation=False)
    assert all(float(p.abs().sum().item()) == 0.0 and p.numel() == 2 for p in parts)
    ctx.close()
