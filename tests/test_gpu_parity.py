"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element.

Tolerances (from the benchmark spec): tuple sets bit-exact; max-plus / min-plus tags 1e-5
relative (expected and reported: bit-equal); logsumexp tags 1e-4 absolute; counts exact.
"""
import numpy as np
import pytest

import oracle
from paper_2609_27203_b200 import synth, workloads as W
from tests import helpers as H

pytestmark = pytest.mark.gpu

MINMAX_REL = 1e-5
LSE_ABS = 1e-4


def gpu_run(program, **kw):
    from paper_2609_27203_b200 import xlog
    kw.setdefault("arena_bytes", 1 << 28)
    kw.setdefault("flags", xlog.FLAG_CHECK_INVARIANTS)
    ctx, ids, rules = xlog.load_program(program, **kw)
    receipt = ctx.fixpoint()
    return ctx, ids, rules, receipt


def oracle_run(program, mode="seminaive"):
    o, ids, rules = oracle.load_program(program)
    stats = o.run(mode)
    return o, ids, rules, stats


def check_program(program, rel_tol=MINMAX_REL, abs_tol=0.0, expect_bit_equal=True, mode="seminaive", **kw):
    """Both evaluation paths of the CUDA engine against the oracle: the default one (a linear max/min recursion goes
    through the tag mirror) and the one that always sorts, reduces by key and merges.  The two must agree with each
    other bit for bit, relation and counters alike."""
    from paper_2609_27203_b200 import xlog
    o, oids, _, stats = oracle_run(program, mode)
    receipts, results = [], []
    # default (tag mirror; the rounds of each first-column value on their own in shared memory where the rule has that shape,
    # else delta rounds resident in one graph) / resident in one graph always / the same rounds launched one by one / host-driven
    # mirror rounds (with the grouped join where the rule has that shape, driven by the changed bitmap where a unit of 32
    # carried values exists) / the grouped join from a delta row list / the row-wise join only / the sorting path
    for extra in (0, xlog.FLAG_NO_ROW_FIXPOINT, xlog.FLAG_NO_GRAPH, xlog.FLAG_NO_RESIDENT_LOOP, xlog.FLAG_NO_RESIDENT_LOOP | xlog.FLAG_NO_BITMAP_JOIN,
                  xlog.FLAG_NO_RESIDENT_LOOP | xlog.FLAG_NO_GROUPED_JOIN, xlog.FLAG_NO_TAG_MIRROR):
        ctx, gids, _, receipt = gpu_run(program, **dict(kw, flags=kw.get("flags", xlog.FLAG_CHECK_INVARIANTS) | extra))
        got = {}
        for name in program.outputs:
            got[name] = ctx.read(gids[name])
            rep = H.compare_relations(got[name], o.read(oids[name]), rel_tol=rel_tol, abs_tol=abs_tol,
                                      what=f"{program.name}:{name}")
            if expect_bit_equal:
                assert rep["bit_unequal"] == 0, rep
        assert receipt["derived_tuples"] == stats["derived_tuples"]
        ctx.close()
        receipts.append(receipt); results.append(got)
    for i in range(1, len(results)):
        for name in program.outputs:
            assert H.compare_relations(results[0][name], results[i][name], what=f"path 0 vs path {i}")["bit_unequal"] == 0
        for k in ("iterations", "candidates", "new_tuples", "improved_tags", "derived_tuples", "strata"):
            assert receipts[0][k] == receipts[i][k], (i, k, receipts[0][k], receipts[i][k])
    assert receipts[-1]["unique_candidates"] >= 0
    return receipts[0], stats


# ---- relation store: load / read ---------------------------------------------------------

@pytest.mark.parametrize("n,arity,sr", [(1, 1, "maxplus"), (7, 2, "minplus"), (5000, 2, "maxplus"),
                                        (100_003, 2, "minplus"), (30_000, 3, "logsumexp"), (20_000, 1, "sumprod"),
                                        # big enough for the high-bit sort + shared-memory table reduction, with groups
                                        # so large that they are split and merged through the spill tables
                                        (2_000_003, 1, "minplus"), (3_000_000, 2, "maxplus"), (1_500_000, 3, "minplus")])
def test_load_sorts_and_combines_duplicates(n, arity, sr):
    from paper_2609_27203_b200 import xlog
    hi = [50, 300, 7, 5][:arity] if n > 10 else [3, 3, 3, 3][:arity]        # small domains force duplicates
    if n > 1_000_000 and arity == 1:
        hi = [5000]
    cols = [synth.randint(9, 20 + c, 0, n, hi[c]).astype(np.int32) for c in range(arity)]
    tags = (synth.normal(9, 30, n)).astype(np.float32)
    if sr == "sumprod":
        tags = np.abs(tags) + 0.5
    ctx = xlog.Context(arena_bytes=1 << 27, flags=xlog.FLAG_CHECK_INVARIANTS)
    r = ctx.relation(arity, sr)
    ctx.load(r, cols, tags)
    o = oracle.Oracle()
    ro = o.relation(arity, sr)
    o.load(ro, cols, tags)
    tol = dict(rel_tol=0, abs_tol=0) if sr in ("maxplus", "minplus") else dict(rel_tol=1e-5, abs_tol=LSE_ABS)
    rep = H.compare_relations(ctx.read(r), o.read(ro), what="load", **tol)
    if sr in ("maxplus", "minplus"):
        assert rep["bit_unequal"] == 0
    # device-resident input gives the same relation
    import torch
    ctx.load(r, [torch.from_numpy(c).cuda() for c in cols], torch.from_numpy(tags).cuda())
    H.compare_relations(ctx.read(r), o.read(ro), what="load(device)", **tol)
    dc, dt = ctx.read_device(r)
    assert np.array_equal(dt.cpu().numpy(), ctx.read(r)[1])
    ctx.close()


def test_rows_that_arrive_in_order_take_the_short_load_path():
    # strictly increasing rows are stored as they come (no sort, no duplicate pass); one swapped pair or one repeated row
    # must send the load down the sorting path again.  All three must match the oracle.
    from paper_2609_27203_b200 import xlog
    n = 200_000
    a = np.sort(synth.randint(5, 1, 0, n, 5000)).astype(np.int32)
    b = np.arange(n, dtype=np.int32)                     # makes every row distinct and the pairs increasing
    t = synth.normal(5, 2, n).astype(np.float32)
    swapped = (a.copy(), b.copy()); swapped[1][[1000, 1001]] = swapped[1][[1001, 1000]]
    repeated = (a.copy(), b.copy()); repeated[0][777] = repeated[0][776]; repeated[1][777] = repeated[1][776]
    for cols in [(a, b), swapped, repeated]:
        ctx = xlog.Context(arena_bytes=1 << 27, flags=xlog.FLAG_CHECK_INVARIANTS)
        r = ctx.relation(2, "minplus")
        ctx.load(r, list(cols), t)
        o = oracle.Oracle()
        ro = o.relation(2, "minplus")
        o.load(ro, list(cols), t)
        assert H.compare_relations(ctx.read(r), o.read(ro), what="in-order load")["bit_unequal"] == 0
        ctx.close()


def test_empty_and_single_relations():
    from paper_2609_27203_b200 import xlog
    ctx = xlog.Context(arena_bytes=1 << 24)
    r = ctx.relation(2, "maxplus")
    assert ctx.size(r) == 0
    ctx.load(r, [np.zeros(0, np.int32), np.zeros(0, np.int32)], np.zeros(0, np.float32))
    assert ctx.size(r) == 0 and len(ctx.read(r)[1]) == 0
    ctx.load(r, [np.array([5], np.int32), np.array([9], np.int32)], None)
    cols, tags = ctx.read(r)
    assert cols[0].tolist() == [5] and cols[1].tolist() == [9] and tags.tolist() == [0.0]
    ctx.close()


def test_wide_keys_use_64_bit_packing():
    # two 31-bit columns: 62 key bits
    from paper_2609_27203_b200 import xlog
    n = 20_000
    a = synth.randint(3, 1, 0, n, (1 << 31) - 1).astype(np.int32)
    b = synth.randint(3, 2, 0, n, (1 << 31) - 1).astype(np.int32)
    a[:100] = a[100:200]                                 # some equal leading columns
    t = synth.normal(3, 3, n).astype(np.float32)
    ctx = xlog.Context(arena_bytes=1 << 26, flags=xlog.FLAG_CHECK_INVARIANTS)
    r = ctx.relation(2, "maxplus")
    ctx.load(r, [a, b], t)
    o = oracle.Oracle()
    ro = o.relation(2, "maxplus")
    o.load(ro, [a, b], t)
    assert H.compare_relations(ctx.read(r), o.read(ro))["bit_unequal"] == 0
    ctx.close()


# ---- golden cases ------------------------------------------------------------------------

def test_golden_listing1_chain():
    g = H.read_golden("listing1_chain_maxplus.txt")
    e, c = g["edges"], g["closure"]
    ctx, ids, _, rc = gpu_run(W.closure_program(e[:, 0], e[:, 1], e[:, 2]))
    rep = H.compare_relations(ctx.read(ids["path"]), ([c[:, 0], c[:, 1]], c[:, 2]))
    assert rep["bit_unequal"] == 0 and rc["derived_tuples"] == 6
    ctx.close()


def test_golden_diamond_and_cycle():
    g = H.read_golden("diamond_sssp_minplus.txt")
    e, d = g["edges"], g["dist"]
    ctx, ids, _, rc = gpu_run(W.sssp_program(e[:, 0], e[:, 1], e[:, 2], 0))
    assert H.compare_relations(ctx.read(ids["dist"]), ([d[:, 0]], d[:, 1]))["bit_unequal"] == 0
    assert rc["improved_tags"] == 2 and rc["new_tuples"] == 3
    ctx.close()
    g = H.read_golden("cycle3_maxplus.txt")
    e, c = g["edges"], g["closure"]
    ctx, ids, _, _ = gpu_run(W.closure_program(e[:, 0], e[:, 1], e[:, 2]))
    assert H.compare_relations(ctx.read(ids["path"]), ([c[:, 0], c[:, 1]], c[:, 2]))["bit_unequal"] == 0
    ctx.close()


# ---- recursive workloads -----------------------------------------------------------------

@pytest.mark.parametrize("n,m", [(4, 5), (50, 120), (200, 800), (1000, 4000)])
def test_closure_maxplus_ladder(n, m):
    check_program(W.config1(n, m))


def test_closure_adversarial_shapes():
    # chain (maximal iteration count), star (one hub), one group holding every candidate
    n = 300
    check_program(W.closure_program(np.arange(n - 1), np.arange(1, n), synth.log_prob_tags(n - 1, 3)))
    hub_out = W.closure_program(np.zeros(n - 1, np.int32), np.arange(1, n), synth.log_prob_tags(n - 1, 4))
    check_program(hub_out)
    src = np.concatenate([np.zeros(n - 1, np.int32), np.arange(1, n)])
    dst = np.concatenate([np.arange(1, n), np.full(n - 1, n, np.int32)])      # 0 -> i -> n: n-1 candidates for (0, n)
    check_program(W.closure_program(src, dst, synth.log_prob_tags(len(src), 5)))
    # complete DAG with +1 weights under max-plus: j-i-1 successive improvements of one tuple
    s, d = np.triu_indices(40, 1)
    check_program(W.closure_program(s, d, np.ones(len(s), np.float32)))
    # zero-improvement cycle
    check_program(W.closure_program(np.arange(9), (np.arange(9) + 1) % 9, np.zeros(9, np.float32)))


@pytest.mark.parametrize("scale", [8, 12, 16])
def test_sssp_minplus_ladder(scale):
    check_program(W.config2(scale=scale))


@pytest.mark.parametrize("scale,ns", [(8, 4), (12, 64), (12, 300), (15, 64)])
def test_multi_source_reach_ladder(scale, ns):
    check_program(W.config5(scale=scale, n_sources=ns))


def test_right_linear_rule_uses_a_transposed_index():
    # path(x,z) :- edge(x,y), path(y,z): the delta sits on the second atom, edge is looked up by its second column
    s, d = synth.uniform_digraph(120, 400, 21)
    t = synth.log_prob_tags(400, 21)
    prog = W.closure_program(s, d, t)
    prog.rules[1] = W.Rule("path", (W.V(0), W.V(2)), (W.Atom("edge", (W.Var(0), W.Var(1))), W.Atom("path", (W.Var(1), W.Var(2)))))
    # fl(w + t) == fl(t + w): still expected bit-equal for two-term products, but sums are folded from
    # the other end of the path, so compare with tolerance only
    check_program(prog, expect_bit_equal=False)


def test_non_linear_and_mutual_recursion():
    # p(x,z) :- p(x,y), p(y,z): two recursive atoms, so each round joins delta with the full relation on both sides
    # (the looked-up side is indexed afresh, once by its first and once by its second column)
    s, d = synth.uniform_digraph(150, 500, 31)
    t = synth.log_prob_tags(500, 31)
    edge = ([s, d], t)
    nl = W.Program("nonlinear", {"e": (2, W.MAXPLUS), "p": (2, W.MAXPLUS)},
                   [W.Rule("p", (W.V(0), W.V(1)), (W.Atom("e", (W.Var(0), W.Var(1))),)),
                    W.Rule("p", (W.V(0), W.V(2)), (W.Atom("p", (W.Var(0), W.Var(1))), W.Atom("p", (W.Var(1), W.Var(2)))))],
                   {"e": edge}, ("p",))
    r_nl, _ = check_program(nl)
    # same relation as the linear closure (tuple set; tags may differ in the last place: other association of the sums)
    from paper_2609_27203_b200 import xlog
    c1, i1, _ = xlog.load_program(nl, arena_bytes=1 << 27)
    c1.fixpoint()
    c2, i2, _ = xlog.load_program(W.closure_program(s, d, t), arena_bytes=1 << 27)
    c2.fixpoint()
    H.compare_relations(c1.read(i1["p"]), c2.read(i2["path"]), rel_tol=1e-5, what="non-linear vs linear closure")
    assert r_nl["iterations"] < c2.last_receipt["iterations"]          # path doubling needs fewer rounds
    c1.close(); c2.close()
    # odd / even length walks: two heads in one recursive component
    w = (1 + 9 * synth.uniform01(31, 9, 0, 500)).astype(np.float32)
    mut = W.Program("odd_even", {"e": (2, W.MINPLUS), "odd": (2, W.MINPLUS), "even": (2, W.MINPLUS)},
                    [W.Rule("odd", (W.V(0), W.V(1)), (W.Atom("e", (W.Var(0), W.Var(1))),)),
                     W.Rule("even", (W.V(0), W.V(2)), (W.Atom("odd", (W.Var(0), W.Var(1))), W.Atom("e", (W.Var(1), W.Var(2))))),
                     W.Rule("odd", (W.V(0), W.V(2)), (W.Atom("even", (W.Var(0), W.Var(1))), W.Atom("e", (W.Var(1), W.Var(2)))))],
                    {"e": ([s, d], w)}, ("odd", "even"))
    check_program(mut)


def test_mutual_recursion_over_one_tag_mirror_per_head():
    # three heads in one component, each rule reading one of them: a one-atom copy rule, heads of different arity, a head
    # that starts with loaded facts (some better, some worse than what gets derived), and a MAXPLUS head beside MINPLUS ones
    # (each head combines with its own oplus; the component has no cycle of positive max-plus weight)
    from paper_2609_27203_b200 import xlog
    n, m = 400, 1500
    s, d = synth.uniform_digraph(n, m, 77)
    w = (1 + 9 * synth.uniform01(77, 2, 0, m)).astype(np.float32)
    seeds = np.array([0, 5, 9], np.int32)
    start = np.array([3, 17, 200], np.int32)
    prog = W.Program("three_heads", {"e": (2, W.MINPLUS), "src": (1, W.MINPLUS), "a": (2, W.MINPLUS), "b": (2, W.MINPLUS), "far": (1, W.MINPLUS)},
                     [W.Rule("a", (W.V(0), W.V(0)), (W.Atom("src", (W.Var(0),)),)),
                      W.Rule("b", (W.V(0), W.V(2)), (W.Atom("a", (W.Var(0), W.Var(1))), W.Atom("e", (W.Var(1), W.Var(2))))),
                      W.Rule("a", (W.V(0), W.V(2)), (W.Atom("b", (W.Var(0), W.Var(1))), W.Atom("e", (W.Var(1), W.Var(2))))),
                      W.Rule("far", (W.V(1),), (W.Atom("b", (W.Var(0), W.Var(1))),)),
                      W.Rule("a", (W.Affine(0, ()), W.V(0)), (W.Atom("far", (W.Var(0),)),))],
                     {"e": ([s, d], w), "src": ([seeds], None),
                      "far": ([start], np.array([0.5, 1000.0, 2.0], np.float32))}, ("a", "b", "far"))
    r, stats = check_program(prog)
    assert r["iterations"] == stats["iterations"] and r["iterations"] > 3
    # the default route took the mirrors (it does not count distinct candidate keys), the sorting route does
    ctx, ids, _ = xlog.load_program(prog, arena_bytes=1 << 28)
    assert ctx.fixpoint()["unique_candidates"] == -1
    ctx.close()
    # a max-plus head fed by a min-plus head, on a DAG (edges u < v only) so that the longest walk is finite
    lo, hi = np.minimum(s, d), np.maximum(s, d)
    keep = lo != hi
    key = np.unique(lo[keep].astype(np.int64) * n + hi[keep])
    s2, d2 = (key // n).astype(np.int32), (key % n).astype(np.int32)
    w2 = (1 + 9 * synth.uniform01(78, 2, 0, len(s2))).astype(np.float32)
    mixed = W.Program("min_and_max", {"e": (2, W.MINPLUS), "lo": (2, W.MINPLUS), "hi": (2, W.MAXPLUS)},
                      [W.Rule("lo", (W.V(0), W.V(1)), (W.Atom("e", (W.Var(0), W.Var(1))),)),
                       W.Rule("hi", (W.V(0), W.V(2)), (W.Atom("lo", (W.Var(0), W.Var(1))), W.Atom("e", (W.Var(1), W.Var(2))))),
                       W.Rule("lo", (W.V(0), W.V(2)), (W.Atom("hi", (W.Var(0), W.Var(1))), W.Atom("e", (W.Var(1), W.Var(2)))))],
                      {"e": ([s2, d2], w2)}, ("lo", "hi"))
    check_program(mixed)
    # which route ran: two binary heads with one key layout and closure-shaped rules take the row-local fixpoint (a row per
    # head in the block); the three heads above, one of them unary, take the host-driven rounds over one mirror per head
    for program, row_local in ((mixed, True), (prog, False)):
        ctx, ids, _ = xlog.load_program(program, arena_bytes=1 << 28, flags=xlog.FLAG_PROFILE)
        ctx.fixpoint()
        assert ("k_row_fixpoint" in ctx.profile()) == row_local
        assert "k_sort_pass" not in ctx.profile() or not row_local
        ctx.close()


def test_recursion_with_head_arithmetic_takes_the_general_join_path():
    # down(x - 1) :- down(x), pos(x): a negative head constant rules out the linear-key shape, so every route goes through
    # the general per-candidate evaluation (with the tag mirror as sink on the default routes)
    n = 3000
    pos = np.arange(1, n + 1, dtype=np.int32)
    w = (1 + 9 * synth.uniform01(41, 1, 0, n)).astype(np.float32)
    prog = W.Program("countdown", {"pos": (1, W.MINPLUS), "down": (1, W.MINPLUS)},
                     [W.Rule("down", (W.Affine(-1, ((0, 1),)),), (W.Atom("down", (W.Var(0),)), W.Atom("pos", (W.Var(0),))))],
                     {"pos": ([pos], w), "down": ([np.array([n, n - 7], np.int32)], np.array([0.0, 100.0], np.float32))}, ("down",))
    r, _ = check_program(prog, max_iterations=n + 5)
    assert r["iterations"] == n + 1 and r["derived_tuples"] == n - 1      # n - 7 is a loaded fact


def test_routes_agree_at_sizes_beyond_the_oracle():
    # mid-size cases where segments of the grouped join hold hundreds of delta rows (several passes of 32 lanes) and hub
    # nodes have tens of thousands of neighbours: every engine route must derive the same relation, bit for bit, with the
    # same counters.  (The oracle would need minutes here; the smaller ladders above pin the routes to it.)
    from paper_2609_27203_b200 import xlog
    hs = synth.randint(71, 1, 0, 40000, 20); hd = synth.randint(71, 2, 0, 40000, 5000)
    s = np.concatenate([hs, hd[:20000]]); t = np.concatenate([hd, hs[:20000]])
    key = np.unique(s[s != t].astype(np.int64) * 10000 + t[s != t])
    s, t = (key // 10000).astype(np.int32), (key % 10000).astype(np.int32)
    w = (1 + 9 * synth.uniform01(71, 3, 0, len(s))).astype(np.float32)
    for prog in (W.closure_program(s, t, w, W.MINPLUS, name="hubs"), W.config5(scale=16, n_sources=300)):
        base = None
        for flags in (xlog.FLAG_NO_TAG_MIRROR, 0, xlog.FLAG_NO_RESIDENT_LOOP | xlog.FLAG_NO_GROUPED_JOIN, xlog.FLAG_NO_RESIDENT_LOOP,
                      xlog.FLAG_NO_RESIDENT_LOOP | xlog.FLAG_NO_BITMAP_JOIN):
            ctx, ids, _ = xlog.load_program(prog, arena_bytes=6 << 30, flags=flags)
            r = ctx.fixpoint()
            out = ctx.read(ids[prog.outputs[0]])
            ctx.close()
            if base is None:
                base = (r, out)
                continue
            assert all(np.array_equal(a, b) for a, b in zip(base[1][0], out[0])) and np.array_equal(base[1][1].view(np.int32), out[1].view(np.int32))
            for k in ("iterations", "candidates", "new_tuples", "improved_tags", "derived_tuples"):
                assert base[0][k] == r[k], (prog.name, flags, k)


def test_chunked_candidates_match_single_batch():
    p = W.config1(300, 1500)
    a, _ = check_program(p)
    b, _ = check_program(p, candidate_chunk_bytes=64 << 10)
    assert a["derived_tuples"] == b["derived_tuples"] and a["candidates"] == b["candidates"]
    check_program(W.config2(scale=12), candidate_chunk_bytes=32 << 10)
    # batches large enough for the high-bit sort + table reduce, several per round, with a dictionary column
    # and a stream that is already ordered by its leading key bits
    c, _ = check_program(W.config5(scale=14, n_sources=32), candidate_chunk_bytes=6 << 20)
    d, _ = check_program(W.config5(scale=14, n_sources=32))
    assert c["derived_tuples"] == d["derived_tuples"] and c["candidates"] == d["candidates"]


def test_resident_graph_is_reused_and_rebuilt_when_the_inputs_change():
    # same context: repeated fixpoints launch the instantiated graph again; a reload that moves or resizes the edge
    # relation (other index pointers, other domain) must rebuild it.  Every result is checked against the oracle.
    from paper_2609_27203_b200 import xlog
    ctx, ids, _ = xlog.load_program(W.config2(scale=10), arena_bytes=1 << 28, flags=xlog.FLAG_CHECK_INVARIANTS)
    for scale in (10, 10, 12, 9, 12):
        prog = W.config2(scale=scale)
        (s, d), w = prog.facts["edge"]
        ctx.load(ids["edge"], [s, d], w)
        ctx.load(ids["dist"], [np.array([0], np.int32)], np.zeros(1, np.float32))
        o, oids, _, stats = oracle_run(prog)
        for _ in range(3):
            ctx.reset_idb()
            r = ctx.fixpoint()
            assert H.compare_relations(ctx.read(ids["dist"]), o.read(oids["dist"]), what=f"sssp scale {scale}")["bit_unequal"] == 0
            assert r["derived_tuples"] == stats["derived_tuples"]
    ctx.close()


def test_fixpoint_idempotent_and_reset():
    p = W.config1(200, 700)
    ctx, ids, _, r1 = gpu_run(p)
    first = ctx.read(ids["path"])
    r2 = ctx.fixpoint()
    assert r2["new_tuples"] == 0 and r2["improved_tags"] == 0
    assert H.compare_relations(ctx.read(ids["path"]), first)["bit_unequal"] == 0
    ctx.reset_idb()
    assert ctx.size(ids["path"]) == 0
    r3 = ctx.fixpoint()
    assert r3["derived_tuples"] == r1["derived_tuples"]
    assert H.compare_relations(ctx.read(ids["path"]), first)["bit_unequal"] == 0
    ctx.close()


def test_row_local_fixpoint_route_edges():
    # the route that runs each first-column value's rounds on its own in shared memory: (1) the iteration cap bites at
    # exactly the round where the other routes stop, (2) rows of 8192 slots (the largest it takes) with a skewed graph,
    # (3) a head that starts with loaded facts, some better and some worse than what the rule derives
    from paper_2609_27203_b200 import xlog
    chain = W.closure_program(np.arange(40), np.arange(1, 41), -np.ones(40, np.float32))
    need = oracle_run(chain, "seminaive")[3]["iterations"]
    for flags in (0, xlog.FLAG_NO_ROW_FIXPOINT):
        ctx, ids, _ = xlog.load_program(chain, arena_bytes=1 << 26, max_iterations=need, flags=flags)
        assert ctx.fixpoint()["iterations"] == need
        ctx.close()
        ctx, ids, _ = xlog.load_program(chain, arena_bytes=1 << 26, max_iterations=need - 1, flags=flags)
        with pytest.raises(xlog.XlogError) as e:
            ctx.fixpoint()
        assert e.value.status == "CONVERGENCE_FAILURE"
        ctx.close()
    prog = W.config5(scale=13, n_sources=24)
    r, _ = check_program(prog)
    ctx, ids, _ = xlog.load_program(prog, arena_bytes=1 << 28, flags=xlog.FLAG_PROFILE)
    ctx.fixpoint()
    assert "k_row_fixpoint" in ctx.profile()
    ctx.close()
    s, d = synth.uniform_digraph(300, 1200, 91)
    w = (1 + 9 * synth.uniform01(91, 2, 0, 1200)).astype(np.float32)
    srcs = np.array([2, 50, 299], np.int32)
    p2 = W.reach_program(s, d, w, srcs, W.MINPLUS, name="reach_with_facts")
    p2.facts["reach"] = ([np.array([2, 2, 50, 7], np.int32), np.array([9, 10, 11, 12], np.int32)], np.array([0.25, 500.0, 3.0, 1.0], np.float32))
    check_program(p2)


def test_typed_failures_leave_the_context_usable():
    from paper_2609_27203_b200 import xlog
    chain = W.closure_program(np.arange(30), np.arange(1, 31), -np.ones(30, np.float32))
    ctx, ids, _ = xlog.load_program(chain, arena_bytes=1 << 26, max_iterations=5)
    with pytest.raises(xlog.XlogError) as e:
        ctx.fixpoint()
    assert e.value.status == "CONVERGENCE_FAILURE"
    with pytest.raises(xlog.XlogError) as e:       # partial counters do not turn it into a result
        ctx.read(ids["path"])
    assert e.value.status == "INVALID_STATE"
    ctx.reset_idb()
    assert ctx.size(ids["path"]) == 0
    ctx.close()
    # arena too small for the closure
    big = W.config1(400, 3000)
    ctx, ids, _ = xlog.load_program(big, arena_bytes=1 << 19)
    with pytest.raises(xlog.XlogError) as e:
        ctx.fixpoint()
    assert e.value.status == "RESOURCE_EXHAUSTED"
    ctx.close()
    # NaN tag, semiring zero, negative key
    ctx = xlog.Context(arena_bytes=1 << 24)
    r = ctx.relation(1, "minplus")
    for cols, tags in [([np.array([1], np.int32)], np.array([np.nan], np.float32)),
                       ([np.array([1], np.int32)], np.array([np.inf], np.float32)),
                       ([np.array([-4], np.int32)], None)]:
        with pytest.raises(xlog.XlogError) as e:
            ctx.load(r, cols, tags)
        assert e.value.status == "INVALID_VALUE"
    ctx.load(r, [np.array([2], np.int32)], None)
    assert ctx.size(r) == 1
    # a recursive component that mixes max/min with logsumexp relations, and a non-linear rule under logsumexp
    mixed = W.Program("mixed", {"e": (1, W.MAXPLUS), "a": (1, W.MAXPLUS), "b": (1, W.LOGSUMEXP)},
                      [W.Rule("a", (W.V(0),), (W.Atom("e", (W.Var(0),)),)), W.Rule("a", (W.V(0),), (W.Atom("b", (W.Var(0),)),)),
                       W.Rule("b", (W.V(0),), (W.Atom("a", (W.Var(0),)),))], {"e": ([np.array([1, 2], np.int32)], None)})
    doubling = W.Program("doubling", {"e": (2, W.LOGSUMEXP), "p": (2, W.LOGSUMEXP)},
                         [W.Rule("p", (W.V(0), W.V(1)), (W.Atom("e", (W.Var(0), W.Var(1))),)),
                          W.Rule("p", (W.V(0), W.V(2)), (W.Atom("p", (W.Var(0), W.Var(1))), W.Atom("p", (W.Var(1), W.Var(2)))))],
                         {"e": ([np.array([0, 1], np.int32), np.array([1, 2], np.int32)], None)})
    for bad in (mixed, doubling):
        ctx2, _, _ = xlog.load_program(bad, arena_bytes=1 << 24)
        with pytest.raises(xlog.XlogError) as e:
            ctx2.fixpoint()
        assert e.value.status == "UNSUPPORTED"
        if bad is mixed:
            ctx2.close()
    # head arithmetic leaving [0, 2^31)
    prog = W.Program("ovf", {"a": (1, W.MAXPLUS), "b": (1, W.MAXPLUS)},
                     [W.Rule("b", (W.Affine(-5, ((0, 1),)),), (W.Atom("a", (W.Var(0),)),))],
                     {"a": ([np.array([1, 9], np.int32)], None)})
    ctx3, _, _ = xlog.load_program(prog, arena_bytes=1 << 24)
    with pytest.raises(xlog.XlogError) as e:
        ctx3.fixpoint()
    assert e.value.status == "CAPACITY_EXCEEDED"
    for c in (ctx, ctx2, ctx3):
        c.close()


def test_join_indices_of_unchanged_relations_are_reused_across_fixpoints():
    # the looked-up side's index (offsets, and for a non-leading column a permuted sorted copy) is built once per
    # relation generation: a second fixpoint after xlog_ctx_reset_idb builds none, a reload of the relation builds it again
    from paper_2609_27203_b200 import xlog
    p = W.config1(300, 1500)
    (s, d), t = p.facts["edge"]
    right = W.Program("right_linear", {"edge": (2, W.MAXPLUS), "path": (2, W.MAXPLUS)},
                      [W.Rule("path", (W.V(0), W.V(1)), (W.Atom("edge", (W.Var(0), W.Var(1))),)),
                       W.Rule("path", (W.V(0), W.V(2)), (W.Atom("edge", (W.Var(0), W.Var(1))), W.Atom("path", (W.Var(1), W.Var(2)))))],
                      {"edge": ([s, d], t)}, ("path",))
    for prog, flags in ((p, 0), (p, xlog.FLAG_NO_TAG_MIRROR), (right, xlog.FLAG_NO_TAG_MIRROR)):
        ctx, ids, _ = xlog.load_program(prog, arena_bytes=1 << 28, flags=flags)
        first = ctx.fixpoint()
        want = ctx.read(ids["path"])
        ctx.reset_idb()
        second = ctx.fixpoint()
        got = ctx.read(ids["path"])
        assert H.compare_relations(got, want, what="after reset")["bit_unequal"] == 0
        assert first["index_builds"] >= 1, first
        if prog is p:
            assert second["index_builds"] == 0, second            # edge's index on column 0 is still valid
        else:
            # the scanned delta of path probes edge on its SECOND column: that permuted copy is reused, the recursion's
            # own relation is not looked up at all
            assert second["index_builds"] == 0, second
        ctx.load(ids["edge"], [s, d], t)                            # a new generation of edge: its index is rebuilt
        third = ctx.fixpoint()
        assert third["index_builds"] == first["index_builds"]
        assert H.compare_relations(ctx.read(ids["path"]), want, what="after reload")["bit_unequal"] == 0
        ctx.close()


def test_path_doubling_through_the_dense_rounds_at_scale():
    # p(x,z) :- p(x,y), p(y,z) on graphs of 300 to 1000 nodes: the default route keeps p as a matrix and applies both delta
    # variants of a round row by row (no sort, no index of p); it must agree bit for bit, relation and counters, with the
    # sorting route, with the oracle where the oracle finishes in seconds, and (tuple set; tags to 1e-5) with the linear closure
    from paper_2609_27203_b200 import xlog
    small = W.nonlinear_config(300, 1200)
    r, stats = check_program(small, expect_bit_equal=True)
    assert r["candidates"] == stats["contributions"]                     # every binding of both delta variants, counted once each
    # hub-skewed, min-plus, with loaded facts of p itself (the seed round then joins the full relation with itself)
    rm = W.nonlinear_rmat_config(8)
    (s, d), w = rm.facts["e"]
    rm.facts["p"] = ([np.array([3, 200], np.int32), np.array([250, 7], np.int32)], np.array([0.5, 40.0], np.float32))
    check_program(rm)
    big = W.nonlinear_config()                                             # configuration 1's graph
    res = {}
    for flags in (0, xlog.FLAG_NO_DENSE_DOUBLING):
        ctx, ids, _ = xlog.load_program(big, arena_bytes=16 << 30, flags=flags)
        receipt = ctx.fixpoint()
        res[flags] = (receipt, ctx.read(ids["p"]))
        again = ctx.fixpoint()
        assert again["new_tuples"] == 0 and again["improved_tags"] == 0   # idempotent on both routes
        ctx.close()
    a, b = res[0], res[xlog.FLAG_NO_DENSE_DOUBLING]
    assert H.compare_relations(a[1], b[1], what="dense rounds vs sorting route")["bit_unequal"] == 0
    for k in ("iterations", "candidates", "new_tuples", "improved_tags", "derived_tuples"):
        assert a[0][k] == b[0][k], k
    lin = W.config1()
    ctx, ids, _ = xlog.load_program(lin, arena_bytes=1 << 28)
    ctx.fixpoint()
    H.compare_relations(a[1], ctx.read(ids["path"]), rel_tol=1e-5, what="path doubling vs linear closure")
    ctx.close()
