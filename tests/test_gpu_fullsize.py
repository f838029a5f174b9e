"""Parity at the full sizes of the five configurations, in the launch configuration bench.py times
(device-resident inputs, the arena sizes of bench.make_program).

Where the oracle finishes in well under a minute the whole relation is compared; otherwise
sampled outputs the oracle can compute one by one are compared (four sources of the multi-source
program, a sample of x for the triangle aggregate) together with properties that hold at any size
and with numpy / scipy restatements that share nothing with either side.
Tolerances as in test_gpu_parity.py / test_gpu_aggregates.py.
"""
import numpy as np
import pytest

import oracle
from paper_2609_27203_b200 import synth, workloads as W
from tests import helpers as H

pytestmark = pytest.mark.gpu


def gpu_fixpoint(program, arena, flags=0):
    from paper_2609_27203_b200 import xlog
    ctx, ids, rules = xlog.load_program(program, arena_bytes=arena, device_inputs=True, flags=flags)
    receipt = ctx.fixpoint()
    return ctx, ids, rules, receipt


def same_on_the_sorting_path(program, arena, name, cols, tags, receipt):
    """The default path evaluates these recursions through the tag mirror; sort -> reduce-by-key -> merge must derive
    the same relation bit for bit, with the same counters."""
    from paper_2609_27203_b200 import xlog
    ctx, ids, _, r2 = gpu_fixpoint(program, arena, xlog.FLAG_NO_TAG_MIRROR)
    c2, t2 = ctx.read(ids[name])
    ctx.close()
    assert all(np.array_equal(a, b) for a, b in zip(cols, c2)) and np.array_equal(tags.view(np.int32), t2.view(np.int32))
    for k in ("iterations", "candidates", "new_tuples", "improved_tags", "derived_tuples"):
        assert receipt[k] == r2[k], k
    assert receipt["unique_candidates"] == -1 and r2["unique_candidates"] > 0


def test_config2_sssp_rmat20_full():
    prog = W.config2()
    ctx, ids, _, receipt = gpu_fixpoint(prog, 4 << 30)
    o, oids, _ = oracle.load_program(prog)
    stats = o.run("seminaive")
    rep = H.compare_relations(ctx.read(ids["dist"]), o.read(oids["dist"]), rel_tol=1e-5, what="sssp_rmat20")
    assert rep["bit_unequal"] == 0 and receipt["derived_tuples"] == stats["derived_tuples"]
    again = ctx.fixpoint()                      # fixpoint idempotence at full size
    assert again["new_tuples"] == 0 and again["improved_tags"] == 0
    cols, tags = ctx.read(ids["dist"])
    ctx.close()
    same_on_the_sorting_path(prog, 4 << 30, "dist", cols, tags, receipt)


def test_config4_digits_full_forward_and_backward():
    import torch
    prog = W.config4()
    B = prog.info["n_pairs"]
    ctx, ids, rules, receipt = gpu_fixpoint(prog, 1 << 30)
    cols, tags = ctx.read(ids["sum"])
    assert len(tags) == 19 * B and receipt["candidates"] == 100 * B
    # closed form for every row: log of the discrete convolution of the two softmax vectors (fp64)
    lt = prog.facts["digit"][1].reshape(2 * B, 10).astype(np.float64)
    P = np.exp(lt)
    conv = np.zeros((B, 19))
    for a in range(10):
        conv[:, a:a + 10] += P[0::2, a:a + 1] * P[1::2]
    assert np.all(np.abs(tags.reshape(B, 19) - np.log(conv)) < 1e-4)
    # the oracle, every row: forward and gradient
    o, oids, orules = oracle.load_program(prog)
    o.run("naive")
    H.compare_relations((cols, tags), o.read(oids["sum"]), abs_tol=1e-4, what="digits")
    g = synth.head_gradient(19 * B, 4)
    got = ctx.backward(rules[0], torch.from_numpy(g).cuda())[0].cpu().numpy().astype(np.float64)
    og = o.backward(orules[0], g)
    ref = og[0].astype(np.float64) + og[1].astype(np.float64)
    assert np.all(np.abs(got - ref) <= 1e-5 + 1e-4 * np.abs(ref))
    # softmax weights of one pair's 19 rows: the gradient of sum_s out(p,s) w.r.t. the ten tags of image 2p sums to 19
    ones = ctx.backward(rules[0], torch.ones(19 * B, device="cuda"))[0].cpu().numpy().reshape(2 * B, 10)
    assert np.allclose(ones.sum(axis=1), 19.0, atol=2e-4)
    ctx.close()


def _triangle_terms_of(x, off, d, w, n):
    """Every term (w_xy + w_yz) + w_zx of x's triangles in float64, straight from the edge arrays (numpy only)."""
    in_w = np.full(n, np.nan)
    zs_in = np.flatnonzero(d == x)                       # edges (z, x): rows whose destination is x
    src_of = np.searchsorted(off, zs_in, side="right") - 1
    in_w[src_of] = w[zs_in]
    terms = []
    ys = d[off[x]:off[x + 1]]
    wxy = w[off[x]:off[x + 1]].astype(np.float64)
    step = 256
    for a in range(0, len(ys), step):
        yb = ys[a:a + step]
        lens = (off[yb + 1] - off[yb]).astype(np.int64)
        if lens.sum() == 0:
            continue
        idx = np.repeat(off[yb].astype(np.int64) - np.concatenate([[0], np.cumsum(lens)[:-1]]), lens) + np.arange(lens.sum())
        z = d[idx]
        hit = ~np.isnan(in_w[z])
        t = (np.repeat(wxy[a:a + step], lens)[hit] + w[idx][hit].astype(np.float64)) + in_w[z[hit]]
        terms.append(t)
    return np.concatenate(terms) if terms else np.zeros(0)


def test_config3_triangles_rmat18_full_sampled():
    import scipy.sparse as sp
    prog = W.config3()
    n = 1 << 18
    ctx, ids, _, receipt = gpu_fixpoint(prog, 2 << 30)
    cols, tags = ctx.read(ids["tri_agg"])
    ctx.close()
    xs, counts = cols[0], cols[1].astype(np.int64)
    assert counts.sum() % 3 == 0 and np.all(counts > 0) and np.all(np.diff(xs) > 0)
    got = {int(x): (int(c), float(t)) for x, c, t in zip(xs, counts, tags)}
    (s, d), w = prog.facts["e"]                          # sorted by (s, d)
    deg = np.bincount(s, minlength=n)
    off = np.concatenate([[0], np.cumsum(deg)])

    # (1) the group with the most terms, against a float64 sum over its terms written out with numpy
    big = int(xs[np.argmax(counts)])
    terms = _triangle_terms_of(big, off, d, w, n)
    assert len(terms) == got[big][0] > 1_000_000, f"count of the largest group x={big}"
    m = terms.max()
    assert abs(got[big][1] - (m + np.log(np.exp(terms - m).sum()))) < 1e-4, f"logsumexp of the largest group x={big}"

    # (2) counts of every x with x % 64 == 0 (4,096 nodes, the hub among them) against a sparse matrix product:
    #     count(x) = sum over y, z of A[x,y] A[y,z] A[z,x]; x without a triangle must be absent
    A = sp.csr_matrix((np.ones(len(s), np.int64), (s, d)), shape=(n, n))
    S = np.arange(0, n, 64)
    ref = np.asarray((A[S] @ A).multiply(A[:, S].T.tocsr()).sum(axis=1)).ravel()
    mine = np.zeros(n, np.int64)
    mine[xs] = counts
    assert np.array_equal(mine[S], ref)
    assert int(ref.sum()) > 10_000_000

    # (3) sampled x computed by the oracle alone with x fixed as a constant: twelve of moderate degree, and four from the
    #     top decile by count (those whose two-paths number at most 3 M, so that the oracle's nested loops finish in seconds),
    #     and the largest group once more, this time by the oracle
    cand = xs[(deg[xs] >= 2) & (deg[xs] <= 300)]
    pick = cand[synth.randint(3, 7, 0, 12, len(cand))].tolist()
    two_paths = np.asarray((A[xs] @ sp.csr_matrix(deg.reshape(-1, 1))).todense()).ravel()
    top = xs[(counts >= np.quantile(counts, 0.9)) & (two_paths <= 3_000_000)]
    assert len(top) >= 4
    pick += top[synth.randint(3, 8, 0, 4, len(top))].tolist() + [big]
    o = oracle.Oracle()
    e = o.relation(2, W.LOGSUMEXP)
    o.load(e, [s, d], w)
    heads = []
    for x in pick:
        h = o.relation(2, W.LOGSUMEXP)
        o.rule(h, [(x, {})], [(e, [("c", x), ("v", 1, 1, 0)]), (e, [("v", 1, 1, 0), ("v", 2, 1, 0)]), (e, [("v", 2, 1, 0), ("c", x)])], True)
        heads.append(h)
    o.run("naive")
    for x, h in zip(pick, heads):
        oc, ot = o.read(h)
        assert len(ot) == 1 and int(oc[0][0]) == x
        assert got[x][0] == int(oc[1][0]), f"count of x={x}"
        assert abs(got[x][1] - float(ot[0])) < 1e-4, f"logsumexp of x={x}"


def _oracle_reach_rows(edges, sources):
    """reach(s, .) of the given sources by the oracle alone (its own instance: callers run several in threads)."""
    (s, d), w = edges
    o, oids, _ = oracle.load_program(W.reach_program(s, d, w, np.asarray(sources, np.int32)))
    o.run("seminaive")
    return o.read(oids["reach"])


def test_config5_reach_rmat22_full_four_sources_by_oracle():
    from concurrent.futures import ThreadPoolExecutor
    prog = W.config5()
    (s, d), w = prog.facts["edge"]
    srcs = prog.facts["src"][0][0]
    deg = np.bincount(s, minlength=1 << 22)
    live = srcs[deg[srcs] > 0]
    # four live sources, the one with the most out-edges among them; two oracle instances run side by side (the C++ engine
    # runs outside the interpreter lock), two sources each
    by_deg = live[np.argsort(-deg[live], kind="stable")]
    chosen = [int(by_deg[0]), int(live[0]) if int(live[0]) != int(by_deg[0]) else int(live[1])]
    chosen += [int(x) for x in live[::-1] if int(x) not in chosen][:2]
    pool = ThreadPoolExecutor(2)
    jobs = [pool.submit(_oracle_reach_rows, prog.facts["edge"], chosen[0:2]), pool.submit(_oracle_reach_rows, prog.facts["edge"], chosen[2:4])]

    ctx, ids, _, receipt = gpu_fixpoint(prog, 56 << 30)
    rc, rt = ctx.read(ids["reach"])
    assert receipt["derived_tuples"] == len(rt) and np.array_equal(np.unique(rc[0]), np.sort(srcs))
    # every source reaches itself at distance 0; keys ascending (s, z)
    key = rc[0].astype(np.int64) << 22 | rc[1]
    assert np.all(np.diff(key) > 0)
    self_rows = rc[0] == rc[1]
    assert self_rows.sum() == len(srcs) and np.all(rt[self_rows] == 0.0)
    # sources without out-edges reach only themselves
    for dead in srcs[deg[srcs] == 0][:5].tolist():
        assert int((rc[0] == dead).sum()) == 1
    ctx.close()
    same_on_the_sorting_path(prog, 56 << 30, "reach", rc, rt, receipt)
    for job in jobs:
        oc, ot = job.result()
        sel = np.isin(rc[0], np.unique(oc[0]))
        assert np.array_equal(rc[0][sel], oc[0]) and np.array_equal(rc[1][sel], oc[1])
        assert np.array_equal(rt[sel].view(np.int32), ot.view(np.int32))
        assert len(ot) > 2_000_000
    pool.shutdown()


def test_resident_rounds_over_a_23_bit_key_space():
    # 128 sources on R-MAT 16: 7 + 16 key bits, the largest class of key space the resident rounds take (up to 2^24) and the
    # only one whose bitmap tiles are swept four times per block; the graph-driven rounds, the same launched one by one, and
    # the sorting path must agree bit for bit, and three sources are checked row by row against the oracle
    from paper_2609_27203_b200 import xlog
    prog = W.config5(scale=16, n_sources=128)
    (s, d), w = prog.facts["edge"]
    srcs = prog.facts["src"][0][0]
    deg = np.bincount(s, minlength=1 << 16)
    live = srcs[deg[srcs] > 0]
    ctx, ids, _, receipt = gpu_fixpoint(prog, 8 << 30)
    rc, rt = ctx.read(ids["reach"])
    ctx.close()
    assert receipt["derived_tuples"] == len(rt) and receipt["kernel_launches"] < 60       # resident: a handful of launches outside the loop
    ctx, ids, _, r1 = gpu_fixpoint(prog, 8 << 30, xlog.FLAG_NO_GRAPH)
    c1, t1 = ctx.read(ids["reach"])
    ctx.close()
    assert all(np.array_equal(a, b) for a, b in zip(rc, c1)) and np.array_equal(rt.view(np.int32), t1.view(np.int32))
    for k in ("iterations", "candidates", "new_tuples", "improved_tags", "derived_tuples"):
        assert receipt[k] == r1[k], k
    same_on_the_sorting_path(prog, 8 << 30, "reach", rc, rt, receipt)
    chosen = [int(live[0]), int(live[len(live) // 2]), int(live[-1])]
    oc, ot = _oracle_reach_rows(prog.facts["edge"], chosen)
    sel = np.isin(rc[0], np.unique(oc[0]))
    assert np.array_equal(rc[0][sel], oc[0]) and np.array_equal(rc[1][sel], oc[1])
    assert np.array_equal(rt[sel].view(np.int32), ot.view(np.int32))


def test_mutual_recursion_full_size_against_the_oracle():
    # odd / even walks on configuration 1's graph: two mutually recursive heads, 1.9 M derived tuples, every row by the oracle
    prog = W.mutual_config()
    ctx, ids, _, receipt = gpu_fixpoint(prog, 2 << 30)
    o, oids, _ = oracle.load_program(prog)
    stats = o.run("seminaive")
    for name in ("odd", "even"):
        rep = H.compare_relations(ctx.read(ids[name]), o.read(oids[name]), rel_tol=1e-5, what=name)
        assert rep["bit_unequal"] == 0
    assert receipt["derived_tuples"] == stats["derived_tuples"] and receipt["candidates"] == stats["contributions"]
    assert receipt["iterations"] == stats["iterations"]
    ctx.close()
