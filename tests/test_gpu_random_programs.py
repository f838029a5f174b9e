"""Differential test: seeded random programs inside the supported plan shapes, every engine route against the oracle.
Tolerances as in the other parity tests: tuple sets exact, max/min tags 1e-5 relative, logsumexp tags 1e-4 absolute."""
import pytest

import oracle
from paper_2609_27203_b200 import workloads as W
from tests import helpers as H
from tests.random_programs import random_program

pytestmark = pytest.mark.gpu

# seeds that once failed: 37 (a rule variant without candidates after a full batch left unreduced rows), 214 (triangle
# chain without two-paths), 219 / 43 / 199 (a recursive head that stays empty)
SEEDS = sorted(set(range(80)) | {199, 214, 219})


@pytest.mark.parametrize("chunk", range(4))
def test_random_programs_agree_with_the_oracle_on_every_route(chunk):
    from paper_2609_27203_b200 import xlog
    routes = (0, xlog.FLAG_NO_ROW_FIXPOINT, xlog.FLAG_NO_GRAPH, xlog.FLAG_NO_RESIDENT_LOOP, xlog.FLAG_NO_RESIDENT_LOOP | xlog.FLAG_NO_BITMAP_JOIN,
              xlog.FLAG_NO_RESIDENT_LOOP | xlog.FLAG_NO_GROUPED_JOIN, xlog.FLAG_NO_TAG_MIRROR)
    for seed in SEEDS[chunk::4]:
        p = random_program(seed)
        o, oids, _ = oracle.load_program(p)
        st = o.run("seminaive")
        for extra in routes:
            ctx, gids, _ = xlog.load_program(p, arena_bytes=1 << 27, flags=xlog.FLAG_CHECK_INVARIANTS | extra)
            r = ctx.fixpoint()
            for name in p.outputs:
                tol = dict(abs_tol=1e-4) if p.relations[name][1] == W.LOGSUMEXP else dict(rel_tol=1e-5)
                H.compare_relations(ctx.read(gids[name]), o.read(oids[name]), what=f"{p.name}:{name}:route {extra}", **tol)
            assert r["derived_tuples"] == st["derived_tuples"], (p.name, extra)
            ctx.close()


def _compare(ctx, gids, o, oids, p, what):
    for name in p.outputs:
        tol = dict(abs_tol=1e-4) if p.relations[name][1] == W.LOGSUMEXP else dict(rel_tol=1e-5)
        H.compare_relations(ctx.read(gids[name]), o.read(oids[name]), what=f"{p.name}:{name}:{what}", **tol)


def test_random_programs_with_wide_keys_small_batches_and_reloaded_facts():
    import numpy as np
    from paper_2609_27203_b200 import xlog
    from tests.random_programs import stretch
    for seed in range(100, 124):
        p = random_program(seed)
        o, oids, _ = oracle.load_program(p)
        st = o.run("seminaive")
        plain = all(tag not in p.name for tag in ("agg3", "agg4", "shape8"))     # affine patterns / more than two columns
        for extra in (0, xlog.FLAG_NO_RESIDENT_LOOP, xlog.FLAG_NO_TAG_MIRROR):
            if plain:
                # every value times 3001 plus 5: columns of about 20 bits, 64-bit packed keys
                q = stretch(p, 3001, 5)
                oq, oqids, _ = oracle.load_program(q)
                stq = oq.run("seminaive")
                ctx, gids, _ = xlog.load_program(q, arena_bytes=1 << 27, flags=xlog.FLAG_CHECK_INVARIANTS | extra)
                assert ctx.fixpoint()["derived_tuples"] == stq["derived_tuples"] == st["derived_tuples"]
                _compare(ctx, gids, oq, oqids, q, f"stretched, route {extra}")
                ctx.close()
            # candidate batches of 4 KB (counted aggregates need one batch: left out)
            if "agg1" not in p.name:
                ctx, gids, _ = xlog.load_program(p, arena_bytes=1 << 27, flags=xlog.FLAG_CHECK_INVARIANTS | extra, candidate_chunk_bytes=4096)
                try:
                    assert ctx.fixpoint()["derived_tuples"] == st["derived_tuples"]
                    _compare(ctx, gids, o, oids, p, f"4 KB batches, route {extra}")
                except xlog.XlogError as ex:
                    assert ex.status == "RESOURCE_EXHAUSTED" and "loaded facts" in str(ex)      # facts must fit one batch
                ctx.close()
            # twice on one context, then e reloaded (rows dropped, tags changed) and evaluated again
            ctx, gids, _ = xlog.load_program(p, arena_bytes=1 << 27, flags=xlog.FLAG_CHECK_INVARIANTS | extra)
            for _ in range(2):
                assert ctx.fixpoint()["derived_tuples"] == st["derived_tuples"]
                _compare(ctx, gids, o, oids, p, f"run twice, route {extra}")
            (a, b), t = p.facts["e"]
            keep = np.arange(len(a)) % 3 != 1
            t2 = t.copy()
            t2[::2] = t2[::2] + np.float32(1.0) if p.relations["e"][1] == W.MINPLUS else t2[::2] * np.float32(0.5)
            q = W.Program(p.name + "_reloaded", dict(p.relations), list(p.rules), dict(p.facts), p.outputs)
            q.facts["e"] = ([a[keep], b[keep]], t2[keep])
            ctx.load(gids["e"], q.facts["e"][0], q.facts["e"][1])
            o2, oids2, _ = oracle.load_program(q)
            st2 = o2.run("seminaive")
            assert ctx.fixpoint()["derived_tuples"] == st2["derived_tuples"]
            _compare(ctx, gids, o2, oids2, q, f"after reload, route {extra}")
            ctx.close()
