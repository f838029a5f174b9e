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
    routes = (0, xlog.FLAG_NO_GRAPH, xlog.FLAG_NO_RESIDENT_LOOP, xlog.FLAG_NO_RESIDENT_LOOP | xlog.FLAG_NO_GROUPED_JOIN,
              xlog.FLAG_NO_TAG_MIRROR)
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
