"""The five benchmark programs as plain data (relations, rules, loaded facts).

A ``Program`` is only a description: which relations exist, which rules derive
them and which arrays are loaded.  It is handed unchanged to the CUDA binding
and (in tests) to the CPU oracle; it performs no evaluation itself.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

from . import synth

MAXPLUS, MINPLUS, LOGSUMEXP, SUMPROD = "maxplus", "minplus", "logsumexp", "sumprod"


@dataclass(frozen=True)
class Const:
    value: int


@dataclass(frozen=True)
class Var:
    """Column pattern ``column == mul * var + add`` (mul > 0)."""
    var: int
    mul: int = 1
    add: int = 0


@dataclass(frozen=True)
class Affine:
    """Head column ``c0 + sum(coef[v] * v)``."""
    c0: int = 0
    coef: Tuple[Tuple[int, int], ...] = ()      # ((var, coefficient), ...)


def V(v: int) -> Affine:
    return Affine(0, ((v, 1),))


@dataclass(frozen=True)
class Atom:
    rel: str
    args: Tuple[object, ...]
    negated: bool = False          # negation as failure over a relation of a lower stratum


@dataclass(frozen=True)
class Rule:
    head: str
    head_exprs: Tuple[Affine, ...]
    atoms: Tuple[Atom, ...]
    emit_count: bool = False


@dataclass
class Program:
    name: str
    relations: Dict[str, Tuple[int, str]]                     # name -> (arity, semiring)
    rules: List[Rule]
    facts: Dict[str, Tuple[List[np.ndarray], Optional[np.ndarray]]] = field(default_factory=dict)
    outputs: Sequence[str] = ()
    info: Dict[str, object] = field(default_factory=dict)


# ----------------------------------------------------------------------------

def closure_program(src, dst, tag, semiring=MAXPLUS, name="closure") -> Program:
    """path(x,y) :- edge(x,y).  path(x,z) :- path(x,y), edge(y,z)."""
    return Program(
        name=name,
        relations={"edge": (2, semiring), "path": (2, semiring)},
        rules=[
            Rule("path", (V(0), V(1)), (Atom("edge", (Var(0), Var(1))),)),
            Rule("path", (V(0), V(2)), (Atom("path", (Var(0), Var(1))), Atom("edge", (Var(1), Var(2))))),
        ],
        facts={"edge": ([np.ascontiguousarray(src, np.int32), np.ascontiguousarray(dst, np.int32)],
                        None if tag is None else np.ascontiguousarray(tag, np.float32))},
        outputs=("path",),
    )


def sssp_program(src, dst, w, source=0, semiring=MINPLUS, name="sssp") -> Program:
    """dist(s) = 0 loaded as a fact.  dist(y) :- dist(x), edge(x,y)."""
    return Program(
        name=name,
        relations={"edge": (2, semiring), "dist": (1, semiring)},
        rules=[Rule("dist", (V(1),), (Atom("dist", (Var(0),)), Atom("edge", (Var(0), Var(1)))))],
        facts={"edge": ([np.ascontiguousarray(src, np.int32), np.ascontiguousarray(dst, np.int32)],
                        np.ascontiguousarray(w, np.float32)),
               "dist": ([np.asarray([source], np.int32)], np.zeros(1, np.float32))},
        outputs=("dist",),
    )


def reach_program(src, dst, w, sources, semiring=MINPLUS, name="reach") -> Program:
    """reach(s,s) :- src(s).  reach(s,z) :- reach(s,y), edge(y,z)."""
    return Program(
        name=name,
        relations={"edge": (2, semiring), "src": (1, semiring), "reach": (2, semiring)},
        rules=[
            Rule("reach", (V(0), V(0)), (Atom("src", (Var(0),)),)),
            Rule("reach", (V(0), V(2)), (Atom("reach", (Var(0), Var(1))), Atom("edge", (Var(1), Var(2))))),
        ],
        facts={"edge": ([np.ascontiguousarray(src, np.int32), np.ascontiguousarray(dst, np.int32)],
                        np.ascontiguousarray(w, np.float32)),
               "src": ([np.ascontiguousarray(sources, np.int32)], None)},
        outputs=("reach",),
    )


def triangle_program(src, dst, w, name="triangles") -> Program:
    """tri_agg(x, count) :- e(x,y), e(y,z), e(z,x); tag = logsumexp of (w_xy + w_yz) + w_zx."""
    return Program(
        name=name,
        relations={"e": (2, LOGSUMEXP), "tri_agg": (2, LOGSUMEXP)},
        rules=[Rule("tri_agg", (V(0),),
                    (Atom("e", (Var(0), Var(1))), Atom("e", (Var(1), Var(2))), Atom("e", (Var(2), Var(0)))),
                    emit_count=True)],
        facts={"e": ([np.ascontiguousarray(src, np.int32), np.ascontiguousarray(dst, np.int32)],
                     np.ascontiguousarray(w, np.float32))},
        outputs=("tri_agg",),
    )


def triangle_rows_program(src, dst, w, semiring=MAXPLUS, name="triangle_rows") -> Program:
    """tri(x,y,z) :- e(x,y), e(y,z), e(z,x): the materialised three-way cyclic join; tag = (w_xy + w_yz) + w_zx."""
    return Program(
        name=name,
        relations={"e": (2, semiring), "tri": (3, semiring)},
        rules=[Rule("tri", (V(0), V(1), V(2)),
                    (Atom("e", (Var(0), Var(1))), Atom("e", (Var(1), Var(2))), Atom("e", (Var(2), Var(0)))))],
        facts={"e": ([np.ascontiguousarray(src, np.int32), np.ascontiguousarray(dst, np.int32)],
                     np.ascontiguousarray(w, np.float32))},
        outputs=("tri",),
    )


def triangle_join_program(r, s, t, semiring=MAXPLUS, name="triangle_join") -> Program:
    """tri(x,y,z) :- r(x,y), s(y,z), t(z,x) over three relations, each given as (col0, col1, tags)."""
    def rel(x):
        return ([np.ascontiguousarray(x[0], np.int32), np.ascontiguousarray(x[1], np.int32)], np.ascontiguousarray(x[2], np.float32))
    return Program(
        name=name,
        relations={"r": (2, semiring), "s": (2, semiring), "t": (2, semiring), "tri": (3, semiring)},
        rules=[Rule("tri", (V(0), V(1), V(2)),
                    (Atom("r", (Var(0), Var(1))), Atom("s", (Var(1), Var(2))), Atom("t", (Var(2), Var(0)))))],
        facts={"r": rel(r), "s": rel(s), "t": rel(t)},
        outputs=("tri",),
    )


def four_cycle_program(r, s, t, u, semiring=MAXPLUS, name="four_cycle") -> Program:
    """c4(x,y,z,w) :- r(x,y), s(y,z), t(z,w), u(w,x) over four relations, each given as (col0, col1, tags)."""
    def rel(x):
        return ([np.ascontiguousarray(x[0], np.int32), np.ascontiguousarray(x[1], np.int32)], np.ascontiguousarray(x[2], np.float32))
    return Program(
        name=name,
        relations={"r": (2, semiring), "s": (2, semiring), "t": (2, semiring), "u": (2, semiring), "c4": (4, semiring)},
        rules=[Rule("c4", (V(0), V(1), V(2), V(3)),
                    (Atom("r", (Var(0), Var(1))), Atom("s", (Var(1), Var(2))), Atom("t", (Var(2), Var(3))), Atom("u", (Var(3), Var(0)))))],
        facts={"r": rel(r), "s": rel(s), "t": rel(t), "u": rel(u)},
        outputs=("c4",),
    )


def uniform_four_cycle(n_rows=3000, domain=120, semiring=MAXPLUS, seed=synth.SEED_BASE + 7) -> Program:
    """Four relations of n_rows distinct uniform pairs over `domain` values (tags: log-probabilities)."""
    rels = []
    for k in range(4):
        a, b = synth.uniform_digraph(domain, n_rows, seed + 17 * k)
        rels.append((a, b, synth.log_prob_tags(n_rows, seed + 17 * k + 1)))
    p = four_cycle_program(*rels, semiring=semiring, name=f"four_cycle_n{n_rows}_d{domain}")
    p.info.update(n_rows=n_rows, domain=domain)
    return p


def hot_domain_triangle(n_rows=65536, domain=406, seed=synth.SEED_BASE + 6) -> Program:
    """Three relations of n_rows distinct uniform pairs over a small domain: every join variable is hot, so the two-paths
    of any two relations far outnumber the triangles (65,536 rows over 406 values: about 10.6 M two-paths, 4.2 M triples)."""
    rels = []
    for k in range(3):
        a, b = synth.uniform_digraph(domain, n_rows, seed + 17 * k)
        rels.append((a, b, synth.log_prob_tags(n_rows, seed + 17 * k + 1)))
    p = triangle_join_program(*rels, name=f"triangle_join_hot{domain}_n{n_rows}")
    p.info.update(n_rows=n_rows, domain=domain)
    return p


def nonlinear_closure_program(src, dst, tag, semiring=MAXPLUS, name="nonlinear_closure") -> Program:
    """p(x,y) :- e(x,y).  p(x,z) :- p(x,y), p(y,z): path doubling, two recursive atoms in one rule."""
    return Program(
        name=name,
        relations={"e": (2, semiring), "p": (2, semiring)},
        rules=[
            Rule("p", (V(0), V(1)), (Atom("e", (Var(0), Var(1))),)),
            Rule("p", (V(0), V(2)), (Atom("p", (Var(0), Var(1))), Atom("p", (Var(1), Var(2))))),
        ],
        facts={"e": ([np.ascontiguousarray(src, np.int32), np.ascontiguousarray(dst, np.int32)],
                     None if tag is None else np.ascontiguousarray(tag, np.float32))},
        outputs=("p",),
    )


def odd_even_program(src, dst, w, semiring=MINPLUS, name="odd_even") -> Program:
    """odd(x,y) :- e(x,y).  even(x,z) :- odd(x,y), e(y,z).  odd(x,z) :- even(x,y), e(y,z): two mutually recursive heads
    (best walks of odd / even length)."""
    return Program(
        name=name,
        relations={"e": (2, semiring), "odd": (2, semiring), "even": (2, semiring)},
        rules=[
            Rule("odd", (V(0), V(1)), (Atom("e", (Var(0), Var(1))),)),
            Rule("even", (V(0), V(2)), (Atom("odd", (Var(0), Var(1))), Atom("e", (Var(1), Var(2))))),
            Rule("odd", (V(0), V(2)), (Atom("even", (Var(0), Var(1))), Atom("e", (Var(1), Var(2))))),
        ],
        facts={"e": ([np.ascontiguousarray(src, np.int32), np.ascontiguousarray(dst, np.int32)],
                     np.ascontiguousarray(w, np.float32))},
        outputs=("odd", "even"),
    )


def nonlinear_config(n_nodes=1000, n_edges=4000) -> Program:
    """Path doubling on configuration 1's graph."""
    seed = synth.SEED_BASE + 1
    s, d = synth.uniform_digraph(n_nodes, n_edges, seed)
    p = nonlinear_closure_program(s, d, synth.log_prob_tags(n_edges, seed), MAXPLUS, name=f"nonlinear_closure_n{n_nodes}_m{n_edges}")
    p.info.update(n_nodes=n_nodes, n_edges=n_edges)
    return p


def nonlinear_rmat_config(scale=10, edge_factor=4) -> Program:
    """Path doubling on a small R-MAT graph (hub-skewed: a few nodes reach and are reached by most of the others)."""
    seed = synth.SEED_BASE + 8
    s, d, w = synth.rmat_graph(scale, edge_factor, seed, "u1_10")
    p = nonlinear_closure_program(s, d, w, MINPLUS, name=f"nonlinear_closure_rmat{scale}")
    p.info.update(scale=scale, n_nodes=1 << scale, n_edges=int(s.size))
    return p


def mutual_config(n_nodes=1000, n_edges=4000) -> Program:
    """Odd / even walks on configuration 1's graph with weights uniform in [1, 10]."""
    seed = synth.SEED_BASE + 1
    s, d = synth.uniform_digraph(n_nodes, n_edges, seed)
    w = (1.0 + 9.0 * synth.uniform01(seed, 9, 0, n_edges)).astype(np.float32)
    p = odd_even_program(s, d, w, MINPLUS, name=f"odd_even_n{n_nodes}_m{n_edges}")
    p.info.update(n_nodes=n_nodes, n_edges=n_edges)
    return p


def digits_program(log_tags: np.ndarray, name="digits") -> Program:
    """sum(p, a+b) :- digit(2p, a), digit(2p+1, b), logsumexp per (p, a+b).

    ``log_tags`` is [2B, 10]; digit(i, d) carries log_tags[i, d]."""
    n_img = log_tags.shape[0]
    img = np.repeat(np.arange(n_img, dtype=np.int32), 10)
    dig = np.tile(np.arange(10, dtype=np.int32), n_img)
    return Program(
        name=name,
        relations={"digit": (2, LOGSUMEXP), "sum": (2, LOGSUMEXP)},
        rules=[Rule("sum", (V(0), Affine(0, ((1, 1), (2, 1)))),
                    (Atom("digit", (Var(0, 2, 0), Var(1))), Atom("digit", (Var(0, 2, 1), Var(2)))))],
        facts={"digit": ([img, dig], np.ascontiguousarray(log_tags.reshape(-1), np.float32))},
        outputs=("sum",),
    )


# ----------------------------------------------------------------------------
# the five configurations, with a size knob each
# ----------------------------------------------------------------------------

def config1(n_nodes=1000, n_edges=4000) -> Program:
    seed = synth.SEED_BASE + 1
    s, d = synth.uniform_digraph(n_nodes, n_edges, seed)
    t = synth.log_prob_tags(n_edges, seed)
    p = closure_program(s, d, t, MAXPLUS, name=f"closure_n{n_nodes}_m{n_edges}")
    p.info.update(n_nodes=n_nodes, n_edges=n_edges)
    return p


def config2(scale=20, edge_factor=16) -> Program:
    seed = synth.SEED_BASE + 2
    s, d, w = synth.rmat_graph(scale, edge_factor, seed, "u1_10")
    p = sssp_program(s, d, w, 0, MINPLUS, name=f"sssp_rmat{scale}")
    p.info.update(scale=scale, n_nodes=1 << scale, n_edges=int(s.size))
    return p


def config3(scale=18, edge_factor=16) -> Program:
    seed = synth.SEED_BASE + 3
    s, d, w = synth.rmat_graph(scale, edge_factor, seed, "n01")
    p = triangle_program(s, d, w, name=f"triangles_rmat{scale}")
    p.info.update(scale=scale, n_nodes=1 << scale, n_edges=int(s.size))
    return p


def config4(n_pairs=65536) -> Program:
    seed = synth.SEED_BASE + 4
    lt = synth.digit_log_tags(2 * n_pairs, seed)
    p = digits_program(lt, name=f"digits_B{n_pairs}")
    p.info.update(n_pairs=n_pairs)
    return p


def config5(scale=22, edge_factor=16, n_sources=64) -> Program:
    seed = synth.SEED_BASE + 5
    s, d, w = synth.rmat_graph(scale, edge_factor, seed, "u1_10")
    srcs = np.sort(synth.distinct_sources(1 << scale, n_sources, seed))
    p = reach_program(s, d, w, srcs, MINPLUS, name=f"reach_rmat{scale}_s{n_sources}")
    p.info.update(scale=scale, n_nodes=1 << scale, n_edges=int(s.size), n_sources=n_sources)
    return p
