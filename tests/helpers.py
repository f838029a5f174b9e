"""Test-only helpers: golden-file reader, relation comparison, independent textbook checkers."""
from __future__ import annotations

import heapq
import itertools
import os
from typing import Dict, List

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def read_golden(name: str) -> Dict[str, np.ndarray]:
    """Sections ``[name]`` of whitespace-separated numeric rows; '#' lines are comments."""
    out: Dict[str, List[List[float]]] = {}
    cur = None
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            if line.startswith("["):
                cur = line.strip("[]")
                out[cur] = []
            else:
                out[cur].append([float(x) for x in line.split()])
    return {k: np.asarray(v, np.float64) for k, v in out.items()}


def relation_dict(cols, tags):
    return {tuple(int(c[i]) for c in cols): np.float32(tags[i]) for i in range(len(tags))}


def compare_relations(got, want, rel_tol=0.0, abs_tol=0.0, what=""):
    """Walk two sorted relations in lock step: keys must be identical; tags within tolerance.

    Returns a report dict (max abs / rel / ulp difference, count of bit-unequal tags)."""
    gc, gt = got
    wc, wt = want
    assert len(gt) == len(wt), f"{what}: row count {len(gt)} != {len(wt)}"
    for c, (a, b) in enumerate(zip(gc, wc)):
        a = np.asarray(a); b = np.asarray(b)
        if not np.array_equal(a, b):
            i = int(np.flatnonzero(a != b)[0])
            raise AssertionError(f"{what}: first key mismatch at row {i} column {c}: {a[i]} != {b[i]}")
    g = np.asarray(gt, np.float32); w = np.asarray(wt, np.float32)
    if len(g) == 0:
        return dict(rows=0, max_abs=0.0, max_rel=0.0, max_ulp=0, bit_unequal=0)
    d = np.abs(g.astype(np.float64) - w.astype(np.float64))
    rel = d / np.maximum(np.abs(w.astype(np.float64)), 1e-300)
    gi = g.view(np.int32).astype(np.int64); wi = w.view(np.int32).astype(np.int64)
    gi = np.where(gi < 0, -(gi & 0x7FFFFFFF), gi); wi = np.where(wi < 0, -(wi & 0x7FFFFFFF), wi)
    rep = dict(rows=len(g), max_abs=float(d.max()), max_rel=float(rel.max()),
               max_ulp=int(np.abs(gi - wi).max()), bit_unequal=int((g.view(np.int32) != w.view(np.int32)).sum()))
    bad = d > (abs_tol + rel_tol * np.abs(w.astype(np.float64)))
    if bad.any():
        i = int(np.flatnonzero(bad)[0])
        raise AssertionError(f"{what}: tag mismatch at row {i}: {g[i]!r} vs {w[i]!r}; report {rep}")
    return rep


# ---- independent textbook routines (none of them shares code with oracle/ or the CUDA path) ----

def csr(n, src, dst, w):
    order = np.lexsort((dst, src))
    s, d, ww = np.asarray(src)[order], np.asarray(dst)[order], np.asarray(w)[order]
    off = np.zeros(n + 1, np.int64)
    np.add.at(off, s + 1, 1)
    return np.cumsum(off), d, ww


def dijkstra_f32(n, off, dst, w, source, start_is_fact=True):
    """Single-source shortest paths with every addition rounded to fp32 (heap Dijkstra).

    With positive weights fl(a+w) is monotone in a, so this equals the min over all walks of the
    left-folded fp32 sum, i.e. exactly the min-plus fixpoint tags."""
    dist = np.full(n, np.inf, np.float32)
    done = np.zeros(n, bool)
    heap = []
    if start_is_fact:
        dist[source] = np.float32(0)
        heap.append((0.0, source))
    while heap:
        du, u = heapq.heappop(heap)
        if done[u]:
            continue
        done[u] = True
        for e in range(off[u], off[u + 1]):
            v = int(dst[e])
            nd = np.float32(np.float32(du) + np.float32(w[e]))
            if nd < dist[v]:
                dist[v] = nd
                heapq.heappush(heap, (float(nd), v))
    return dist


def floyd_warshall(n, src, dst, w, maximize):
    """All-pairs best walk value in fp64 with the diagonal initialised to the semiring zero
    (a tuple (x,x) needs at least one edge)."""
    zero = -np.inf if maximize else np.inf
    D = np.full((n, n), zero, np.float64)
    for s, d, ww in zip(src, dst, w):
        D[s, d] = max(D[s, d], ww) if maximize else min(D[s, d], ww)
    for k in range(n):
        via = D[:, k:k + 1] + D[k:k + 1, :]
        D = np.maximum(D, via) if maximize else np.minimum(D, via)
    return D


def reachable_pairs(n, src, dst):
    """Set of (x,y) with a walk of length >= 1 from x to y, by BFS per source."""
    adj = [[] for _ in range(n)]
    for s, d in zip(src, dst):
        adj[int(s)].append(int(d))
    out = set()
    for x in range(n):
        seen, frontier = set(), list(adj[x])
        while frontier:
            y = frontier.pop()
            if y in seen:
                continue
            seen.add(y)
            frontier.extend(adj[y])
        out.update((x, y) for y in seen)
    return out


def best_simple_paths_f32(n, src, dst, w, maximize):
    """Brute force: best left-folded fp32 sum over every walk that repeats no edge endpoint
    except possibly returning to its start (enough when cycles never improve)."""
    edges = {}
    for s, d, ww in zip(src, dst, w):
        edges[(int(s), int(d))] = np.float32(ww)
    best = {}

    def consider(x, y, t):
        k = (x, y)
        if k not in best or (t > best[k] if maximize else t < best[k]):
            best[k] = t

    def walk(x, cur, t, visited):
        for (a, b), ww in edges.items():
            if a != cur:
                continue
            nt = np.float32(t + ww) if t is not None else ww
            if b == x:
                consider(x, b, nt)
            elif b not in visited:
                consider(x, b, nt)
                walk(x, b, nt, visited | {b})

    for x in range(n):
        walk(x, x, None, {x})
    return best
