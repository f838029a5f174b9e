"""Seeded synthetic inputs for the five workloads.

This module only *generates inputs* (graphs, weights, logits, source sets); it
holds none of the fixpoint method's arithmetic and imports neither the CUDA
library nor the CPU oracle, so both sides can be fed the very same arrays.

Random numbers come from a counter-based generator: the i-th draw of a stream is
``mix64(seed + GOLDEN * (stream * 2**40 + i + 1))`` with the splitmix64 finaliser,
so any element can be produced independently and results do not depend on
chunking.  Uniforms use the top 53 bits; normals use Box-Muller in float64.
"""
from __future__ import annotations

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)

SEED_BASE = 0x5EED0000


def _mix64(z: np.ndarray) -> np.ndarray:
    z = z.copy()
    z ^= z >> np.uint64(30)
    z *= _M1
    z ^= z >> np.uint64(27)
    z *= _M2
    z ^= z >> np.uint64(31)
    return z


def rand_u64(seed: int, stream: int, start: int, n: int) -> np.ndarray:
    """Draws ``start .. start+n-1`` of (seed, stream) as uint64."""
    with np.errstate(over="ignore"):
        ctr = np.arange(start + 1, start + n + 1, dtype=np.uint64)
        ctr += np.uint64((stream << 40) & 0xFFFFFFFFFFFFFFFF)
        z = ctr * _GOLDEN + np.uint64(seed & 0xFFFFFFFFFFFFFFFF)
        return _mix64(z)


def uniform01(seed: int, stream: int, start: int, n: int) -> np.ndarray:
    """float64 uniforms in [0, 1)."""
    return (rand_u64(seed, stream, start, n) >> np.uint64(11)).astype(np.float64) * (1.0 / (1 << 53))


def normal(seed: int, stream: int, n: int) -> np.ndarray:
    """float64 standard normals (Box-Muller on draws 2i, 2i+1 of the stream)."""
    u = uniform01(seed, stream, 0, 2 * n)
    u1 = 1.0 - u[0::2]          # (0, 1]
    u2 = u[1::2]
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


def randint(seed: int, stream: int, start: int, n: int, hi: int) -> np.ndarray:
    """int64 in [0, hi) (floor of uniform * hi; hi < 2**31 so the bias is < 2**-22)."""
    return np.minimum((uniform01(seed, stream, start, n) * hi).astype(np.int64), hi - 1)


# ----------------------------------------------------------------------------
# graphs
# ----------------------------------------------------------------------------

def uniform_digraph(n_nodes: int, n_edges: int, seed: int):
    """Exactly ``n_edges`` distinct directed non-loop edges with uniform endpoints.

    Draw i gives (src, dst); loops and repeats of an earlier pair are skipped and
    drawing continues until enough edges exist.  Returned in draw order.
    """
    assert n_edges <= n_nodes * (n_nodes - 1)
    src_l, dst_l = [], []
    seen = set()
    pos = 0
    while len(src_l) < n_edges:
        m = max(1024, 2 * (n_edges - len(src_l)))
        s = randint(seed, 1, pos, m, n_nodes)
        d = randint(seed, 2, pos, m, n_nodes)
        pos += m
        for a, b in zip(s.tolist(), d.tolist()):
            if a == b or (a, b) in seen:
                continue
            seen.add((a, b))
            src_l.append(a)
            dst_l.append(b)
            if len(src_l) == n_edges:
                break
    return np.asarray(src_l, dtype=np.int32), np.asarray(dst_l, dtype=np.int32)


def rmat_raw(scale: int, n_raw: int, seed: int, a=0.57, b=0.19, c=0.19, d=0.05):
    """Raw R-MAT edge list: ``scale`` quadrant draws per edge, most significant
    bit first, no vertex permutation, no parameter noise.  Quadrant a = (0,0),
    b = (0,1), c = (1,0), d = (1,1) as (src bit, dst bit)."""
    assert abs(a + b + c + d - 1.0) < 1e-12
    src = np.zeros(n_raw, dtype=np.int64)
    dst = np.zeros(n_raw, dtype=np.int64)
    chunk = 1 << 22
    for lo in range(0, n_raw, chunk):
        m = min(chunk, n_raw - lo)
        s = np.zeros(m, dtype=np.int64)
        t = np.zeros(m, dtype=np.int64)
        for lvl in range(scale):
            r = uniform01(seed, 16 + lvl, lo, m)
            sb = r >= a + b
            db = ((r >= a) & (r < a + b)) | (r >= a + b + c)
            s = (s << 1) | sb
            t = (t << 1) | db
        src[lo:lo + m] = s
        dst[lo:lo + m] = t
    return src, dst


def canonical_edges(src: np.ndarray, dst: np.ndarray, w: np.ndarray):
    """Drop self-loops; of a repeated (src, dst) pair keep the first occurrence and
    its weight.  Result sorted by (src, dst)."""
    keep = src != dst
    s = src[keep].astype(np.uint64)
    t = dst[keep].astype(np.uint64)
    ww = w[keep]
    key = (s << np.uint64(32)) | t
    _, first = np.unique(key, return_index=True)      # index of first occurrence, keys ascending
    return (s[first].astype(np.int32), t[first].astype(np.int32), ww[first])


def rmat_graph(scale: int, edge_factor: int, seed: int, weights: str):
    """Canonical R-MAT graph with per-raw-edge weights.

    weights = "u1_10": float32 uniform in [1, 10];  "n01": float32 N(0, 1).
    """
    n_raw = edge_factor << scale
    src, dst = rmat_raw(scale, n_raw, seed)
    if weights == "u1_10":
        w = (1.0 + 9.0 * uniform01(seed, 3, 0, n_raw)).astype(np.float32)
    elif weights == "n01":
        w = normal(seed, 3, n_raw).astype(np.float32)
    else:
        raise ValueError(weights)
    return canonical_edges(src, dst, w)


def distinct_sources(n_nodes: int, k: int, seed: int) -> np.ndarray:
    """k distinct node ids, uniform over all ids, in draw order."""
    out, seen, pos = [], set(), 0
    while len(out) < k:
        for v in randint(seed, 4, pos, 2 * k, n_nodes).tolist():
            if v not in seen:
                seen.add(v)
                out.append(v)
                if len(out) == k:
                    break
        pos += 2 * k
    return np.asarray(out, dtype=np.int32)


def log_prob_tags(n: int, seed: int, lo=0.5, hi=0.99) -> np.ndarray:
    """float32 tags uniform (in log space) on [ln lo, ln hi]."""
    a, b = np.log(lo), np.log(hi)
    return (a + (b - a) * uniform01(seed, 3, 0, n)).astype(np.float32)


def digit_log_tags(n_images: int, seed: int) -> np.ndarray:
    """[n_images, 10] float32 log-softmax of N(0,1) logits (softmax done in float64)."""
    z = normal(seed, 5, n_images * 10).reshape(n_images, 10)
    m = z.max(axis=1, keepdims=True)
    lse = m + np.log(np.exp(z - m).sum(axis=1, keepdims=True))
    return (z - lse).astype(np.float32)


def head_gradient(n_rows: int, seed: int) -> np.ndarray:
    """float32 N(0,1) upstream gradient, one per head row."""
    return normal(seed, 6, n_rows).astype(np.float32)
