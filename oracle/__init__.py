"""ctypes front end of the CPU oracle (``xlog_oracle.cpp``).  TEST INFRASTRUCTURE ONLY.

The oracle is the plain definition the CUDA path is checked against; the product
never imports this package.  ``build()`` compiles the C++ file with g++ into
``liboracle.so`` beside it.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Dict, List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "xlog_oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle.so")

MAXV, MAXA = 8, 4
SEMIRING = {"maxplus": 0, "minplus": 1, "logsumexp": 2, "sumprod": 3}
STATUS = {0: "OK", 1: "INVALID", 3: "UNSUPPORTED", 5: "CAPACITY_EXCEEDED", 6: "CONVERGENCE_FAILURE"}


class OracleError(RuntimeError):
    def __init__(self, code):
        super().__init__(STATUS.get(code, str(code)))
        self.code = code
        self.status = STATUS.get(code, str(code))


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-ffp-contract=off",
                               "-o", _LIB, _SRC])
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.orc_create.restype = C.c_void_p
        L.orc_destroy.argtypes = [C.c_void_p]
        L.orc_relation.argtypes = [C.c_void_p, C.c_int, C.c_int]
        L.orc_load.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int64]
        L.orc_rule.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p]
        L.orc_reset.argtypes = [C.c_void_p]
        L.orc_run.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_void_p]
        L.orc_delta_trace.argtypes = [C.c_void_p, C.c_void_p, C.c_int64]
        L.orc_delta_trace.restype = C.c_int64
        L.orc_size.argtypes = [C.c_void_p, C.c_int]
        L.orc_size.restype = C.c_int64
        L.orc_read.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
        L.orc_backward.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
        _lib = L
    return _lib


class Oracle:
    """One tagged-Datalog program evaluated on the CPU."""

    def __init__(self):
        self._L = _load()
        self._h = C.c_void_p(self._L.orc_create())
        self._arity: List[int] = []
        self._rule_atoms: List[List[int]] = []

    def __del__(self):
        if getattr(self, "_h", None):
            self._L.orc_destroy(self._h)
            self._h = None

    def relation(self, arity: int, semiring: str) -> int:
        r = self._L.orc_relation(self._h, arity, SEMIRING[semiring])
        if r < 0:
            raise ValueError("bad relation")
        self._arity.append(arity)
        return r

    def load(self, rel: int, cols: Sequence[np.ndarray], tags: Optional[np.ndarray]):
        k = self._arity[rel]
        assert len(cols) == k
        n = len(cols[0])
        rows = np.ascontiguousarray(np.stack([np.asarray(c, np.int32) for c in cols], axis=1)) if n else np.zeros((0, k), np.int32)
        t = None if tags is None else np.ascontiguousarray(tags, np.float32)
        st = self._L.orc_load(self._h, rel, rows.ctypes.data, None if t is None else t.ctypes.data, n)
        if st:
            raise OracleError(st)

    def rule(self, head: int, head_exprs, atoms, emit_count: bool = False, negated=()) -> int:
        """head_exprs: [(c0, {var: coef})]; atoms: [(rel, [("c", value) | ("v", var, mul, add)])];
        negated: indices of atoms under negation as failure."""
        he = np.zeros((len(head_exprs), 1 + MAXV), np.int64)
        for i, (c0, coef) in enumerate(head_exprs):
            he[i, 0] = c0
            for v, k in dict(coef).items():
                he[i, 1 + v] = k
        rel_ids = np.asarray([a[0] for a in atoms], np.int32)
        args = np.zeros((len(atoms), MAXA, 4), np.int64)
        for j, (_, al) in enumerate(atoms):
            for c, a in enumerate(al):
                if a[0] == "c":
                    args[j, c] = (0, 0, 1, a[1])
                else:
                    args[j, c] = (1, a[1], a[2], a[3])
        neg = np.zeros(len(atoms), np.int32)
        for j in negated:
            neg[j] = 1
        r = self._L.orc_rule(self._h, head, len(head_exprs), he.ctypes.data, len(atoms),
                             rel_ids.ctypes.data, args.ctypes.data, int(emit_count), neg.ctypes.data)
        if r < 0:
            raise ValueError("bad rule")
        self._rule_atoms.append([int(x) for x in rel_ids])
        return r

    def reset(self):
        self._L.orc_reset(self._h)

    def run(self, mode: str = "naive", max_iterations: int = 1 << 20) -> Dict[str, int]:
        stats = np.zeros(4, np.int64)
        st = self._L.orc_run(self._h, {"naive": 0, "seminaive": 1}[mode], max_iterations, stats.ctypes.data)
        if st:
            raise OracleError(st)
        return dict(iterations=int(stats[0]), contributions=int(stats[1]), delta_total=int(stats[2]),
                    derived_tuples=int(stats[3]))

    def delta_trace(self) -> List[int]:
        buf = np.zeros(1 << 16, np.int64)
        n = self._L.orc_delta_trace(self._h, buf.ctypes.data, buf.size)
        return [int(x) for x in buf[:n]]

    def size(self, rel: int) -> int:
        return int(self._L.orc_size(self._h, rel))

    def read(self, rel: int):
        n, k = self.size(rel), self._arity[rel]
        rows = np.zeros((n, k), np.int32)
        tags = np.zeros(n, np.float32)
        self._L.orc_read(self._h, rel, rows.ctypes.data, tags.ctypes.data)
        return [np.ascontiguousarray(rows[:, c]) for c in range(k)], tags

    def backward(self, rule: int, g: np.ndarray) -> List[np.ndarray]:
        g = np.ascontiguousarray(g, np.float32)
        outs = [np.zeros(self.size(r), np.float32) for r in self._rule_atoms[rule]]
        ptrs = (C.c_void_p * len(outs))(*[o.ctypes.data for o in outs])
        st = self._L.orc_backward(self._h, rule, g.ctypes.data, ptrs)
        if st:
            raise OracleError(st)
        return outs


def load_program(program) -> "tuple[Oracle, Dict[str, int], List[int]]":
    """Instantiate a ``workloads.Program`` (plain data) on a fresh oracle."""
    o = Oracle()
    ids = {name: o.relation(ar, sr) for name, (ar, sr) in program.relations.items()}
    for name, (cols, tags) in program.facts.items():
        o.load(ids[name], cols, tags)
    rule_ids = []
    for r in program.rules:
        he = [(e.c0, dict(e.coef)) for e in r.head_exprs]
        atoms = []
        for a in r.atoms:
            al = []
            for g in a.args:
                if hasattr(g, "value"):
                    al.append(("c", g.value))
                else:
                    al.append(("v", g.var, g.mul, g.add))
            atoms.append((ids[a.rel], al))
        rule_ids.append(o.rule(ids[r.head], he, atoms, r.emit_count, [j for j, a in enumerate(r.atoms) if a.negated]))
    return o, ids, rule_ids
