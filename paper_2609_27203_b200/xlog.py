"""Thin ctypes binding over ``libxlog.so`` (the C ABI declared in ``include/xlog.h``).

Argument marshalling only: every step of the fixpoint runs in the CUDA library.  PyTorch
supplies device memory (the arena and any device-resident inputs) and the stream.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libxlog.so")

MAX_ARITY, MAX_ATOMS, MAX_VARS = 4, 4, 8
SEMIRING = {"maxplus": 0, "minplus": 1, "logsumexp": 2, "sumprod": 3}
STATUS = ["OK", "INVALID_ARGUMENT", "INVALID_VALUE", "UNSUPPORTED", "RESOURCE_EXHAUSTED", "CAPACITY_EXCEEDED",
          "CONVERGENCE_FAILURE", "BUFFER_TOO_SMALL", "INVALID_STATE", "CUDA", "INTERNAL"]
MEM_HOST, MEM_DEVICE = 0, 1
FLAG_CHECK_INVARIANTS = 1
FLAG_PROFILE = 2
FLAG_NO_TAG_MIRROR = 4
FLAG_NO_RESIDENT_LOOP = 8
FLAG_NO_GRAPH = 16
FLAG_FORCE_WCOJ = 32
FLAG_FORCE_CHAIN = 64
FLAG_NO_GROUPED_JOIN = 128
FLAG_NO_BITMAP_JOIN = 256
FLAG_NO_DENSE_DOUBLING = 512
FLAG_NO_TRIANGLE_BITMAP = 1024
FLAG_NO_ROW_FIXPOINT = 2048
PLAN_NONE, PLAN_WCOJ, PLAN_CHAIN = 0, 1, 2

EXPORTS = ["xlog_ctx_create", "xlog_ctx_destroy", "xlog_last_error", "xlog_relation_create", "xlog_relation_load",
           "xlog_relation_size", "xlog_relation_read", "xlog_relation_view", "xlog_rule_add", "xlog_fixpoint",
           "xlog_ctx_reset_idb", "xlog_rule_backward", "xlog_profile_read", "xlog_profile_reset",
           "xlog_reduce_by_key_static", "xlog_sort_pairs", "xlog_debug_set_poll_limit", "xlog_debug_sort_pass_without_first_tile", "xlog_device_copy", "xlog_device_read", "xlog_device_gather"]


class XlogError(RuntimeError):
    def __init__(self, code: int, msg: str):
        self.code = code
        self.status = STATUS[code] if 0 <= code < len(STATUS) else str(code)
        super().__init__(f"{self.status}: {msg}")


class Config(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("device", C.c_int32), ("stream", C.c_void_p), ("arena", C.c_void_p),
                ("arena_bytes", C.c_uint64), ("max_iterations", C.c_int64), ("candidate_chunk_bytes", C.c_uint64),
                ("flags", C.c_uint32)]


class Arg(C.Structure):
    _fields_ = [("kind", C.c_int32), ("var", C.c_int32), ("mul", C.c_int32), ("add", C.c_int32)]


class AtomS(C.Structure):
    _fields_ = [("rel", C.c_int32), ("args", Arg * MAX_ARITY), ("negated", C.c_int32)]


class Expr(C.Structure):
    _fields_ = [("c0", C.c_int64), ("coef", C.c_int32 * MAX_VARS)]


class Plan(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("head_rel", C.c_int32), ("n_head_cols", C.c_int32),
                ("head", Expr * MAX_ARITY), ("n_atoms", C.c_int32), ("atoms", AtomS * MAX_ATOMS),
                ("emit_count_column", C.c_int32)]


class Receipt(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("status", C.c_int32), ("strata", C.c_int64), ("iterations", C.c_int64),
                ("derived_tuples", C.c_int64), ("candidates", C.c_int64), ("unique_candidates", C.c_int64),
                ("new_tuples", C.c_int64), ("improved_tags", C.c_int64), ("h2d_bytes", C.c_int64),
                ("d2h_bytes", C.c_int64), ("kernel_launches", C.c_int64), ("peak_arena_bytes", C.c_int64),
                ("device_ms", C.c_double), ("triangle_plan", C.c_int32), ("index_builds", C.c_int32)]

    def as_dict(self) -> Dict[str, object]:
        return {k: getattr(self, k) for k, _ in self._fields_ if k != "struct_size"}


class KernelStat(C.Structure):
    _fields_ = [("name", C.c_char * 48), ("launches", C.c_int64), ("device_ms", C.c_double),
                ("algorithmic_bytes", C.c_int64)]


_lib = None


def lib():
    """Load the CUDA library; its absence is an error (there is no fallback path)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} is missing: build it with `python -m paper_2609_27203_b200.build`")
        L = C.CDLL(_LIB_PATH)
        vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
        L.xlog_ctx_create.argtypes = [C.POINTER(Config), C.POINTER(vp)]
        L.xlog_ctx_destroy.argtypes = [vp]
        L.xlog_last_error.argtypes = [vp]
        L.xlog_last_error.restype = C.c_char_p
        L.xlog_relation_create.argtypes = [vp, i32, i32, C.c_char_p, C.POINTER(i32)]
        L.xlog_relation_load.argtypes = [vp, i32, C.POINTER(vp), vp, i64, i32]
        L.xlog_relation_size.argtypes = [vp, i32, C.POINTER(i64)]
        L.xlog_relation_read.argtypes = [vp, i32, C.POINTER(vp), vp, i64, C.POINTER(i64), i32]
        L.xlog_relation_view.argtypes = [vp, i32, C.POINTER(vp), C.POINTER(vp), C.POINTER(i64)]
        L.xlog_rule_add.argtypes = [vp, C.POINTER(Plan), C.POINTER(i32)]
        L.xlog_fixpoint.argtypes = [vp, C.POINTER(Receipt)]
        L.xlog_ctx_reset_idb.argtypes = [vp]
        L.xlog_rule_backward.argtypes = [vp, i32, vp, C.POINTER(vp)]
        L.xlog_profile_read.argtypes = [vp, C.POINTER(KernelStat), i32, C.POINTER(i32)]
        L.xlog_profile_reset.argtypes = [vp]
        L.xlog_sort_pairs.argtypes = [vp, vp, vp, i64, i32, i32]
        L.xlog_device_copy.argtypes = [vp, vp, vp, C.c_uint64, i32]
        L.xlog_device_read.argtypes = [vp, vp, C.c_uint64, i32, vp]
        L.xlog_device_gather.argtypes = [vp, vp, C.c_uint64, C.c_uint64, vp]
        L.xlog_debug_set_poll_limit.argtypes = [vp, C.c_uint32]
        L.xlog_debug_sort_pass_without_first_tile.argtypes = [vp, vp, vp, vp, vp, i64, i32]
        L.xlog_reduce_by_key_static.argtypes = [vp, i32, vp, vp, i64, vp, vp, C.POINTER(i64), C.c_char_p, C.c_size_t]
        for name in EXPORTS:
            if name != "xlog_last_error":
                getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


class Context:
    """One engine context over a caller-owned device arena (a torch uint8 CUDA tensor)."""

    def __init__(self, arena_bytes: int = 1 << 30, device: int = 0, max_iterations: int = 0,
                 candidate_chunk_bytes: int = 0, flags: int = 0, stream=None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("paper_2609_27203_b200 needs a CUDA device; there is no CPU path")
        self._L = lib()
        self._torch = torch
        self.device = device
        torch.cuda.set_device(device)
        self._arena = torch.empty(arena_bytes, dtype=torch.uint8, device=f"cuda:{device}")
        self._stream = stream if stream is not None else torch.cuda.current_stream(device)
        cfg = Config(C.sizeof(Config), device, self._stream.cuda_stream, self._arena.data_ptr(), arena_bytes,
                     max_iterations, candidate_chunk_bytes, flags)
        h = C.c_void_p()
        st = self._L.xlog_ctx_create(C.byref(cfg), C.byref(h))
        if st:
            raise XlogError(st, "xlog_ctx_create failed")
        self._h = h
        self._arity: List[int] = []
        self._rule_atoms: List[List[int]] = []

    def close(self):
        if getattr(self, "_h", None):
            self._L.xlog_ctx_destroy(self._h)
            self._h = None
            self._arena = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st: int):
        if st:
            raise XlogError(st, (self._L.xlog_last_error(self._h) or b"").decode())

    # ---- relations ----
    def relation(self, arity: int, semiring: str, name: str = "") -> int:
        out = C.c_int32()
        self._check(self._L.xlog_relation_create(self._h, arity, SEMIRING[semiring], name.encode(), C.byref(out)))
        self._arity.append(arity)
        return out.value

    def load(self, rel: int, cols: Sequence, tags=None):
        """cols/tags: numpy arrays (host) or torch CUDA tensors (device), int32 / float32, all of one length."""
        torch = self._torch
        k = self._arity[rel]
        if len(cols) != k:
            raise ValueError(f"relation of arity {k} loaded with {len(cols)} columns")
        on_device = isinstance(cols[0], torch.Tensor)
        n = check_load_shapes(cols, tags, self.device if on_device else None)
        keep = []
        ptrs = (C.c_void_p * k)()
        if on_device:
            for i, c in enumerate(cols):
                c = c.to(torch.int32).contiguous()
                keep.append(c)
                ptrs[i] = c.data_ptr()
            tp = None
            if tags is not None:
                t = tags.to(torch.float32).contiguous()
                keep.append(t)
                tp = t.data_ptr()
            # the conversions above ran on torch's current stream: the library's stream must see their results
            if keep and torch.cuda.current_stream(self.device).cuda_stream != self._stream.cuda_stream:
                self._stream.wait_stream(torch.cuda.current_stream(self.device))
        else:
            for i, c in enumerate(cols):
                c = np.ascontiguousarray(c, np.int32)
                keep.append(c)
                ptrs[i] = c.ctypes.data
            tp = None
            if tags is not None:
                t = np.ascontiguousarray(tags, np.float32)
                keep.append(t)
                tp = t.ctypes.data
        self._check(self._L.xlog_relation_load(self._h, rel, ptrs, tp, n, MEM_DEVICE if on_device else MEM_HOST))

    def size(self, rel: int) -> int:
        n = C.c_int64()
        self._check(self._L.xlog_relation_size(self._h, rel, C.byref(n)))
        return n.value

    def read(self, rel: int):
        """Host copy: ([col arrays], tags) in ascending lexicographic order."""
        n, k = self.size(rel), self._arity[rel]
        # page-locked destinations (torch's caching host allocator hands freed blocks out again), so that the copy runs
        # at PCIe speed instead of through the driver's staging buffer
        torch = self._torch
        cols = [torch.empty(n, dtype=torch.int32, pin_memory=True).numpy() for _ in range(k)]
        tags = torch.empty(n, dtype=torch.float32, pin_memory=True).numpy()
        ptrs = (C.c_void_p * k)(*[c.ctypes.data for c in cols])
        got = C.c_int64()
        self._check(self._L.xlog_relation_read(self._h, rel, ptrs, tags.ctypes.data, n, C.byref(got), MEM_HOST))
        assert got.value == n
        return cols, tags

    def read_device(self, rel: int):
        torch = self._torch
        n, k = self.size(rel), self._arity[rel]
        cols = [torch.empty(n, dtype=torch.int32, device=f"cuda:{self.device}") for _ in range(k)]
        tags = torch.empty(n, dtype=torch.float32, device=f"cuda:{self.device}")
        ptrs = (C.c_void_p * k)(*[c.data_ptr() for c in cols])
        got = C.c_int64()
        self._check(self._L.xlog_relation_read(self._h, rel, ptrs, tags.data_ptr(), n, C.byref(got), MEM_DEVICE))
        return cols, tags

    def view(self, rel: int):
        """Borrowed device pointers (ints) to the stored columns and tags, and the row count."""
        k = self._arity[rel]
        ptrs = (C.c_void_p * k)()
        tp = C.c_void_p()
        n = C.c_int64()
        self._check(self._L.xlog_relation_view(self._h, rel, ptrs, C.byref(tp), C.byref(n)))
        return [int(p or 0) for p in ptrs], int(tp.value or 0), n.value

    # ---- rules ----
    def rule(self, head: int, head_exprs, atoms, emit_count: bool = False, negated=()) -> int:
        """head_exprs: [(c0, {var: coef})]; atoms: [(rel, [("c", value) | ("v", var, mul, add)])];
        negated: indices of atoms under negation as failure."""
        p = Plan()
        p.struct_size = C.sizeof(Plan)
        p.head_rel = head
        p.n_head_cols = len(head_exprs)
        for i, (c0, coef) in enumerate(head_exprs):
            p.head[i].c0 = c0
            for v, kf in dict(coef).items():
                p.head[i].coef[v] = kf
        p.n_atoms = len(atoms)
        for j, (rel, al) in enumerate(atoms):
            p.atoms[j].rel = rel
            for c, a in enumerate(al):
                if a[0] == "c":
                    p.atoms[j].args[c] = Arg(0, 0, 1, a[1])
                else:
                    p.atoms[j].args[c] = Arg(1, a[1], a[2], a[3])
        for j in negated:
            p.atoms[j].negated = 1
        p.emit_count_column = int(emit_count)
        out = C.c_int32()
        self._check(self._L.xlog_rule_add(self._h, C.byref(p), C.byref(out)))
        self._rule_atoms.append([rel for rel, _ in atoms])
        return out.value

    # ---- evaluation ----
    def fixpoint(self) -> Dict[str, object]:
        r = Receipt()
        r.struct_size = C.sizeof(Receipt)
        st = self._L.xlog_fixpoint(self._h, C.byref(r))
        self.last_receipt = r.as_dict()
        self._check(st)
        return self.last_receipt

    def profile(self) -> Dict[str, Dict[str, float]]:
        """Per-kernel launches / device ms / algorithmic bytes (needs FLAG_PROFILE)."""
        n = C.c_int32()
        self._check(self._L.xlog_profile_read(self._h, None, 0, C.byref(n)))
        buf = (KernelStat * max(n.value, 1))()
        self._check(self._L.xlog_profile_read(self._h, buf, n.value, C.byref(n)))
        return {buf[i].name.decode(): dict(launches=buf[i].launches, ms=buf[i].device_ms, bytes=buf[i].algorithmic_bytes)
                for i in range(n.value)}

    def profile_reset(self):
        self._check(self._L.xlog_profile_reset(self._h))

    def sort_pairs(self, keys, payload, key_bits: int):
        """In-place stable sort of torch CUDA tensors: keys int32/int64 (non-negative), payload 4-byte."""
        assert keys.is_contiguous() and payload.is_contiguous() and payload.element_size() == 4
        self._check(self._L.xlog_sort_pairs(self._h, keys.data_ptr(), payload.data_ptr(), keys.numel(),
                                            keys.element_size(), key_bits))

    def debug_set_poll_limit(self, polls: int):
        """Test hook: how many polls a look-back wait makes before it gives up (default 2^22)."""
        self._check(self._L.xlog_debug_set_poll_limit(self._h, polls))

    def debug_sort_pass_without_first_tile(self, keys, payload, out_keys, out_payload):
        """Test hook: one sort pass whose first tile never runs; raises XlogError(INTERNAL) once the waits give up."""
        self._check(self._L.xlog_debug_sort_pass_without_first_tile(self._h, keys.data_ptr(), payload.data_ptr(), out_keys.data_ptr(),
                                                                    out_payload.data_ptr(), keys.numel(), keys.element_size()))

    def reset_idb(self):
        self._check(self._L.xlog_ctx_reset_idb(self._h))

    def backward(self, rule: int, grad_head, same_buffer_for_same_relation: bool = True):
        """grad_head: torch CUDA float32 tensor over head rows.  Returns one torch tensor per atom
        (atoms naming the same relation share one tensor, which then holds the sum)."""
        torch = self._torch
        g = grad_head.to(torch.float32).contiguous()
        rels = self._rule_atoms[rule]
        bufs: Dict[int, object] = {}
        outs = []
        for j, r in enumerate(rels):
            key = r if same_buffer_for_same_relation else (r, j)
            if key not in bufs:
                bufs[key] = torch.empty(self.size(r), dtype=torch.float32, device=f"cuda:{self.device}")
            outs.append(bufs[key])
        ptrs = (C.c_void_p * len(outs))(*[o.data_ptr() for o in outs])
        self._check(self._L.xlog_rule_backward(self._h, rule, g.data_ptr(), ptrs))
        return outs


STATIC_REDUCE_MAX_ROWS = 1 << 24


def copy_bandwidth_gbs(n_bytes: int, repeats: int = 50, device: int = 0) -> float:
    """GB/s (bytes read + bytes written) of the library's own copy kernel on a pair of n_bytes buffers: with a pair that
    fits L2 this is the L2 bandwidth, with a large pair the HBM bandwidth.  CUDA events on torch's current stream."""
    import torch
    with torch.cuda.device(device):
        a = torch.empty(n_bytes, dtype=torch.uint8, device=f"cuda:{device}").fill_(1)
        b = torch.empty_like(a)
        s = torch.cuda.current_stream(device)
        L = lib()
        if L.xlog_device_copy(s.cuda_stream, b.data_ptr(), a.data_ptr(), n_bytes, 5):
            raise XlogError(9, "xlog_device_copy failed")
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(s)
        if L.xlog_device_copy(s.cuda_stream, b.data_ptr(), a.data_ptr(), n_bytes, repeats):
            raise XlogError(9, "xlog_device_copy failed")
        e1.record(s)
        e1.synchronize()
        return 2.0 * n_bytes * repeats / (e0.elapsed_time(e1) * 1e-3) / 1e9


def read_bandwidth_gbs(n_bytes: int, repeats: int = 50, device: int = 0) -> float:
    """GB/s (bytes read) of the library's own read-only kernel on a buffer of n_bytes: the L2 read rate when it fits L2."""
    import torch
    with torch.cuda.device(device):
        a = torch.empty(n_bytes, dtype=torch.uint8, device=f"cuda:{device}").fill_(1)
        sink = torch.zeros(1, dtype=torch.int32, device=f"cuda:{device}")
        s = torch.cuda.current_stream(device)
        L = lib()
        if L.xlog_device_read(s.cuda_stream, a.data_ptr(), n_bytes, 5, sink.data_ptr()):
            raise XlogError(9, "xlog_device_read failed")
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(s)
        if L.xlog_device_read(s.cuda_stream, a.data_ptr(), n_bytes, repeats, sink.data_ptr()):
            raise XlogError(9, "xlog_device_read failed")
        e1.record(s)
        e1.synchronize()
        return 1.0 * n_bytes * repeats / (e0.elapsed_time(e1) * 1e-3) / 1e9


def gather_rate(n_bytes: int, reads: int = 1 << 28, device: int = 0) -> float:
    """Random 4-byte reads per second from a table of n_bytes with the library's own gather kernel (each read touches one
    32-byte sector): with a table that fits L2, the rate a kernel that reads one table slot per unit of work can reach."""
    import torch
    with torch.cuda.device(device):
        a = torch.empty(n_bytes, dtype=torch.uint8, device=f"cuda:{device}").fill_(1)
        sink = torch.zeros(1, dtype=torch.int32, device=f"cuda:{device}")
        s = torch.cuda.current_stream(device)
        L = lib()
        threads = 148 * 8 * 256
        done = ((reads + threads - 1) // threads + 7) // 8 * 8 * threads
        if L.xlog_device_gather(s.cuda_stream, a.data_ptr(), n_bytes, reads // 8, sink.data_ptr()):
            raise XlogError(9, "xlog_device_gather failed")
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(s)
        if L.xlog_device_gather(s.cuda_stream, a.data_ptr(), n_bytes, reads, sink.data_ptr()):
            raise XlogError(9, "xlog_device_gather failed")
        e1.record(s)
        e1.synchronize()
        return done / (e0.elapsed_time(e1) * 1e-3)


def check_load_shapes(cols, tags, device) -> int:
    """Every column and the tags must have one length (and, for device inputs, live on `device`).  Returns that length."""
    def length(x):
        return int(x.numel()) if hasattr(x, "numel") else len(x)
    n = length(cols[0])
    for i, c in enumerate(cols):
        if length(c) != n:
            raise ValueError(f"column {i} has {length(c)} rows, column 0 has {n}")
        if getattr(c, "ndim", 1) != 1:
            raise ValueError(f"column {i} is not one-dimensional")
        if device is not None and (not getattr(c, "is_cuda", False) or c.device.index != device):
            raise ValueError(f"column {i} does not live on cuda:{device}")
    if tags is not None:
        if length(tags) != n:
            raise ValueError(f"tags have {length(tags)} rows, the columns have {n}")
        if device is not None and (not getattr(tags, "is_cuda", False) or tags.device.index != device):
            raise ValueError(f"tags do not live on cuda:{device}")
    return n


def check_static_reduce_args(keys, tags, out_keys, out_tags) -> None:
    """Everything the C entry point takes on trust: dtypes, contiguity, one device, lengths, room in the outputs and
    outputs that do not overlap the inputs.  Raises ValueError before anything is launched."""
    import torch
    named = {"keys": (keys, torch.int32), "tags": (tags, torch.float32), "out_keys": (out_keys, torch.int32), "out_tags": (out_tags, torch.float32)}
    for name, (t, dt) in named.items():
        if not isinstance(t, torch.Tensor):
            raise ValueError(f"{name} must be a torch tensor")
        if t.dtype != dt:
            raise ValueError(f"{name} must be {dt}, not {t.dtype}")
        if not t.is_cuda:
            raise ValueError(f"{name} must be a CUDA tensor")
        if not t.is_contiguous():
            raise ValueError(f"{name} must be contiguous")
        if t.device != keys.device:
            raise ValueError(f"{name} lives on {t.device}, keys on {keys.device}")
    n = keys.numel()
    if tags.numel() != n:
        raise ValueError(f"tags have {tags.numel()} rows, keys have {n}")
    if out_keys.numel() < n or out_tags.numel() < n:
        raise ValueError(f"the outputs need room for {n} rows")

    def span(t):
        return t.data_ptr(), t.data_ptr() + t.numel() * t.element_size()
    if n:
        for o in (out_keys, out_tags):
            for i in (keys, tags):
                (a0, a1), (b0, b1) = span(o), span(i)
                if a0 < b1 and b0 < a1:
                    raise ValueError("an output overlaps an input")
        (a0, a1), (b0, b1) = span(out_keys), span(out_tags)
        if a0 < b1 and b0 < a1:
            raise ValueError("the two outputs overlap")


def reduce_by_key_static(semiring: str, keys, tags, out_keys, out_tags, stream=None) -> int:
    """Reduce-by-key for callers that must not allocate device memory during the call (no context,
    no arena: the library's own fixed scratch array is used).  keys (int32, ascending) / tags
    (float32) and the two output tensors are torch CUDA tensors the caller already owns, all on one
    device; the outputs have room for as many rows as the input and overlap nothing.  Returns the
    number of groups written.  At most STATIC_REDUCE_MAX_ROWS rows."""
    import torch
    check_static_reduce_args(keys, tags, out_keys, out_tags)
    n_out = C.c_int64()
    err = C.create_string_buffer(256)
    # the C side resolves its scratch array and the stream on the CURRENT device: make that the tensors' device
    with torch.cuda.device(keys.device):
        s = stream if stream is not None else torch.cuda.current_stream(keys.device)
        st = lib().xlog_reduce_by_key_static(s.cuda_stream, SEMIRING[semiring], keys.data_ptr(), tags.data_ptr(), keys.numel(),
                                             out_keys.data_ptr(), out_tags.data_ptr(), C.byref(n_out), err, len(err))
    if st:
        raise XlogError(st, err.value.decode())
    return n_out.value


def load_program(program, ctx: Optional[Context] = None, device_inputs: bool = False, **ctx_kw):
    """Instantiate a ``workloads.Program`` on a context.  Returns (ctx, relation ids, rule ids)."""
    if ctx is None:
        ctx = Context(**ctx_kw)
    ids = {name: ctx.relation(ar, sr, name) for name, (ar, sr) in program.relations.items()}
    for name, (cols, tags) in program.facts.items():
        if device_inputs:
            import torch
            dev = f"cuda:{ctx.device}"
            cols = [torch.from_numpy(np.ascontiguousarray(c, np.int32)).to(dev) for c in cols]
            tags = None if tags is None else torch.from_numpy(np.ascontiguousarray(tags, np.float32)).to(dev)
        ctx.load(ids[name], cols, tags)
    rule_ids = []
    for r in program.rules:
        he = [(e.c0, dict(e.coef)) for e in r.head_exprs]
        atoms = []
        for a in r.atoms:
            al = []
            for g in a.args:
                al.append(("c", g.value) if hasattr(g, "value") else ("v", g.var, g.mul, g.add))
            atoms.append((ids[a.rel], al))
        rule_ids.append(ctx.rule(ids[r.head], he, atoms, r.emit_count, [j for j, a in enumerate(r.atoms) if a.negated]))
    return ctx, ids, rule_ids
