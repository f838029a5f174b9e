"""The allocation-free reduce-by-key entry point against the engine's ordinary path.

Some users of this library run where device memory cannot be allocated at call time: all memory was
handed out at start-up, or the pool belongs to another component, or the stream must not stall on an
allocation.  xlog_reduce_by_key_static serves them with scratch that is built into the library.  Here
it is called twice in a row through the C ABI and each result is compared with what
xlog_relation_load + xlog_relation_read (the ordinary, arena-backed path) produce for the same rows, with the CPU
oracle's load of those rows, and with a per-group numpy reduction in float64; the second call must also leave the
device's free memory and torch's allocation count where they were.

Collected last on purpose (file name), so a run that stops at the first failure has already run
every other test.
"""
import numpy as np
import pytest

import oracle
from paper_2609_27203_b200 import synth

pytestmark = pytest.mark.gpu


def _case(n, n_keys, seed, sr):
    keys = np.sort(synth.randint(seed, 1, 0, n, n_keys)).astype(np.int32)
    tags = synth.normal(seed, 2, n).astype(np.float32)
    if sr == "sumprod":
        tags = np.abs(tags) + 0.25
    return keys, tags


def _reference(ctx, rel, keys, tags):
    ctx.load(rel, [keys], tags)
    cols, t = ctx.read(rel)
    return cols[0], t


def _oracle_reference(sr, keys, tags):
    o = oracle.Oracle()
    r = o.relation(1, sr)
    o.load(r, [keys], tags)
    cols, t = o.read(r)
    return cols[0], t


def _numpy_reference(sr, keys, tags):
    """Per-group reduction written out with numpy in float64 (keys ascending, so groups are runs)."""
    uk, first = np.unique(keys, return_index=True)
    t = tags.astype(np.float64)
    if sr == "minplus":
        return uk, np.minimum.reduceat(t, first)
    if sr == "maxplus":
        return uk, np.maximum.reduceat(t, first)
    if sr == "sumprod":
        return uk, np.add.reduceat(t, first)
    m = np.maximum.reduceat(t, first)
    grp = np.repeat(np.arange(len(uk)), np.diff(np.append(first, len(keys))))
    return uk, m + np.log(np.add.reduceat(np.exp(t - m[grp]), first))


def _check(sr, got_k, got_t, want_k, want_t, what):
    assert np.array_equal(got_k, want_k), what
    if sr in ("minplus", "maxplus"):
        assert np.array_equal(got_t, want_t.astype(np.float32)), what
    else:
        assert np.all(np.abs(got_t.astype(np.float64) - want_t) <= 1e-4 + 1e-5 * np.abs(want_t)), what


@pytest.mark.parametrize("sr", ["minplus", "maxplus", "logsumexp", "sumprod"])
def test_static_reduce_matches_the_arena_path_twice_in_a_row(sr):
    import torch
    from paper_2609_27203_b200 import xlog
    ctx = xlog.Context(arena_bytes=1 << 27)
    rel = ctx.relation(1, sr)
    # first call: many tiles, a ragged tail, one key owning tens of thousands of rows;
    # second call: a smaller input, so slots the first call filled are still lying in the scratch array
    for n, n_keys, seed in [(300_007, 5_000, 11), (4_099, 37, 12)]:
        keys, tags = _case(n, n_keys, seed, sr)
        keys[n // 3: n // 3 + n // 8] = keys[n // 3]           # one long group spanning several tiles
        keys.sort()
        want_k, want_t = _reference(ctx, rel, keys, tags)
        dk, dt = torch.from_numpy(keys).cuda(), torch.from_numpy(tags).cuda()
        ok, ot = torch.empty_like(dk), torch.empty_like(dt)
        u = xlog.reduce_by_key_static(sr, dk, dt, ok, ot)
        assert u == len(want_k)
        got_k, got_t = ok[:u].cpu().numpy(), ot[:u].cpu().numpy()
        assert np.array_equal(got_k, want_k)
        if sr in ("minplus", "maxplus"):
            assert np.array_equal(got_t.view(np.int32), want_t.view(np.int32))
        else:
            assert np.all(np.abs(got_t.astype(np.float64) - want_t) <= 1e-4 + 1e-5 * np.abs(want_t))
        # the same rows through the CPU oracle's load, and reduced group by group with numpy
        _check(sr, got_k, got_t, *_oracle_reference(sr, keys, tags), "oracle.load")
        _check(sr, got_k, got_t, *_numpy_reference(sr, keys, tags), "numpy")
    ctx.close()


def test_static_reduce_allocates_nothing_and_takes_the_largest_input():
    import torch
    from paper_2609_27203_b200 import xlog
    n = xlog.STATIC_REDUCE_MAX_ROWS
    keys = (np.arange(n, dtype=np.int64) // 3).astype(np.int32)            # groups of three rows
    tags = synth.normal(21, 2, n).astype(np.float32)
    dk, dt = torch.from_numpy(keys).cuda(), torch.from_numpy(tags).cuda()
    ok, ot = torch.empty_like(dk), torch.empty_like(dt)
    xlog.reduce_by_key_static("minplus", dk, dt, ok, ot)                   # warm-up: resolves the scratch array's address
    torch.cuda.synchronize()
    free0, alloc0, count0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated(), torch.cuda.memory_stats()["allocation.all.allocated"]
    u = xlog.reduce_by_key_static("minplus", dk, dt, ok, ot)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0 and torch.cuda.memory_allocated() == alloc0
    assert torch.cuda.memory_stats()["allocation.all.allocated"] == count0
    want_k, want_t = _numpy_reference("minplus", keys, tags)
    assert u == len(want_k)
    _check("minplus", ok[:u].cpu().numpy(), ot[:u].cpu().numpy(), want_k, want_t, "largest input")


def test_static_reduce_rejects_overlapping_buffers():
    import torch
    from paper_2609_27203_b200 import xlog
    k = torch.arange(1024, dtype=torch.int32, device="cuda")
    t = torch.zeros(1024, dtype=torch.float32, device="cuda")
    o = torch.empty(2048, dtype=torch.int32, device="cuda")
    with pytest.raises(ValueError):
        xlog.reduce_by_key_static("minplus", k, t, k, torch.empty_like(t))            # output on top of an input
    with pytest.raises(ValueError):
        xlog.reduce_by_key_static("minplus", k, t, o[:1024], o[512:1536].view(torch.float32))   # the two outputs overlap
    # the C entry point makes the same check for callers that do not come through the binding
    import ctypes as C
    n_out, err = C.c_int64(), C.create_string_buffer(256)
    st = xlog.lib().xlog_reduce_by_key_static(torch.cuda.current_stream().cuda_stream, 1, k.data_ptr(), t.data_ptr(), 1024, k.data_ptr(),
                                               o.data_ptr(), C.byref(n_out), err, len(err))
    assert xlog.STATUS[st] == "INVALID_ARGUMENT" and b"overlap" in err.value


def test_static_reduce_rejects_more_rows_than_its_scratch_covers():
    import torch
    from paper_2609_27203_b200 import xlog
    n = xlog.STATIC_REDUCE_MAX_ROWS + 1
    k = torch.zeros(n, dtype=torch.int32, device="cuda")
    t = torch.zeros(n, dtype=torch.float32, device="cuda")
    ok, ot = torch.empty_like(k), torch.empty_like(t)
    with pytest.raises(xlog.XlogError) as e:
        xlog.reduce_by_key_static("minplus", k, t, ok, ot)
    assert e.value.status == "CAPACITY_EXCEEDED" and "limit" in str(e.value)
    assert xlog.reduce_by_key_static("minplus", k[:0], t[:0], ok[:0], ot[:0]) == 0
