"""The allocation-free reduce-by-key entry point against the engine's ordinary path.

Some users of this library run where device memory cannot be allocated at call time: all memory was
handed out at start-up, or the pool belongs to another component, or the stream must not stall on an
allocation.  xlog_reduce_by_key_static serves them with scratch that is built into the library.  Here
it is called twice in a row through the C ABI and each result is compared with what
xlog_relation_load + xlog_relation_read (the ordinary, arena-backed path) produce for the same rows.

Collected last on purpose (file name), so a run that stops at the first failure has already run
every other test.
"""
import numpy as np
import pytest

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
    ctx.close()


def test_static_reduce_rejects_more_rows_than_its_scratch_covers():
    import torch
    from paper_2609_27203_b200 import xlog
    n = xlog.STATIC_REDUCE_MAX_ROWS + 1
    k = torch.zeros(n, dtype=torch.int32, device="cuda")
    t = torch.zeros(n, dtype=torch.float32, device="cuda")
    with pytest.raises(xlog.XlogError) as e:
        xlog.reduce_by_key_static("minplus", k, t, k, t)
    assert e.value.status == "CAPACITY_EXCEEDED" and "limit" in str(e.value)
    assert xlog.reduce_by_key_static("minplus", k[:0], t[:0], k[:0], t[:0]) == 0
