"""Unit parity of single kernels against plain numpy restatements (stable sort by the low key bits)."""
import numpy as np
import pytest

from paper_2609_27203_b200 import synth

pytestmark = pytest.mark.gpu


def _keys(n, bits, seed, skew):
    u = synth.uniform01(seed, 1, 0, n)
    if skew == "uniform":
        k = (u * (1 << bits)).astype(np.uint64)
    elif skew == "hot":                       # a few hot keys own most rows (hub-like)
        k = np.where(u < 0.7, (u * 8).astype(np.uint64), (u * (1 << bits)).astype(np.uint64))
    else:                                     # constant high digits: every tile sees one value in the top pass
        k = (u * (1 << min(bits, 9))).astype(np.uint64) | (np.uint64(1) << np.uint64(max(bits - 1, 0)))
    return k & np.uint64((1 << bits) - 1)


@pytest.mark.parametrize("n,bits,kb,skew", [
    (1, 8, 4, "uniform"), (2, 1, 4, "uniform"), (4097, 7, 4, "uniform"), (100_003, 20, 4, "uniform"),
    (1_000_000, 28, 4, "hot"), (3_000_017, 28, 4, "top"), (500_000, 32, 4, "uniform"),
    (250_000, 38, 8, "uniform"), (1_200_007, 62, 8, "hot"), (70_000, 9, 8, "top"), (65_536, 0, 4, "uniform"),
    # a thousand tiles and more
    (4_200_011, 30, 4, "hot"), (5_000_000, 19, 4, "uniform"), (4_500_003, 10, 4, "top"), (4_300_000, 47, 8, "uniform")])
def test_sort_pairs_is_a_stable_sort_on_the_low_bits(n, bits, kb, skew):
    import torch
    from paper_2609_27203_b200 import xlog
    k = _keys(n, bits, 5 + n % 7, skew) if bits else np.zeros(n, np.uint64)
    if bits < kb * 8 - 1:                     # bits above key_bits must not influence the order
        junk = (synth.rand_u64(9, 2, 0, n) >> np.uint64(64 - (kb * 8 - 1 - bits))) << np.uint64(bits)
        k = k | junk
    keys = k.astype(np.int64) if kb == 8 else k.astype(np.uint32).view(np.int32)
    payload = np.arange(n, dtype=np.int32)
    ctx = xlog.Context(arena_bytes=1 << 28)
    dk = torch.from_numpy(keys.copy()).cuda()
    dp = torch.from_numpy(payload.copy()).cuda()
    ctx.sort_pairs(dk, dp, bits)
    low = (k & np.uint64((1 << bits) - 1)) if bits else np.zeros(n, np.uint64)
    order = np.argsort(low, kind="stable")
    assert np.array_equal(dp.cpu().numpy(), payload[order])          # stable: ties keep input order
    assert np.array_equal(dk.cpu().numpy(), keys[order])
    ctx.close()


def test_a_look_back_wait_that_runs_out_fails_the_call_and_leaves_the_context_usable():
    # failure path of the bounded waits: one sort pass is launched without its first tile, so the status words every other
    # tile looks back to stay empty; with a poll limit of a thousand each wait gives up within a millisecond or so
    import time
    import torch
    from paper_2609_27203_b200 import xlog
    n = 64 * 4096 + 777                                   # 65 tiles, the last one ragged
    ctx = xlog.Context(arena_bytes=1 << 27)
    ctx.debug_set_poll_limit(1000)
    keys = torch.from_numpy(_keys(n, 20, 5, False).astype(np.int32)).cuda()
    vals = torch.arange(n, dtype=torch.int32, device="cuda")
    out_k = torch.full_like(keys, -7)
    out_v = torch.full_like(vals, -9)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    with pytest.raises(xlog.XlogError) as e:
        ctx.debug_sort_pass_without_first_tile(keys, vals, out_k, out_v)
    dt = time.perf_counter() - t0
    assert e.value.status == "INTERNAL"
    assert dt < 1.0, dt                                   # the kernel gave up on its own, in milliseconds (first-launch overhead included)
    assert bool((out_k == -7).all()) and bool((out_v == -9).all())          # no tile wrote anything
    # the context still works: an ordinary sort of the same rows, then a fixpoint
    k2, v2 = keys.clone(), vals.clone()
    ctx.sort_pairs(k2, v2, 20)
    order = np.argsort(keys.cpu().numpy(), kind="stable")
    assert np.array_equal(k2.cpu().numpy(), keys.cpu().numpy()[order]) and np.array_equal(v2.cpu().numpy(), order.astype(np.int32))
    ctx.reset_idb()
    e_rel = ctx.relation(2, "minplus")
    p_rel = ctx.relation(2, "minplus")
    ctx.load(e_rel, [np.array([0, 1], np.int32), np.array([1, 2], np.int32)], np.array([1.0, 2.0], np.float32))
    ctx.rule(p_rel, [(0, {0: 1}), (0, {1: 1})], [(e_rel, [("v", 0, 1, 0), ("v", 1, 1, 0)])])
    ctx.rule(p_rel, [(0, {0: 1}), (0, {2: 1})], [(p_rel, [("v", 0, 1, 0), ("v", 1, 1, 0)]), (e_rel, [("v", 1, 1, 0), ("v", 2, 1, 0)])])
    assert ctx.fixpoint()["derived_tuples"] == 3
    ctx.close()


def test_bandwidth_probe_kernels_copy_exactly_and_write_nothing_else():
    # the measuring kernels of the benchmark: the copy must copy, the two read-only probes must leave their sink untouched
    import torch
    from paper_2609_27203_b200 import xlog
    L = xlog.lib()
    s = torch.cuda.current_stream()
    n = (3 << 20) + 48                                            # a ragged tail of three 16-byte words
    src = torch.from_numpy(synth.randint(3, 1, 0, n // 4, 1 << 30).astype(np.int32)).cuda()
    dst = torch.zeros_like(src)
    assert L.xlog_device_copy(s.cuda_stream, dst.data_ptr(), src.data_ptr(), n, 2) == 0
    torch.cuda.synchronize()
    assert torch.equal(src, dst)
    sink = torch.zeros(1, dtype=torch.int32, device="cuda")
    assert L.xlog_device_read(s.cuda_stream, src.data_ptr(), n, 20, sink.data_ptr()) == 0
    assert L.xlog_device_gather(s.cuda_stream, src.data_ptr(), n, 1 << 20, sink.data_ptr()) == 0
    torch.cuda.synchronize()
    assert int(sink.item()) == 0 and torch.equal(src, dst)
    # bad arguments are refused before any launch
    assert L.xlog_device_copy(s.cuda_stream, dst.data_ptr(), src.data_ptr(), n + 4, 1) == 1
    assert L.xlog_device_read(s.cuda_stream, src.data_ptr() + 4, n - 16, 1, sink.data_ptr()) == 1
    assert L.xlog_device_read(s.cuda_stream, src.data_ptr(), n, 0, sink.data_ptr()) == 1
    assert L.xlog_device_gather(s.cuda_stream, src.data_ptr(), 0, 8, sink.data_ptr()) == 1
    assert L.xlog_device_gather(s.cuda_stream, None, n, 8, sink.data_ptr()) == 1
    for rate in (xlog.copy_bandwidth_gbs(8 << 20, 4), xlog.read_bandwidth_gbs(8 << 20, 16), xlog.gather_rate(8 << 20, 1 << 22)):
        assert rate > 0
