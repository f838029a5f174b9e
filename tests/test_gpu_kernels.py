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
