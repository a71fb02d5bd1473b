"""Host arithmetic of the attention kernels' context-split schedules (Sec. 4.3 leaves the partition open; the oracle's
tiled mode takes it as data): no GPU needed - the balanced schedule's grid size is passed in instead of asked of a
device."""
import numpy as np
import pytest

from paper_2605_13915_b200 import binding

TILE = 128


@pytest.fixture(autouse=True)
def _reset_options():
    yield
    binding.debug_reset_options()


def _runs(starts, seqlens):
    """The splits of all sequences laid end to end, in tiles: list of (first tile, tiles) per split of head 0."""
    out, base = [], 0
    for b, L in enumerate(seqlens):
        s = starts[b, 0, 0]
        nb = (L + TILE - 1) // TILE
        for a, e in zip(s[:-1], s[1:]):
            if e > a:
                out.append((base + a // TILE, (min(e, nb * TILE) - a + TILE - 1) // TILE))
        base += nb
    return out


@pytest.mark.parametrize("seed,B,Hq,Hkv,lo,hi,ctas", [(0, 32, 32, 8, 2048, 8192, 444), (1, 300, 8, 2, 0, 1200, 444),
                                                     (2, 5, 16, 2, 1, 40000, 444), (3, 7, 4, 4, 0, 300, 296)])
def test_balanced_schedule_cuts_equal_runs(seed, B, Hq, Hkv, lo, hi, ctas):
    binding.debug_set_option("MSD_ATTN_BALANCED", 1)
    rng = np.random.default_rng(seed)
    L = rng.integers(lo, hi + 1, B).astype(np.int32)
    L[rng.integers(0, B)] = 0                                     # an empty sequence somewhere
    tile, ns, st = binding.attn_decode_schedule(B, Hq, Hkv, 128, 128, int(L.max()))
    assert tile == TILE and st == 0                               # balanced: no fixed split size
    starts, _ = binding.attn_decode_split_starts(L, Hq, Hkv, 128, 128, int(L.max()), resident_ctas=ctas)
    assert starts.shape == (B, Hkv, Hq // Hkv, ns + 1)
    assert np.all(starts == starts[:, :1, :1])                   # the same for every head of a sequence
    s = starts[:, 0, 0]
    assert np.all(s[:, 0] == 0) and np.all(s[:, -1] == L) and np.all(np.diff(s, axis=1) >= 0)
    inner = s[:, 1:][s[:, 1:] < L[:, None]]
    assert np.all(inner % TILE == 0)                              # every cut on a tile boundary
    # the splits are the pieces of R equal consecutive runs of the list of all tiles, cut again at sequence ends
    nb = (L.astype(np.int64) + TILE - 1) // TILE
    W = int(nb.sum())
    pieces = _runs(starts, L)
    assert sum(n for _, n in pieces) == W and [f for f, _ in pieces] == sorted(f for f, _ in pieces)
    assert all(f2 == f1 + n1 for (f1, n1), (f2, _) in zip(pieces[:-1], pieces[1:]))      # no gap, no overlap
    cuts = {f for f, _ in pieces}
    seq_starts = set(np.cumsum(np.concatenate([[0], nb]))[:-1].tolist())
    max_runs = max(ctas // Hkv, 1)                                # one CTA per run and KV head (one head group each here)
    fits = [R for R in range(1, max_runs + 1)
            if {i * W // R for i in range(R)} <= cuts and cuts <= {i * W // R for i in range(R)} | seq_starts]
    assert fits, "the cuts are not those of equal runs"
    R = max(fits)
    sizes = np.diff(sorted({i * W // R for i in range(R)}) + [W])
    assert sizes.max() - sizes.min() <= 1
    assert R == max_runs or sizes.min() < 2 * 8                   # fewer runs only to keep them a few tiles long
    assert (np.diff(s, axis=1) > 0).sum(axis=1).max() <= ns       # as many partial results as the workspace holds


def test_fixed_schedule_is_uniform():
    binding.debug_set_option("MSD_ATTN_BALANCED", 0)
    L = np.array([100, 0, 5000, 2048], np.int32)
    tile, ns, st = binding.attn_decode_schedule(4, 32, 8, 128, 128, 5000)
    assert st > 0 and st % tile == 0 and ns == -(-5000 // st)
    starts, _ = binding.attn_decode_split_starts(L, 32, 8, 128, 128, 5000, resident_ctas=444)
    want = np.minimum(L[:, None], np.arange(ns + 1)[None, :] * st)
    assert np.array_equal(starts[:, 0, 0], want) and np.all(starts == starts[:, :1, :1])


def test_schedule_choice_by_shape():
    """Balanced where full-size fixed splits would leave the resident CTAs one to three items each and the sequences
    are long; fixed splits elsewhere; wide head groups always fixed."""
    sched = binding.attn_decode_schedule
    assert sched(32, 32, 8, 128, 128, 8192)[2] == 0
    assert sched(32, 64, 8, 128, 128, 8192)[2] == 0
    assert sched(512, 32, 8, 128, 128, 8192)[2] > 0
    assert sched(1, 32, 8, 128, 128, 8192)[2] > 0
    assert sched(256, 32, 8, 128, 128, 1024)[2] > 0
    assert sched(32, 128, 8, 128, 128, 8192)[2] > 0
    assert sched(64, 64, 1, 576, 512, 16384)[2] > 0
    assert sched(32, 32, 8, 256, 256, 8192)[2] > 0
