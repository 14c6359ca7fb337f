"""Host-side range cutting for the key split of a decode step (no GPU, no process group)."""
import numpy as np
import pytest

from paper_2604_07394_b200 import keysplit


@pytest.mark.parametrize("world", [1, 2, 3, 8])
@pytest.mark.parametrize("align", [1, 16, 64])
def test_key_ranges_cover_every_position_once(world, align):
    lens = [0, 1, 15, 16, 17, 4224, 65536, 131073]
    r = keysplit.key_ranges(lens, world, align)
    assert r.shape == (world, len(lens), 2) and r.dtype == np.int32
    n = np.asarray(lens)
    assert (r[0, :, 0] == 0).all() and (r[-1, :, 1] == n).all()          # first range starts at 0, last ends at n
    assert (r[1:, :, 0] == r[:-1, :, 1]).all()                           # consecutive, no gap, no overlap
    assert (r[:, :, 1] >= r[:, :, 0]).all()                              # possibly empty, never negative
    inner = r[:-1, :, 1]
    assert ((inner % align == 0) | (inner == n[None, :])).all()          # inner bounds on the kernels' tile grid
    if world > 1:                                                        # long requests are cut almost evenly
        sizes = (r[:, -1, 1] - r[:, -1, 0]).astype(np.int64)
        assert sizes.max() - sizes.min() <= 2 * align


def test_key_ranges_hand_typed():
    r = keysplit.key_ranges([100, 5], 2, 16)
    assert r.tolist() == [[[0, 64], [0, 5]], [[64, 100], [5, 5]]]        # 50 rounded up to 64; 2.5 -> 16, clipped to 5
    assert keysplit.key_ranges([48], 3, 16).tolist() == [[[0, 16]], [[16, 32]], [[32, 48]]]


def test_exchange_sequence_numbers_and_buffer_sets():
    seqs = [keysplit.exchange_seq(t) for t in range(6)] + [keysplit.exchange_seq(0xFFFFFFFE), keysplit.exchange_seq(0xFFFFFFFF)]
    assert seqs[:3] == [1, 2, 3] and all(0 < s <= 0xFFFFFFFF for s in seqs)
    assert all(a != b for a, b in zip(seqs, seqs[1:]))                   # also across the wrap: 0xFFFFFFFF then 1
    assert [keysplit.buffer_set(t, l, 3) for t in range(2) for l in range(3)] == [0, 1, 2, 0, 1, 2]
    assert [keysplit.buffer_set(t, 0, 1) for t in range(4)] == [0, 1, 0, 1]
