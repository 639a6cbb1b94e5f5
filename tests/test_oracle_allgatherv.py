"""Pins for the CPU checker's allgatherv: numpy's cumsum and concatenate are the
library special cases; sentinels show which slots were written."""
import numpy as np
import pytest

import oracle

SENT = np.int64(-0x0123456789ABCDEF)


def mask_words(arrived):
    P = len(arrived)
    W = (P + 63) // 64
    out = np.zeros(W, dtype=np.uint64)
    for r, a in enumerate(arrived):
        if a:
            out[r // 64] |= np.uint64(1 << (r % 64))
    return out


@pytest.mark.parametrize("P", [1, 3, 64, 65, 256])
def test_all_arrived_is_concatenation(P):
    rng = np.random.default_rng(P)
    counts = rng.integers(0, 50, size=P).astype(np.int64)
    counts[0] = 7
    bufs = [rng.integers(-2 ** 63, 2 ** 63 - 1, size=int(c), dtype=np.int64) for c in counts]
    total = int(counts.sum())
    out = np.full(total + 4, SENT, dtype=np.int64)
    for mask in (None, mask_words([True] * P)):
        out[:] = SENT
        displs, status = oracle.allgatherv(bufs, counts, mask, out)
        assert status == 0
        assert displs[0] == 0 and np.array_equal(displs[1:], np.cumsum(counts))
        assert np.array_equal(out[:total], np.concatenate(bufs))
        assert (out[total:] == SENT).all()


def test_equal_counts_closed_form():
    P, c = 10, 13
    counts = np.full(P, c, dtype=np.int64)
    bufs = [np.full(c, r, dtype=np.int64) for r in range(P)]
    out = np.empty(P * c, dtype=np.int64)
    displs, _ = oracle.allgatherv(bufs, counts, None, out)
    assert displs.tolist() == [r * c for r in range(P + 1)]
    assert np.array_equal(out, np.repeat(np.arange(P), c))


def test_missing_ranks_keep_their_slots_untouched():
    P = 70
    rng = np.random.default_rng(2)
    counts = rng.integers(1, 30, size=P).astype(np.int64)
    bufs = [rng.integers(0, 1000, size=int(c), dtype=np.int64) for c in counts]
    arrived = rng.random(P) < 0.6
    arrived[64] = True
    arrived[63] = False
    poisoned = [b if arrived[r] else np.full_like(b, 0x5A5A5A5A5A5A5A5A) for r, b in enumerate(bufs)]
    out = np.full(int(counts.sum()), SENT, dtype=np.int64)
    displs, status = oracle.allgatherv(poisoned, counts, mask_words(arrived), out)
    assert status == 0
    for r in range(P):
        slot = out[displs[r]:displs[r + 1]]
        assert np.array_equal(slot, bufs[r]) if arrived[r] else (slot == SENT).all()
    # a late arrival later is one more copy into the same slot
    late = ~arrived
    displs2, _ = oracle.allgatherv(bufs, counts, mask_words(late), out)
    assert np.array_equal(displs, displs2)
    assert np.array_equal(out, np.concatenate(bufs))


def test_capacity_exceeded_writes_nothing():
    counts = np.array([5, 6, 7], dtype=np.int64)
    bufs = [np.arange(int(c), dtype=np.int64) for c in counts]
    out = np.full(17, SENT, dtype=np.int64)          # needs 18
    displs, status = oracle.allgatherv(bufs, counts, None, out)
    assert status != 0 and (out == SENT).all()
    assert displs.tolist() == [0, 5, 11, 18]


def test_other_element_sizes():
    counts = np.array([3, 0, 5], dtype=np.int64)
    for dt in (np.float32, np.uint16, np.float64):
        bufs = [np.arange(int(c)).astype(dt) + 10 * r for r, c in enumerate(counts)]
        out = np.zeros(8, dtype=dt)
        oracle.allgatherv(bufs, counts, None, out)
        assert np.array_equal(out, np.concatenate(bufs))


def test_compact_reading_is_the_concatenation_of_the_arrived_ranks():
    P = 70
    rng = np.random.default_rng(8)
    counts = rng.integers(0, 30, size=P).astype(np.int64)
    bufs = [rng.integers(0, 1000, size=int(c), dtype=np.int64) for c in counts]
    arrived = rng.random(P) < 0.6
    total = int(counts[arrived].sum())
    out = np.full(total + 3, SENT, dtype=np.int64)
    displs, status = oracle.allgatherv(bufs, counts, mask_words(arrived), out, compact=True)
    assert status == 0
    assert np.array_equal(out[:total], np.concatenate([b for b, a in zip(bufs, arrived) if a]))
    assert (out[total:] == SENT).all()
    assert displs[0] == 0 and np.array_equal(np.diff(displs), np.where(arrived, counts, 0))
    # with everything arrived both readings coincide
    out2 = np.empty(int(counts.sum()), dtype=np.int64)
    d1, _ = oracle.allgatherv(bufs, counts, None, out2, compact=True)
    out3 = np.empty_like(out2)
    d2, _ = oracle.allgatherv(bufs, counts, None, out3)
    assert np.array_equal(d1, d2) and np.array_equal(out2, out3)
