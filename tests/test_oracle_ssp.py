"""Pins for the CPU checker's stale-synchronous allreduce: the examples the paper prints for
Algorithm 1 (tests/golden/ssp_examples.txt), exact integer sums over the accepted set, and the
equivalence with the notification-bit allreduce when the accepted set is given as a mask."""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "ssp_examples.txt")


def cases():
    out = []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        name, clock, slack, clocks, acc, red = [t.strip() for t in line.split("|")]
        out.append((name, int(clock), int(slack), [int(c) for c in clocks.split()], [int(a) for a in acc.split()], int(red)))
    return out


@pytest.mark.parametrize("name,clock,slack,clocks,accepted,red_clock", cases(), ids=[c[0] for c in cases()])
def test_printed_examples(name, clock, slack, clocks, accepted, red_clock):
    P = len(clocks)
    bufs = [np.array([10 ** r], dtype=np.int64) for r in range(P)]          # each rank contributes a distinct decimal digit
    res, cnt, seg_clock, wait = oracle.allreduce_ssp(bufs, oracle.I64, oracle.SUM, 1, np.array([clocks]), clock, slack)
    assert res[0] == sum(10 ** r for r in range(P) if accepted[r])
    assert cnt[0] == sum(accepted) and wait[0] == P - sum(accepted)
    assert seg_clock[0] == red_clock


def test_nothing_received_yet_and_identity():
    bufs = [np.arange(6, dtype=np.float32) + r for r in range(3)]
    clocks = np.zeros((2, 3), dtype=np.uint32)          # clock 0 = nothing received
    clocks[1] = [4, 0, 9]
    res, cnt, seg_clock, wait = oracle.allreduce_ssp(bufs, oracle.F32, oracle.SUM, 3, clocks, 9, 2)
    assert (res[:3] == 0).all() and cnt[0] == 0 and seg_clock[0] == 0 and wait[0] == 3
    assert np.array_equal(res[3:], bufs[2][3:]) and cnt[1] == 1 and seg_clock[1] == 9 and wait[1] == 2
    res, cnt, seg_clock, wait = oracle.allreduce_ssp(bufs, oracle.F32, oracle.MAX, 3, clocks, 9, 5)
    assert (res[:3] == -np.inf).all()
    assert np.array_equal(res[3:], np.maximum(bufs[0][3:], bufs[2][3:])) and seg_clock[1] == 4 and wait[1] == 1


def test_equals_masked_allreduce_and_exact_sums():
    P, n, seg = 70, 500, 32
    S = (n + seg - 1) // seg
    rng = np.random.default_rng(4)
    ints = rng.integers(-1000, 1000, size=(P, n))
    clocks = rng.integers(0, 12, size=(S, P)).astype(np.uint32)
    clock, slack = 11, 3
    accepted = (clocks >= clock - slack)                                  # [S][P]; clock 0 never reaches 8
    for dtype, npdt in ((oracle.I64, np.int64), (oracle.F32, np.float32)):
        bufs = [ints[r].astype(npdt) for r in range(P)]
        res, cnt, seg_clock, wait = oracle.allreduce_ssp(bufs, dtype, oracle.SUM, seg, clocks, clock, slack)
        expect = np.zeros(n, dtype=np.int64)
        for r in range(P):
            expect += np.where(np.repeat(accepted[:, r], seg)[:n], ints[r], 0)
        assert np.array_equal(res.astype(np.int64), expect)
        assert np.array_equal(cnt, accepted.sum(1)) and np.array_equal(wait, P - accepted.sum(1))
        want_clock = np.where(accepted, clocks, 2 ** 31).min(1)
        assert np.array_equal(seg_clock, np.where(accepted.any(1), want_clock, 0))
    # the same accepted set as notification bits through the stateful allreduce: same bits
    vals = [rng.standard_normal(n).astype(np.float32) for _ in range(P)]
    res, _, _, _ = oracle.allreduce_ssp(vals, oracle.F32, oracle.SUM, seg, clocks, clock, slack)
    words = np.zeros((S, 2), dtype=np.uint64)
    for s in range(S):
        for r in range(P):
            if accepted[s, r]:
                words[s, r // 64] |= np.uint64(1 << (r % 64))
    ar = oracle.Allreduce(P, n, oracle.F32, oracle.SUM, seg)
    ref = np.empty(n, dtype=np.float32)
    ar.apply(vals, words, ref, None)
    assert np.array_equal(res.view(np.uint32), ref.view(np.uint32))


def test_large_slack_accepts_everything_received():
    P, n = 5, 20
    bufs = [np.full(n, r + 1, dtype=np.int64) for r in range(P)]
    clocks = np.array([[1, 2, 3, 0, 50]], dtype=np.uint32)
    res, cnt, seg_clock, wait = oracle.allreduce_ssp(bufs, oracle.I64, oracle.SUM, n, clocks, 50, 64)   # slack beyond the clock
    assert res[0] == 1 + 2 + 3 + 5 and cnt[0] == 4 and wait[0] == 1 and seg_clock[0] == 1
