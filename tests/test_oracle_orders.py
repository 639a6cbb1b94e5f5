"""Pins for the schedule-faithful accumulation orders: the checker's ring and pairwise orders must give,
bit for bit, what literal simulations of the paper's exchange schedules give in fp32."""
import numpy as np
import pytest

import oracle


def simulate_ring_scatter_reduce(bufs):
    """Segmented pipelined ring, Scatter-Reduce stage (Sec. IV-A): P nodes, P chunks; in step k node i sends
    chunk i-k to its clockwise neighbour and receives chunk i-k-1 from the other one, reducing it into its own
    data of that chunk.  After P-1 steps every node holds the complete result of one chunk."""
    P = len(bufs)
    n = bufs[0].size
    chunk = (n + P - 1) // P
    data = [b.copy() for b in bufs]

    def sl(c):
        return slice(c * chunk, min(n, (c + 1) * chunk))

    for k in range(P - 1):
        sent = [data[i][sl((i - k) % P)].copy() for i in range(P)]           # all nodes send at once
        for i in range(P):
            c = (i - k - 1) % P                                              # chunk received from node i-1
            data[i][sl(c)] = data[i][sl(c)] + sent[(i - 1) % P]              # existing (+) received
    out = np.empty(n, dtype=bufs[0].dtype)
    for i in range(P):
        c = (i + 1) % P                                                      # = i - (P-1): the chunk node i completed
        out[sl(c)] = data[i][sl(c)]
    return out


@pytest.mark.parametrize("P,n,seg", [(4, 64, 4), (5, 100, 10), (8, 1024, 32), (16, 160, 10), (3, 30, 10)])
def test_ring_order_equals_the_simulated_ring(P, n, seg):
    rng = np.random.default_rng(P)
    bufs = [(rng.standard_normal(n) * 10.0 ** rng.integers(-3, 4)).astype(np.float32) for _ in range(P)]
    sim = simulate_ring_scatter_reduce(bufs)
    ar = oracle.Allreduce(P, n, oracle.F32, oracle.SUM, seg)
    res = np.empty(n, dtype=np.float32)
    ar.apply(bufs, None, res, None, order=oracle.ORDER_RING)
    assert np.array_equal(res.view(np.uint32), sim.view(np.uint32))
    # and it differs from plain rank order somewhere (the orders are really different)
    ar2 = oracle.Allreduce(P, n, oracle.F32, oracle.SUM, seg)
    res2 = np.empty(n, dtype=np.float32)
    ar2.apply(bufs, None, res2, None)
    if P > 2:
        assert not np.array_equal(res.view(np.uint32), res2.view(np.uint32))


@pytest.mark.parametrize("P", [2, 4, 8, 16])
def test_pairwise_order_equals_the_simulated_hypercube(P):
    """Hypercube allreduce (Sec. III-A): log2(P) steps; in step k process i exchanges its partial reduction
    with process i xor 2^k and reduces.  Process 0 hears from 1, 2, 4, ... as the paper's example says."""
    n = 500
    rng = np.random.default_rng(100 + P)
    bufs = [(rng.standard_normal(n) * 10.0 ** rng.integers(-3, 4)).astype(np.float32) for _ in range(P)]
    part = [b.copy() for b in bufs]
    heard_by_0 = []
    k = 0
    while (1 << k) < P:
        heard_by_0.append(0 ^ (1 << k))
        part = [part[i] + part[i ^ (1 << k)] for i in range(P)]
        k += 1
    assert heard_by_0 == [1, 2, 4, 8][:k]
    ar = oracle.Allreduce(P, n, oracle.F32, oracle.SUM, 64)
    res = np.empty(n, dtype=np.float32)
    ar.apply(bufs, None, res, None, order=oracle.ORDER_PAIRWISE)
    for i in range(P):                                    # every process ends with the same bits
        assert np.array_equal(part[i].view(np.uint32), res.view(np.uint32))


def test_ring_order_with_late_arrivals():
    """Each apply folds its new ranks in the chunk's cyclic order; int64 keeps it order-free, fp32 is
    checked against a hand-rolled fold."""
    P, n, seg = 6, 36, 3
    rng = np.random.default_rng(9)
    bufs = [rng.standard_normal(n).astype(np.float32) for _ in range(P)]
    rounds = rng.integers(1, 3, size=(P, n // seg))
    ar = oracle.Allreduce(P, n, oracle.F32, oracle.SUM, seg)
    res = np.empty(n, dtype=np.float32)
    for t in (1, 2):
        arrived = rounds <= t
        words = np.zeros((n // seg, 1), dtype=np.uint64)
        for s in range(n // seg):
            for r in range(P):
                if arrived[r, s]:
                    words[s, 0] |= np.uint64(1 << r)
        ar.apply(bufs, words, res, None, order=oracle.ORDER_RING)
    chunk = n // P
    for i in range(n):
        s, c = i // seg, i // chunk
        acc = np.float32(0)
        for t in (1, 2):
            for step in range(P):
                r = (c + step) % P
                if rounds[r, s] == t:
                    acc = np.float32(acc + bufs[r][i])
        assert res[i] == acc
