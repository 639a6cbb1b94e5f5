"""Pins for the CPU checker's allreduce: each test fixes the checker against
something that is not the checker itself (exact integer arithmetic, hand-worked
IEEE-754 cases, numpy library routines, rounding-error bounds, brute force)."""
import itertools
import math
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "fp32_order_cases.txt")


def words_for(arrived):
    """Notification words [S][W] from a boolean [P][S] table, written with Python
    integers (independent of the generator module's packer)."""
    P, S = len(arrived), len(arrived[0])
    W = (P + 63) // 64
    out = np.zeros((S, W), dtype=np.uint64)
    for s in range(S):
        for w in range(W):
            word = 0
            for r in range(w * 64, min(P, w * 64 + 64)):
                if arrived[r][s]:
                    word |= 1 << (r - w * 64)
            out[s, w] = np.uint64(word)
    return out


# ---------------------------------------------------------------------------
# brute force: every mask, tiny sizes, data on which the sum is exact
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("P,n,seg", [(1, 5, 2), (2, 6, 3), (3, 4, 2), (3, 8, 8), (4, 3, 1), (2, 7, 3)])
@pytest.mark.parametrize("dtype", [oracle.F32, oracle.I64, oracle.BF16, oracle.F64])
def test_every_mask_exact_sum(P, n, seg, dtype):
    S = (n + seg - 1) // seg
    rng = np.random.default_rng(7 + P * 100 + n)
    ints = rng.integers(-100, 100, size=(P, n))            # small integers: every dtype holds them exactly
    if dtype == oracle.BF16:
        bufs = [(np.asarray(ints[r], np.float32).view(np.uint32) >> 16).astype(np.uint16) for r in range(P)]
        # integers below 128 need at most 7 significand bits: truncation to bf16 loses nothing
        assert all(np.array_equal(((b.astype(np.uint32) << 16).view(np.float32)), ints[r].astype(np.float32))
                   for r, b in enumerate(bufs))
    else:
        bufs = [ints[r].astype({oracle.F32: np.float32, oracle.I64: np.int64, oracle.F64: np.float64}[dtype])
                for r in range(P)]
    out_np = {oracle.F32: np.float32, oracle.BF16: np.float32, oracle.I64: np.int64, oracle.F64: np.float64}[dtype]
    for bits in itertools.product([False, True], repeat=P * S):
        arrived = [[bits[r * S + s] for s in range(S)] for r in range(P)]
        ar = oracle.Allreduce(P, n, dtype, oracle.SUM, seg)
        res = np.full(n, 77, dtype=out_np)
        cnt = np.full(S, 99, dtype=np.uint32)
        ar.apply(bufs, words_for(arrived), res, cnt)
        for i in range(n):
            s = i // seg
            expect = sum(int(ints[r][i]) for r in range(P) if arrived[r][s])
            assert res[i] == expect, (arrived, i)
        for s in range(S):
            assert cnt[s] == sum(1 for r in range(P) if arrived[r][s])


@pytest.mark.parametrize("P,n,seg", [(2, 4, 2), (3, 3, 2), (2, 5, 5)])
def test_every_two_round_split(P, n, seg):
    """Each contribution arrives in round 1, in round 2 or never: 3^(P*S) schedules."""
    S = (n + seg - 1) // seg
    rng = np.random.default_rng(11)
    ints = rng.integers(-1000, 1000, size=(P, n))
    bufs = [ints[r].astype(np.int64) for r in range(P)]
    for when in itertools.product([0, 1, 2], repeat=P * S):          # 0 = never
        w = [[when[r * S + s] for s in range(S)] for r in range(P)]
        ar = oracle.Allreduce(P, n, oracle.I64, oracle.SUM, seg)
        res = np.full(n, -12345, dtype=np.int64)
        cnt = np.zeros(S, dtype=np.uint32)
        m1 = words_for([[w[r][s] == 1 for s in range(S)] for r in range(P)])
        ar.apply(bufs, m1, res, cnt)
        for i in range(n):
            assert res[i] == sum(int(ints[r][i]) for r in range(P) if w[r][i // seg] == 1)
        before = res.copy()
        m2 = words_for([[w[r][s] in (1, 2) for s in range(S)] for r in range(P)])
        ar.apply(bufs, m2, res, cnt)
        for i in range(n):
            s = i // seg
            assert res[i] == sum(int(ints[r][i]) for r in range(P) if w[r][s] in (1, 2))
            if not any(w[r][s] == 2 for r in range(P)):
                assert res[i] == before[i]
        for s in range(S):
            assert cnt[s] == sum(1 for r in range(P) if w[r][s] in (1, 2))


# ---------------------------------------------------------------------------
# order of accumulation: hand-worked binary32 cases
# ---------------------------------------------------------------------------
def _golden_cases():
    cases = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, vals, rounds, mode, expect = [t.strip() for t in line.split("|")]
            cases.append((name, [float(v) for v in vals.split()], [int(v) for v in rounds.split()], mode, float(expect)))
    return cases


@pytest.mark.parametrize("name,vals,rounds,mode,expect", _golden_cases(), ids=[c[0] for c in _golden_cases()])
def test_order_golden(name, vals, rounds, mode, expect):
    P = len(vals)
    bufs = [np.array([v], dtype=np.float32) for v in vals]
    ar = oracle.Allreduce(P, 1, oracle.F32, oracle.SUM, 1)
    res = np.full(1, np.nan, dtype=np.float32)
    order = oracle.ORDER_PAIRWISE if mode == "pairwise" else oracle.ORDER_FIXED
    for t in range(1, max(rounds) + 1):
        ar.apply(bufs, words_for([[rounds[r] <= t] for r in range(P)]), res, None, order=order)
    assert res[0] == np.float32(expect)
    # bf16 holds the same values (powers of two and one): same answers through the widening path
    if all(abs(v) in (1.0, 16777216.0) for v in vals):
        bb = [(b.view(np.uint32) >> 16).astype(np.uint16) for b in bufs]
        ar = oracle.Allreduce(P, 1, oracle.BF16, oracle.SUM, 1)
        res = np.full(1, np.nan, dtype=np.float32)
        for t in range(1, max(rounds) + 1):
            ar.apply(bb, words_for([[rounds[r] <= t] for r in range(P)]), res, None, order=order)
        assert res[0] == np.float32(expect)


def test_incremental_equals_oneshot_in_canonical_order():
    """Random three-round schedule: applying round by round gives the same bits as
    one fold per segment in the order (round of arrival, rank)."""
    P, n, seg = 9, 200, 16
    S = (n + seg - 1) // seg
    rng = np.random.default_rng(3)
    bufs = [(rng.standard_normal(n) * 10 ** rng.uniform(-3, 3)).astype(np.float32) for _ in range(P)]
    rounds = rng.integers(1, 5, size=(P, S))                 # 4 = never arrives
    rounds[:, 0] = 3                                          # a segment where everyone is late
    rounds[:, 1] = 4                                          # a segment nobody reaches
    ar = oracle.Allreduce(P, n, oracle.F32, oracle.SUM, seg)
    res = np.full(n, np.nan, dtype=np.float32)
    for t in (1, 2, 2, 3):                                    # round 2 applied twice: the repeat must change nothing
        ar.apply(bufs, words_for((rounds <= t).tolist()), res, None)
    order = np.full((S, P), -1, dtype=np.int32)
    for s in range(S):
        seq = sorted((int(rounds[r, s]), r) for r in range(P) if rounds[r, s] <= 3)
        order[s, :len(seq)] = [r for _, r in seq]
    one = oracle.allreduce_oneshot(bufs, oracle.F32, oracle.SUM, seg, order)
    assert np.array_equal(res.view(np.uint32), one.view(np.uint32))
    # and the oneshot itself against a scalar numpy-float32 fold of a few elements
    for i in (0, 17, 33, 199):
        acc = np.float32(0.0)
        for r in order[i // seg]:
            if r < 0:
                break
            acc = np.float32(acc + bufs[r][i])
        assert one[i] == acc


# ---------------------------------------------------------------------------
# closed forms and library special cases
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("P", [1, 2, 63, 64, 65, 128, 255, 256])
def test_word_boundaries_single_rank_bits(P):
    """Exactly one rank notified per segment, chosen to hit bit 0, 63 and word edges."""
    n, seg = 12, 1
    picks = [0, P - 1, min(P - 1, 63), min(P - 1, 64), min(P - 1, 127), min(P - 1, 128), P // 2, max(0, P - 2), 0, 0, 0, 0]
    bufs = [np.full(n, r + 1, dtype=np.int64) for r in range(P)]
    W = (P + 63) // 64
    mask = np.zeros((n, W), dtype=np.uint64)
    for s, r in enumerate(picks):
        mask[s, r // 64] = np.uint64(1 << (r % 64))
    # garbage above bit P-1 must be ignored
    if P % 64:
        mask[:, W - 1] |= np.uint64(((1 << 64) - 1) ^ ((1 << (P % 64)) - 1))
    ar = oracle.Allreduce(P, n, oracle.I64, oracle.SUM, seg)
    res = np.zeros(n, dtype=np.int64)
    cnt = np.zeros(n, dtype=np.uint32)
    ar.apply(bufs, mask, res, cnt)
    assert res.tolist() == [r + 1 for r in picks]
    assert cnt.tolist() == [1] * n


def test_full_mask_equals_numpy_reductions():
    P, n, seg = 37, 1000, 64
    rng = np.random.default_rng(5)
    raw = rng.integers(0, 2 ** 64, size=(P, n), dtype=np.uint64)
    bufs = [raw[r].view(np.int64).copy() for r in range(P)]
    for mask in (None, np.full(((n + seg - 1) // seg, 1), np.uint64(2 ** 64 - 1))):
        for op, ref in ((oracle.SUM, np.add.reduce(raw, axis=0).view(np.int64)),       # uint64 add wraps mod 2^64
                        (oracle.MAX, np.max(raw.view(np.int64), axis=0)),
                        (oracle.MIN, np.min(raw.view(np.int64), axis=0))):
            ar = oracle.Allreduce(P, n, oracle.I64, op, seg)
            res = np.zeros(n, dtype=np.int64)
            cnt = np.zeros(ar.S, dtype=np.uint32)
            ar.apply(bufs, mask, res, cnt)
            assert np.array_equal(res, ref)
            assert (cnt == P).all()


def test_float_max_min_equal_numpy():
    P, n, seg = 11, 300, 32
    rng = np.random.default_rng(6)
    bufs = [rng.standard_normal(n).astype(np.float32) for _ in range(P)]
    for op, fn in ((oracle.MAX, np.max), (oracle.MIN, np.min)):
        ar = oracle.Allreduce(P, n, oracle.F32, op, seg)
        res = np.zeros(n, dtype=np.float32)
        ar.apply(bufs, None, res, None)
        assert np.array_equal(res, fn(np.stack(bufs), axis=0))


def test_integer_valued_floats_match_integer_sum():
    """|partial sums| < 2^24: the fp32 sum is exact and order-free, so it must equal the integer sum."""
    P, n, seg = 16, 4096, 100
    S = (n + seg - 1) // seg
    rng = np.random.default_rng(8)
    ints = rng.integers(-(2 ** 19), 2 ** 19, size=(P, n))
    arrived = rng.random((P, S)) < 0.6
    mask = words_for(arrived.tolist())
    expect = np.zeros(n, dtype=np.int64)
    for r in range(P):
        sel = np.repeat(arrived[r], seg)[:n]
        expect += np.where(sel, ints[r], 0)
    for order in (oracle.ORDER_FIXED, oracle.ORDER_PAIRWISE):
        ar = oracle.Allreduce(P, n, oracle.F32, oracle.SUM, seg)
        res = np.empty(n, dtype=np.float32)
        ar.apply([ints[r].astype(np.float32) for r in range(P)], mask, res, None, order=order)
        assert np.array_equal(res.astype(np.int64), expect)
    # bf16: integers up to 255 are exact in 8 significand bits
    small = rng.integers(-255, 256, size=(P, n))
    bufs = [(small[r].astype(np.float32).view(np.uint32) >> 16).astype(np.uint16) for r in range(P)]
    expect = np.zeros(n, dtype=np.int64)
    for r in range(P):
        expect += np.where(np.repeat(arrived[r], seg)[:n], small[r], 0)
    ar = oracle.Allreduce(P, n, oracle.BF16, oracle.SUM, seg)
    res = np.empty(n, dtype=np.float32)
    ar.apply(bufs, mask, res, None)
    assert np.array_equal(res.astype(np.int64), expect)


def test_rounding_error_bounds_against_exact_sum():
    """Sequential fp32 summation of P terms errs by at most gamma_(P-1) * sum|x|, the pairwise
    tree by gamma_ceil(log2 P) * sum|x| (Higham, Accuracy and Stability, Sec. 4.2); exact sums by math.fsum."""
    P, n, seg = 32, 2000, 128
    rng = np.random.default_rng(9)
    bufs = [rng.standard_normal(n).astype(np.float32) for _ in range(P)]
    u = 2.0 ** -24

    def gamma(k):
        return k * u / (1 - k * u)

    exact = np.array([math.fsum(float(b[i]) for b in bufs) for i in range(n)])
    mag = np.array([math.fsum(abs(float(b[i])) for b in bufs) for i in range(n)])
    for order, k in ((oracle.ORDER_FIXED, P - 1), (oracle.ORDER_PAIRWISE, 5)):
        ar = oracle.Allreduce(P, n, oracle.F32, oracle.SUM, seg)
        res = np.empty(n, dtype=np.float32)
        ar.apply(bufs, None, res, None, order=order)
        err = np.abs(res.astype(np.float64) - exact)
        assert (err <= gamma(k) * mag).all()
        assert err.max() > 0                       # it really is fp32 arithmetic, not a double sum rounded once
    ref, mag64 = oracle.allreduce_ref64(bufs, oracle.F32, seg, None)
    assert np.allclose(ref, exact, rtol=0, atol=1e-12)
    assert np.allclose(mag64, mag, rtol=1e-14)


def test_ref64_respects_mask():
    P, n, seg = 5, 40, 8
    rng = np.random.default_rng(10)
    bufs = [rng.standard_normal(n).astype(np.float32) for _ in range(P)]
    arrived = rng.random((P, 5)) < 0.5
    ref, mag = oracle.allreduce_ref64(bufs, oracle.F32, seg, words_for(arrived.tolist()))
    for i in range(n):
        xs = [float(bufs[r][i]) for r in range(P) if arrived[r][i // seg]]
        assert abs(ref[i] - math.fsum(xs)) < 1e-12
        assert abs(mag[i] - math.fsum(abs(x) for x in xs)) < 1e-12


def test_special_cases():
    # P = 1: identity (+) buf_0 is a copy, except that -0.0 becomes +0.0 under sum
    b = np.array([1.5, -0.0, 0.0, -3.25, np.inf], dtype=np.float32)
    ar = oracle.Allreduce(1, 5, oracle.F32, oracle.SUM, 2)
    res = np.full(5, 9, dtype=np.float32)
    ar.apply([b], None, res, None)
    assert np.array_equal(res, b) and not np.signbit(res[1])
    ar = oracle.Allreduce(1, 5, oracle.F32, oracle.MAX, 2)
    ar.apply([b], None, res, None)
    assert np.array_equal(res.view(np.uint32), b.view(np.uint32))        # max keeps -0.0 (it is > -inf)
    # constant buffers: result is the fold of the constants over the notified ranks
    P, n = 6, 50
    consts = [0.1, 0.2, 0.3, 0.4, 0.5, 0.6]
    bufs = [np.full(n, c, dtype=np.float32) for c in consts]
    for seg in (1, 7, 50, 64):                                           # seg = 1, ragged, seg = n, seg > n
        S = (n + seg - 1) // seg
        arrived = [[(r + s) % 2 == 0 for s in range(S)] for r in range(P)]
        ar = oracle.Allreduce(P, n, oracle.F32, oracle.SUM, seg)
        res = np.full(n, np.nan, dtype=np.float32)
        cnt = np.zeros(S, dtype=np.uint32)
        ar.apply(bufs, words_for(arrived), res, cnt)
        for i in range(n):
            acc = np.float32(0)
            for r in range(P):
                if arrived[r][i // seg]:
                    acc = np.float32(acc + np.float32(consts[r]))
            assert res[i] == acc
        assert cnt.tolist() == [sum(arrived[r][s] for r in range(P)) for s in range(S)]


def test_unnotified_bytes_never_reach_the_result():
    """Validity rule: data counts only once its notification is visible.  Poison what has not arrived."""
    P, n, seg = 7, 90, 10
    S = 9
    rng = np.random.default_rng(12)
    clean = [rng.standard_normal(n).astype(np.float32) for _ in range(P)]
    rounds = rng.integers(1, 4, size=(P, S))
    ar = oracle.Allreduce(P, n, oracle.F32, oracle.SUM, seg)
    ref = oracle.Allreduce(P, n, oracle.F32, oracle.SUM, seg)
    res = np.full(n, 5, dtype=np.float32)
    res_ref = np.full(n, 5, dtype=np.float32)
    for t in (1, 2, 3):
        arrived = rounds <= t
        poisoned = []
        for r in range(P):
            b = clean[r].copy()
            b[~np.repeat(arrived[r], seg)[:n]] = np.nan
            poisoned.append(b)
        ar.apply(poisoned, words_for(arrived.tolist()), res, None)
        ref.apply(clean, words_for(arrived.tolist()), res_ref, None)
        assert not np.isnan(res).any()
        assert np.array_equal(res.view(np.uint32), res_ref.view(np.uint32))
    # int64 with a byte pattern as poison
    ints = [rng.integers(0, 1 << 20, size=n, dtype=np.int64) for _ in range(P)]
    arrived = rounds <= 1
    bufs = []
    for r in range(P):
        b = ints[r].copy()
        b[~np.repeat(arrived[r], seg)[:n]] = 0x5A5A5A5A5A5A5A5A
        bufs.append(b)
    ar = oracle.Allreduce(P, n, oracle.I64, oracle.MAX, seg)
    res = np.zeros(n, dtype=np.int64)
    ar.apply(bufs, words_for(arrived.tolist()), res, None)
    assert res.max() < (1 << 20) or (res == np.iinfo(np.int64).min).any()
    assert not (res == 0x5A5A5A5A5A5A5A5A).any()


def test_first_apply_writes_identity_and_later_applies_leave_idle_segments_alone():
    P, n, seg = 3, 12, 4
    bufs = [np.arange(n, dtype=np.float32) + r for r in range(P)]
    for op, ident in ((oracle.SUM, 0.0), (oracle.MAX, -np.inf), (oracle.MIN, np.inf)):
        ar = oracle.Allreduce(P, n, oracle.F32, op, seg)
        res = np.full(n, 123.0, dtype=np.float32)
        cnt = np.full(3, 9, dtype=np.uint32)
        arrived = [[True, False, False], [False, False, False], [True, False, False]]
        ar.apply(bufs, words_for(arrived), res, cnt)
        assert (res[4:] == ident).all() and cnt.tolist() == [2, 0, 0]
        res[8:] = 555.0                                       # scribble over an idle segment
        arrived[1][1] = True
        ar.apply(bufs, words_for(arrived), res, cnt)
        assert (res[8:] == 555.0).all()                       # untouched: nothing new arrived there
        assert np.array_equal(res[4:8], bufs[1][4:8] if op != oracle.SUM else bufs[1][4:8] + 0.0)
        assert cnt.tolist() == [2, 1, 0]
        # clearing a bit later does not un-apply anything
        arrived[0][0] = False
        before = res.copy()
        ar.apply(bufs, words_for(arrived), res, cnt)
        assert np.array_equal(res, before) and cnt.tolist() == [2, 1, 0]
        # a new epoch starts over
        ar.reset()
        ar.apply(bufs, words_for([[False] * 3] * 3), res, cnt)
        assert (res == ident).all() and cnt.tolist() == [0, 0, 0]
    i64 = oracle.Allreduce(2, 4, oracle.I64, oracle.MAX, 2)
    r64 = np.zeros(4, dtype=np.int64)
    i64.apply([np.zeros(4, np.int64)] * 2, words_for([[False, False]] * 2), r64, None)
    assert (r64 == np.iinfo(np.int64).min).all()


def test_permutation_invariance_of_integer_paths():
    P, n, seg = 8, 64, 8
    rng = np.random.default_rng(13)
    bufs = [rng.integers(0, 2 ** 64, size=n, dtype=np.uint64).view(np.int64) for _ in range(P)]
    outs = []
    for trial in range(4):
        perm = rng.permutation(P)
        rounds = rng.integers(1, 4, size=(P, 8))
        for op in (oracle.SUM, oracle.MAX):
            ar = oracle.Allreduce(P, n, oracle.I64, op, seg)
            res = np.zeros(n, dtype=np.int64)
            for t in (1, 2, 3):
                ar.apply([bufs[p] for p in perm], words_for((rounds <= t).tolist()), res, None)
            outs.append((op, res.copy()))
    for op, res in outs:
        first = next(r for o, r in outs if o == op)
        assert np.array_equal(res, first)


def test_threads_do_not_change_bits():
    P, n, seg = 12, 5000, 97
    rng = np.random.default_rng(14)
    bufs = [rng.standard_normal(n).astype(np.float32) for _ in range(P)]
    S = (n + seg - 1) // seg
    mask = words_for((rng.random((P, S)) < 0.7).tolist())
    outs = []
    for th in (1, 4):
        ar = oracle.Allreduce(P, n, oracle.F32, oracle.SUM, seg)
        res = np.empty(n, dtype=np.float32)
        ar.apply(bufs, mask, res, None, threads=th)
        outs.append(res)
    assert np.array_equal(outs[0].view(np.uint32), outs[1].view(np.uint32))
