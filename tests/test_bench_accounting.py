"""The benchmark's algorithmic byte count (what the roofline fraction is computed from) against a
plain loop over (rank, segment) pairs and against the closed forms of the all-arrived case."""
import numpy as np

import bench
from paper_2203_17063_b200 import inputs


def brute(prev_rounds_done, rounds, t, P, n, seg, in_b, out_b):
    """Bytes of apply number t (1-based) of a schedule rounds[r][s]: new inputs + result written (+ read back)."""
    S = (n + seg - 1) // seg
    total = 0
    for s in range(S):
        length = min(seg, n - s * seg)
        new = sum(1 for r in range(P) if rounds[r, s] == t)
        had = any(rounds[r, s] < t for r in range(P))
        if new:
            total += new * length * in_b + length * out_b + (length * out_b if had else 0)
        elif t == 1 and not had:
            total += length * out_b                                   # the identity is written
    W = (P + 63) // 64
    return total + S * W * 8 * 2 + S * 4


def test_rounds_against_a_plain_loop():
    for P, n, seg, in_b, out_b in [(5, 1000, 64, 4, 4), (70, 5000, 512, 2, 4), (16, 4096, 4096, 8, 8)]:
        S = (n + seg - 1) // seg
        rounds = inputs.arrival_rounds(9, P, S, 0.6)
        masks = inputs.cumulative_masks(rounds)
        got = bench.epoch_bytes(dict(P=P, n=n, seg=seg), masks, in_b, out_b)
        want = [brute(None, rounds, t, P, n, seg, in_b, out_b) for t in (1, 2, 3)]
        assert got == want


def test_all_arrived_closed_form_and_headline_totals():
    # everything at once: all inputs read once, the result written once
    P, n, seg = 16, 1 << 24, 65536
    S = n // seg
    assert bench.apply_bytes(None, None, P, n, seg, 4, 4, True) == P * n * 4 + n * 4 + S * 8 * 2 + S * 4
    # the headline epoch: every contribution is read exactly once over the three rounds
    rounds = inputs.arrival_rounds(bench.HEADLINE["seed_sched"], P, S, bench.HEADLINE["p_first"])
    per_round = bench.epoch_bytes(dict(P=P, n=n, seg=seg), inputs.cumulative_masks(rounds), 4, 4)
    words = 3 * (S * 8 * 2 + S * 4)
    result_traffic = sum(per_round) - words - P * n * 4
    touched = [(rounds == t).any(axis=0).sum() for t in (1, 2, 3)]           # segments written per round
    reread = [0] + [int(((rounds == t).any(axis=0) & (rounds < t).any(axis=0)).sum()) for t in (2, 3)]
    assert result_traffic == (sum(int(x) for x in touched) + sum(reread)) * seg * 4
    assert abs(per_round[0] - 818.7e6) < 3e6                                 # about 0.7 GiB of inputs + the 64 MiB result
