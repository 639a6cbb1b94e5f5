"""Seeded random shapes through ec_allreduce_apply against the CPU checker: every dtype, operator and
order, rank counts around the 64-rank word and table boundaries, segment lengths around the limits of
the short-segment and the 128-bit paths, misaligned buffers, odd tile shapes; bit for bit after every round."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from paper_2203_17063_b200 import inputs
from tests.gpu_util import ec, run_schedule

KINDS = {ec.F32: "normal_f32", ec.BF16: "normal_bf16", ec.I64: "int64_full"}
PER_VEC = {ec.F32: 4, ec.BF16: 8, ec.I64: 2, ec.F64: 2}


@pytest.mark.parametrize("seed", [11, 12, 13, 14])
def test_random_shapes(cuda_device, seed):
    rng = np.random.default_rng(seed)
    for it in range(30):
        dtype = int(rng.choice([ec.F32, ec.BF16, ec.I64, ec.F64]))
        P = int(rng.choice([1, 2, 3, 4, 5, 6, 8, 15, 16, 17, 31, 33, 63, 64, 65, 66, 100, 129, 257]))
        per_vec = PER_VEC[dtype]
        pick = int(rng.integers(0, 4))
        if pick == 0:
            seg = int(rng.integers(1, 40)) * per_vec                      # short, whole vectors
        elif pick == 1:
            seg = int(rng.integers(1, 300))                                # anything, maybe no whole vector
        elif pick == 2:
            seg = int(rng.choice([32, 64, 128, 256])) * per_vec            # around the short-segment limit
        else:
            seg = int(rng.integers(1000, 20000))
        S = int(rng.integers(1, 12))
        n = max(1, (S - 1) * seg + int(rng.integers(1, seg + 1)))
        S = (n + seg - 1) // seg
        op = int(rng.choice([ec.SUM, ec.MAX, ec.MIN])) if dtype != ec.BF16 else ec.SUM
        order = ec.ORDER_FIXED
        if op == ec.SUM and dtype != ec.I64 and rng.random() < 0.25:
            order = ec.ORDER_PAIRWISE
        if dtype == ec.F64:
            bufs = [b.astype(np.float64) * (1 + 2.0 ** -29) for b in inputs.rank_buffers("normal_f32", seed * 1000 + it, P, n)]
        else:
            bufs = inputs.rank_buffers(KINDS[dtype], seed * 1000 + it, P, n)
        masks = inputs.cumulative_masks(inputs.arrival_rounds(seed * 2000 + it, P, S, float(rng.choice([0.2, 0.5, 0.9]))))
        if rng.random() < 0.3:
            masks = masks[:2] + [None]
        threads = int(rng.choice([0, 64, 128, 256]))
        tile = None if threads == 0 else (threads, int(rng.choice([16, 100, 1000, 4096])))
        try:
            run_schedule(P, n, seg, dtype, op, bufs, masks, order=order, offset_elems=int(rng.choice([0, 0, 0, 1, 3])),
                         result_offset=int(rng.choice([0, 0, 1])), tile=tile)
        except AssertionError as e:
            raise AssertionError(f"case {it}: dtype={dtype} P={P} n={n} seg={seg} op={op} order={order} tile={tile}: {e}")
