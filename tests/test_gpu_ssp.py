"""GPU parity of ec_allreduce_ssp_apply (Algorithm 1) against the CPU checker: bit-exact results,
counts, reduction clocks and wait counts, through the C ABI."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle
from paper_2203_17063_b200 import inputs
from tests.gpu_util import bits, ec, sentinel, to_dev, to_host


@pytest.fixture(autouse=True)
def _need_gpu(cuda_device):
    yield


def run_ssp(P, n, seg, dtype, op, bufs, clocks, clock, slack, tile=None, order=ec.ORDER_FIXED):
    S = (n + seg - 1) // seg
    ar = ec.Allreduce(P, n, dtype, op, seg, order)
    if tile:
        ar.set_tile(*tile)
    d_bufs = [to_dev(b) for b in bufs]
    d_res = to_dev(sentinel(np.float32 if dtype in (ec.F32, ec.BF16) else (np.int64 if dtype == ec.I64 else np.float64), n))
    d_cnt = torch.full((S,), -1, dtype=torch.int32, device="cuda")
    d_clk = torch.full((S,), -1, dtype=torch.int32, device="cuda")
    d_wait = torch.full((S,), -1, dtype=torch.int32, device="cuda")
    ar.ssp_apply(d_bufs, to_dev(np.ascontiguousarray(clocks, dtype=np.uint32)), clock, slack, d_res, d_cnt, d_clk, d_wait)
    torch.cuda.synchronize()
    res, cnt, seg_clock, wait = oracle.allreduce_ssp(bufs, dtype, op, seg, clocks, clock, slack)
    g = to_host(d_res)
    assert np.array_equal(bits(g), bits(res))
    assert np.array_equal(d_cnt.cpu().numpy().view(np.uint32), cnt)
    assert np.array_equal(d_clk.cpu().numpy().view(np.uint32), seg_clock)
    assert np.array_equal(d_wait.cpu().numpy().view(np.uint32), wait)
    ar.destroy()
    return g, cnt, seg_clock, wait


def test_paper_examples_on_the_gpu():
    # iteration 5, slack 1: clocks 5 and 4 are used, 3 is not; the reduction carries clock 4
    bufs = [np.full(8, 10.0 ** r, dtype=np.float32) for r in range(3)]
    g, cnt, clk, wait = run_ssp(3, 8, 8, ec.F32, ec.SUM, bufs, np.array([[5, 4, 3]]), 5, 1)
    assert (g == 11.0).all() and cnt[0] == 2 and clk[0] == 4 and wait[0] == 1
    # clock 2 reduced with clock 3 is clock 2
    g, cnt, clk, wait = run_ssp(2, 8, 8, ec.F32, ec.SUM, bufs[:2], np.array([[2, 3]]), 3, 1)
    assert clk[0] == 2 and wait[0] == 0


@pytest.mark.parametrize("P", [1, 5, 32, 33, 64, 65, 200, 1024])
def test_rank_counts(P):
    n, seg = 3000, 256
    S = (n + seg - 1) // seg
    rng = np.random.default_rng(P)
    bufs = inputs.rank_buffers("normal_f32", 40 + P, P, n)
    clocks = rng.integers(0, 20, size=(S, P)).astype(np.uint32)
    clocks[0] = 0                      # nothing received for segment 0
    clocks[1] = 19                     # everything fresh for segment 1
    run_ssp(P, n, seg, ec.F32, ec.SUM, bufs, clocks, 19, 4)
    run_ssp(P, n, seg, ec.F32, ec.SUM, bufs, clocks, 19, 0)          # synchronous
    run_ssp(P, n, seg, ec.F32, ec.SUM, bufs, clocks, 19, 100)        # slack beyond the clock: all but the never-received


@pytest.mark.parametrize("dtype,kind", [(ec.F32, "normal_f32"), (ec.BF16, "normal_bf16"), (ec.I64, "int64_full")])
@pytest.mark.parametrize("op", [ec.SUM, ec.MAX])
def test_dtypes_ops_and_ragged_shapes(dtype, kind, op):
    P, n, seg = 9, 10007, 1000
    S = (n + seg - 1) // seg
    bufs = inputs.rank_buffers(kind, 77, P, n)
    clocks = np.random.default_rng(5).integers(0, 9, size=(S, P)).astype(np.uint32)
    run_ssp(P, n, seg, dtype, op, bufs, clocks, 8, 2)
    run_ssp(P, n, seg, dtype, op, bufs, clocks, 8, 2, tile=(64, 96))


def test_config2_shape_with_clocks_and_state_is_untouched():
    """P = 16, 2^22 elements: clocks drawn so that about 70 % are fresh, 15 % one behind, 15 % two behind."""
    P, n, seg = 16, 1 << 22, 65536
    S = n // seg
    bufs = inputs.rank_buffers("normal_f32", 1002, P, n)
    rounds = inputs.arrival_rounds(2002, P, S, 0.7)                   # 1, 2, 3
    clocks = (10 - (rounds.T - 1)).astype(np.uint32)                  # [S][P]: 10, 9 or 8
    for slack in (0, 1, 2):
        g, cnt, clk, wait = run_ssp(P, n, seg, ec.F32, ec.SUM, bufs, clocks, 10, slack)
        assert ((cnt + wait) == P).all()
    assert (cnt == P).all() and (clk == clocks.min(1)).all()
    # a stale-synchronous apply between two ordinary applies does not disturb the epoch's state
    ar = ec.Allreduce(P, n, ec.F32, ec.SUM, seg)
    masks = inputs.cumulative_masks(rounds)
    d_bufs = [to_dev(b) for b in bufs]
    d_res = torch.empty(n, device="cuda")
    d_other = torch.empty(n, device="cuda")
    d_cnt = torch.empty(S, dtype=torch.int32, device="cuda")
    ar.apply(d_bufs, to_dev(masks[0]), d_res, d_cnt)
    ar.ssp_apply(d_bufs, to_dev(clocks), 10, 1, d_other)
    ar.apply(d_bufs, to_dev(masks[1]), d_res, d_cnt)
    ar.apply(d_bufs, to_dev(masks[2]), d_res, d_cnt)
    torch.cuda.synchronize()
    ref = oracle.Allreduce(P, n, oracle.F32, oracle.SUM, seg)
    c = np.empty(n, dtype=np.float32)
    for m in masks:
        ref.apply(bufs, m, c, None, threads=8)
    assert np.array_equal(bits(to_host(d_res)), bits(c))
    ar.destroy()


@pytest.mark.parametrize("order,P,n,seg", [(ec.ORDER_PAIRWISE, 8, 5000, 500), (ec.ORDER_PAIRWISE, 16, 1 << 16, 4096),
                                           (ec.ORDER_PAIRWISE, 100, 3000, 256), (ec.ORDER_RING, 16, 1 << 16, 1024),
                                           (ec.ORDER_RING, 6, 6 * 700, 100)])
def test_stale_synchronous_apply_in_hypercube_and_ring_order(order, P, n, seg):
    """Algorithm 1 is a hypercube allreduce: with the pairwise order the accepted contributions are summed as the
    recursive-doubling tree sums them (an excluded process contributes the identity).  The checker composes its
    own pieces: acceptance by clock gives a mask, the mask goes through its order-aware apply."""
    S = (n + seg - 1) // seg
    bufs = inputs.rank_buffers("normal_f32", 300 + P, P, n)
    clocks = np.random.default_rng(P).integers(0, 8, size=(S, P)).astype(np.uint32)
    clock, slack = 7, 2
    accepted = (clocks >= clock - slack) & (clocks > 0)                       # [S][P]
    ref = oracle.Allreduce(P, n, oracle.F32, oracle.SUM, seg)
    want = np.full(n, np.nan, dtype=np.float32)
    want_cnt = np.zeros(S, dtype=np.uint32)
    ref.apply(bufs, inputs.pack_mask(accepted.T.copy()), want, want_cnt, order=order)
    ar = ec.Allreduce(P, n, ec.F32, ec.SUM, seg, order)
    d_res = torch.full((n,), float("nan"), device="cuda")
    d_cnt = torch.zeros(S, dtype=torch.int32, device="cuda")
    d_clk = torch.zeros(S, dtype=torch.int32, device="cuda")
    d_wait = torch.zeros(S, dtype=torch.int32, device="cuda")
    ar.ssp_apply([to_dev(b) for b in bufs], to_dev(clocks), clock, slack, d_res, d_cnt, d_clk, d_wait)
    torch.cuda.synchronize()
    assert np.array_equal(bits(to_host(d_res)), bits(want))
    assert np.array_equal(d_cnt.cpu().numpy().view(np.uint32), want_cnt)
    masked = np.where(accepted, clocks, np.uint32(0xFFFFFFFF)).min(axis=1)
    assert np.array_equal(d_clk.cpu().numpy().view(np.uint32), np.where(accepted.any(axis=1), masked, 0).astype(np.uint32))
    assert np.array_equal(d_wait.cpu().numpy().view(np.uint32), (P - accepted.sum(axis=1)).astype(np.uint32))
    ar.destroy()
