"""GPU parity of ec_mf_* (matrix factorisation over the stale-synchronous allreduce) against the checker."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle
from paper_2203_17063_b200 import binding as ec
from paper_2203_17063_b200 import inputs

KEYS = ("user_ptr", "user_item", "user_val", "rank_item_ptr", "item_user", "item_val")


def _setup(U, I, k, nnz, P, seg, seed, lr=0.01, lam=0.05):
    d = inputs.mf_ratings(seed, U, I, 6, nnz, P)
    pu, qi = inputs.mf_init_factors(seed, U, I, k, 0.3)
    dev = {key: torch.from_numpy(d[key]).cuda() for key in KEYS}
    gpu = ec.MatrixFactorization(dev, U, I, P, torch.from_numpy(pu).cuda(), torch.from_numpy(qi).cuda(), lr, lam, seg)
    ref = oracle.MatrixFactorization(d, pu, qi, lr, lam, seg)
    return d, gpu, ref


def _state(gpu):
    pu = torch.empty(gpu.U, gpu.k, device="cuda")
    qi = torch.empty(gpu.I, gpu.k, device="cuda")
    sse = torch.empty(1, dtype=torch.float64, device="cuda")
    seg_clock = torch.empty(gpu.S, dtype=torch.int32, device="cuda")
    notif = torch.empty(gpu.S, gpu.P, dtype=torch.int32, device="cuda")
    wait = torch.empty(gpu.S, dtype=torch.int32, device="cuda")
    gpu.get(pu, qi, sse, seg_clock, notif, wait)
    torch.cuda.synchronize()
    return (pu.cpu().numpy().astype(np.float64), qi.cpu().numpy().astype(np.float64), float(sse.item()),
            seg_clock.cpu().numpy().view(np.uint32), notif.cpu().numpy().view(np.uint32), wait.cpu().numpy().view(np.uint32))


def _rows_close(got, want, tol):
    err = np.linalg.norm(got - want, axis=1)
    return bool((err <= tol * np.linalg.norm(want, axis=1) + 1e-12).all())


@pytest.mark.parametrize("k,P,slack,U,I,nnz,seg,iters", [(32, 8, 2, 1500, 200, 30000, 16, 6), (64, 5, 1, 1500, 200, 30000, 16, 6),
                                                         (32, 1, 0, 1500, 200, 30000, 16, 6), (32, 70, 3, 1500, 200, 30000, 16, 6),
                                                         # more rows than resident warps, item segments of the bench's size
                                                         (32, 16, 1, 24000, 3000, 400000, 64, 2)])
def test_lock_step_iterations(cuda_device, k, P, slack, U, I, nnz, seg, iters):
    d, gpu, ref = _setup(U, I, k, nnz, P, seg, 21 + P)
    masks = inputs.mf_refresh_masks(31, iters, P, gpu.S, 0.5)
    for t, m in enumerate(masks):
        # both sides start the iteration from the checker's factors (rounded to fp32)
        gpu.set_factors(torch.from_numpy(ref.pu.astype(np.float32)).cuda(), torch.from_numpy(ref.qi.astype(np.float32)).cuda())
        ref.pu = ref.pu.astype(np.float32).astype(np.float64)
        ref.qi = ref.qi.astype(np.float32).astype(np.float64)
        arrived = np.zeros((P, gpu.S), dtype=bool)
        for r in range(P):
            arrived[r] = (m[:, r // 64] >> np.uint64(r % 64)) & np.uint64(1)
        gpu.iterate(torch.from_numpy(m.view(np.int64)).cuda(), slack)
        sse, seg_clock, refreshed = ref.iterate(arrived, slack)
        pu, qi, g_sse, g_clk, g_notif, g_wait = _state(gpu)
        assert np.array_equal(g_notif, ref.notif_clock) and np.array_equal(g_clk, seg_clock)     # integer state: exact
        assert (g_wait == 0).all() and (t + 1 - g_clk.astype(np.int64) <= slack).all()
        assert abs(g_sse - sse) <= 1e-5 * sse
        assert _rows_close(pu, ref.pu, 1e-4) and _rows_close(qi, ref.qi, 1e-4)
    gpu.destroy()


def test_free_running_all_fresh_error_falls_and_repeats_bit_for_bit(cuda_device):
    U, I, k, nnz, P, seg = 3000, 400, 32, 120000, 16, 25
    d, gpu, ref = _setup(U, I, k, nnz, P, seg, 5, lr=1e-3)          # small enough for the most popular item's thousands of ratings
    _, gpu2, _ = _setup(U, I, k, nnz, P, seg, 5, lr=1e-3)
    sses = []
    for t in range(12):
        gpu.iterate(None, 0)
        gpu2.iterate(None, 0)
        sse, _, _ = ref.iterate(None, 0)
        pu, qi, g_sse, *_ = _state(gpu)
        sses.append(g_sse)
        assert abs(g_sse - sse) <= 1e-4 * sse
    assert sses[-1] < 0.7 * sses[0] and all(b < a for a, b in zip(sses, sses[1:]))
    assert _rows_close(pu, ref.pu, 1e-3) and _rows_close(qi, ref.qi, 1e-3)
    pu2, qi2, sse2, *_ = _state(gpu2)
    assert np.array_equal(pu, pu2) and np.array_equal(qi, qi2) and sse2 == g_sse       # fixed order of every sum
    gpu.destroy(); gpu2.destroy()


def test_unsupported_shapes_are_rejected(cuda_device):
    d = inputs.mf_ratings(1, 64, 16, 4, 500, 2)
    dev = {key: torch.from_numpy(d[key]).cuda() for key in KEYS}
    pu = torch.zeros(64, 48, device="cuda"); qi = torch.zeros(16, 48, device="cuda")
    with pytest.raises(ec.EcError) as err:
        ec.MatrixFactorization(dev, 64, 16, 2, pu, qi, 0.01, 0.05, 4)            # k = 48
    assert err.value.code == ec.ERR_UNSUPPORTED
