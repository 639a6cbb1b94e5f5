"""K-means at the sizes the benchmark times, against the CPU checker, through the C ABI.

The library's default path (running sums after the first iteration, distance bounds that skip tiles) is compared
with the checker here, not with another mode of the library:

* the 20 free-running iterations of the fifth workload at its stated size (N = 2^22, D = 32, K = 64, P = 64, one
  centroid per mixture component to start from, arrival probability 0.75): every label by the near-tie rule, every
  centroid row to 1e-4;
* an overlapping mixture at N > 2^21, where one resident block works through several runs and labels keep moving:
  once with the checker's centroids fed to the library before every iteration (running sums, every tile searched),
  once with the library on its own trajectory (running sums and tiles skipped behind the distance bounds) and the
  checker re-doing each iteration from the centroids the library started it with.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle
from paper_2203_17063_b200 import inputs
from tests.gpu_util import ec, to_dev, to_host


@pytest.fixture(autouse=True)
def _need_gpu(cuda_device):
    yield


THREADS = max(1, oracle.max_threads())


def check_labels(g_labels, points, centroids):
    """Near-tie rule: a label may differ from the checker's only where the two closest centroids are within a relative
    gap of 1e-5, and then it must be the checker's second closest.  Returns the number of such points."""
    c_labels, d1, d2, second = oracle.kmeans_assign(points, centroids, THREADS)
    diff = np.nonzero(g_labels != c_labels)[0]
    if diff.size:
        near = (d2[diff] - d1[diff]) <= 1e-5 * d2[diff]
        assert near.all(), f"{(~near).sum()} label mismatches away from near-ties"
        assert np.array_equal(g_labels[diff], second[diff]), "a mismatching label is not the second closest"
    return int(diff.size)


def rows_close(g, c, rel=1e-4):
    num = np.linalg.norm(g.astype(np.float64) - c.astype(np.float64), axis=-1)
    den = np.linalg.norm(c.astype(np.float64), axis=-1)
    return bool((num <= rel * den + 1e-30).all())


def checker_combine(points, labels, centroids, P, mask):
    """Partial sums of the given labels, one allreduce epoch with this iteration's notifications, centroid update:
    the checker's steps after the assignment.  Returns (new centroids, reduced [K][D+4], contributor counts)."""
    K, D = centroids.shape
    partials = oracle.kmeans_partials(points, labels, K, P, THREADS)
    n = K * (D + 4)
    ar = oracle.Allreduce(P, n, oracle.F32, oracle.SUM, D + 4)
    reduced = np.empty(n, dtype=np.float32)
    count = np.empty(K, dtype=np.uint32)
    ar.apply([partials[r].reshape(-1) for r in range(P)], mask, reduced, count)
    reduced = reduced.reshape(K, D + 4)
    return oracle.kmeans_update(reduced, centroids), reduced, count


def test_config5_full_size_free_running_20_iterations():
    N, D, K, P, iters = 1 << 22, 32, 64, 64, 20
    points, comp, _ = inputs.kmeans_mixture(1005, N, D, K)
    cents0 = inputs.kmeans_first_of_component(points, comp, K)
    masks = inputs.kmeans_masks(2005, iters, P, K, 0.75)
    km = ec.KMeans(to_dev(points), K, P, to_dev(cents0))          # the default path: what the benchmark times
    d_masks = [to_dev(m) for m in masks]
    for t in range(iters):
        km.iterate(d_masks[t])
    d_cent = torch.empty(K, D, device="cuda")
    d_labels = torch.empty(N, dtype=torch.int32, device="cuda")
    d_red = torch.empty(K, D + 4, device="cuda")
    d_cnt = torch.empty(K, dtype=torch.int32, device="cuda")
    km.get(d_cent, d_labels, d_red, d_cnt)
    torch.cuda.synchronize()
    assert km.tc_status() == 0
    cents = cents0
    for t in range(iters):
        prev = cents
        cents, c_labels, c_red, c_cnt = oracle.kmeans_iterate(points, cents, P, masks[t], THREADS)
    assert rows_close(to_host(d_cent), cents), "centroids after 20 iterations"
    # the labels of the last iteration were taken against the centroids before the last update
    g_labels = to_host(d_labels)
    nmis = check_labels(g_labels, points, prev)
    assert np.array_equal(to_host(d_cnt).view(np.uint32), c_cnt)
    if nmis == 0:
        assert np.array_equal(to_host(d_red)[:, D], c_red[:, D]), "point counts of the last iteration"
        assert rows_close(to_host(d_red)[:, :D], c_red[:, :D]), "running sums after 20 iterations"
    km.destroy()


def blocky_mixture(seed, N, D, K):
    """Points in blocks of 4096: even blocks from well separated components (their tiles settle and are skipped behind
    the distance bounds), odd blocks from components that overlap heavily (their points keep changing hands)."""
    sep, _, _ = inputs.kmeans_mixture(seed, N, D, K // 2, sigma=1.0, box=10.0)
    mix, _, _ = inputs.kmeans_mixture(seed + 1, N, D, K - K // 2, sigma=1.0, box=1.5)
    mix += np.float32(25.0)                                    # away from the separated half
    block = (np.arange(N) // 4096) % 2 == 1
    points = np.where(block[:, None], mix, sep).astype(np.float32)
    rng = np.random.default_rng(seed + 2)
    init = np.concatenate([sep[rng.choice(N, K // 2, replace=False)], mix[rng.choice(N, K - K // 2, replace=False)]])
    return np.ascontiguousarray(points), np.ascontiguousarray(init.astype(np.float32))


@pytest.mark.parametrize("N,K,D", [((1 << 21) + 1234, 64, 32),    # four epilogue groups, a sums slot each
                                   ((1 << 20) + 777, 90, 32),     # 96 score columns: three groups, three search accumulators
                                   ((1 << 20) + 555, 128, 16),    # 128 score columns: two groups, two accumulators
                                   ((1 << 20) + 333, 24, 16),     # 32 score columns, 64-byte rows
                                   ((1 << 19) + 111, 200, 32)])   # beyond the warp-specialised kernel: the register-staged one alone
@pytest.mark.parametrize("fed_by", ["checker", "library"])
def test_many_runs_per_block_with_churn_against_the_checker(fed_by, N, K, D):
    P, iters = 64, 5
    points, init = blocky_mixture(4242, N, D, K)
    masks = inputs.kmeans_masks(4243, iters, P, K, 0.8)
    km = ec.KMeans(to_dev(points), K, P, to_dev(init))
    d_cent = torch.empty(K, D, device="cuda")
    d_labels = torch.empty(N, dtype=torch.int32, device="cuda")
    d_red = torch.empty(K, D + 4, device="cuda")
    d_cnt = torch.empty(K, dtype=torch.int32, device="cuda")
    cents = init
    prev_labels = None
    moved = 0
    for t in range(iters):
        if fed_by == "checker" and t > 0:
            km.set_centroids(to_dev(cents))                     # voids the bounds: running sums, every tile searched
        km.iterate(to_dev(masks[t]))
        km.get(d_cent, d_labels, d_red, d_cnt)
        torch.cuda.synchronize()
        g_labels = to_host(d_labels)
        check_labels(g_labels, points, cents)
        # sums, counts and centroids: the checker's steps on the labels the library took (they may differ from the
        # checker's own at near-ties, which the rule above allows)
        new, c_red, c_cnt = checker_combine(points, g_labels, cents, P, masks[t])
        assert np.array_equal(to_host(d_cnt).view(np.uint32), c_cnt), f"iteration {t}: contributor counts"
        assert np.array_equal(to_host(d_red)[:, D], c_red[:, D]), f"iteration {t}: point counts"
        assert rows_close(to_host(d_red)[:, :D], c_red[:, :D]), f"iteration {t}: sums"
        assert rows_close(to_host(d_cent), new), f"iteration {t}: centroids"
        if prev_labels is not None:
            moved += int((g_labels != prev_labels).sum())
        prev_labels = g_labels
        cents = new if fed_by == "checker" else to_host(d_cent)
    assert km.tc_status() == 0
    assert moved > 5000                                         # labels did keep moving
    km.destroy()
