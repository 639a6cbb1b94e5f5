"""GPU parity of the K-means driver against the CPU checker, through the C ABI.

Labels must equal the checker's except at near-ties (relative gap between the two
closest centroids below 1e-5), where the second-closest is also accepted;
partial sums and centroids within 1e-4 relative (row norm); counts exact."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle
from paper_2203_17063_b200 import inputs
from tests.gpu_util import check_guards, ec, guarded, to_dev, to_host


@pytest.fixture(autouse=True)
def _need_gpu(cuda_device):
    yield


def check_labels(g_labels, points, centroids, threads=8):
    c_labels, d1, d2, second = oracle.kmeans_assign(points, centroids, threads)
    diff = np.nonzero(g_labels != c_labels)[0]
    if diff.size:
        near = (d2[diff] - d1[diff]) <= 1e-5 * d2[diff]
        assert near.all(), f"{(~near).sum()} label mismatches away from near-ties"
        assert np.array_equal(g_labels[diff], second[diff]), "a mismatching label is not the second closest"
    return c_labels, diff.size


def rows_close(g, c, rel=1e-4):
    num = np.linalg.norm(g.astype(np.float64) - c.astype(np.float64), axis=-1)
    den = np.linalg.norm(c.astype(np.float64), axis=-1)
    return (num <= rel * den + 1e-30).all()


def lockstep(N, D, K, P, iters, seed, p_arrive=0.75, path=None):
    points, comp, _ = inputs.kmeans_mixture(seed, N, D, K)
    cents = inputs.kmeans_first_of_component(points, comp, K)
    masks = inputs.kmeans_masks(seed + 1000, iters, P, K, p_arrive)
    d_points = to_dev(points)
    km = ec.KMeans(d_points, K, P, to_dev(cents))
    if path is not None:
        km.set_path(path)
    lab_all, d_labels = guarded(np.zeros(N, dtype=np.int32))           # sentinels on either side of the outputs
    part_all, d_part = guarded(np.zeros(P * K * (D + 4), dtype=np.float32))
    d_part = d_part.view(P, K, D + 4)
    d_cent = torch.empty(K, D, device="cuda")
    d_red = torch.empty(K, D + 4, device="cuda")
    d_cnt = torch.empty(K, dtype=torch.int32, device="cuda")
    for t in range(iters):
        # the GPU is fed the checker's current centroids
        km.set_centroids(to_dev(cents))
        km.assign(to_dev(cents), d_labels)
        g_labels = to_host(d_labels)
        check_guards(lab_all, d_labels, "labels")
        c_labels, nmis = check_labels(g_labels, points, cents)
        # partials from the checker's labels: sums within tolerance, counts exact
        km.partials(to_dev(c_labels), d_part)
        g_part = to_host(d_part)
        check_guards(part_all, d_part.view(-1), "partials")
        c_part = oracle.kmeans_partials(points, c_labels, K, P, 8)
        assert np.array_equal(g_part[:, :, D], c_part[:, :, D])
        assert (g_part[:, :, D + 1:] == 0).all()
        assert rows_close(g_part[:, :, :D], c_part[:, :, :D])
        # whole iteration on the GPU vs the checker's iteration
        km.iterate(to_dev(masks[t]))
        km.get(d_cent, None, d_red, d_cnt)
        torch.cuda.synchronize()
        new, _, c_red, c_cnt = oracle.kmeans_iterate(points, cents, P, masks[t], 8)
        assert np.array_equal(to_host(d_cnt).view(np.uint32), c_cnt)
        if nmis == 0:
            assert np.array_equal(to_host(d_red)[:, D], c_red[:, D])
        assert rows_close(to_host(d_cent), new)
        cents = new
    km.destroy()


def test_lockstep_small():
    lockstep(N=1 << 15, D=32, K=64, P=64, iters=4, seed=1005)


@pytest.mark.parametrize("N,D,K,P", [(5000, 8, 5, 3), (4099, 16, 7, 1), (3000, 4, 3, 7), (2048, 64, 9, 2),
                                     (3001, 12, 6, 5), (2500, 128, 4, 2), (20000, 32, 200, 4),
                                     # the warp-specialised kernel with three and with two epilogue groups (96 and 128 score columns)
                                     (9000, 32, 90, 3), (7001, 16, 128, 2), (6000, 32, 33, 5)])
def test_lockstep_shapes(N, D, K, P):
    lockstep(N, D, K, P, iters=2, seed=77 + D)


@pytest.mark.parametrize("path", [2, 3])
@pytest.mark.parametrize("N,D,K,P", [(9000, 32, 90, 3), (7001, 16, 128, 2), (8000, 32, 64, 4)])
def test_lockstep_each_tensor_core_kernel_on_its_own(N, D, K, P, path):
    """The automatic choice mixes the two tensor-core kernels (one for passes that sum every point, one for the others);
    here each does every kind of pass alone: 2 = warp-specialised, 3 = register-staged."""
    lockstep(N, D, K, P, iters=3, seed=500 + K, path=path)


@pytest.mark.parametrize("path", [0, 2, 3])
@pytest.mark.parametrize("N,D,K,P", [(600011, 16, 128, 7), (500000, 32, 96, 5), (450001, 16, 33, 3), (700001, 32, 17, 9),
                                     (520000, 16, 90, 64)])
def test_lockstep_at_a_size_where_every_block_takes_many_tiles(N, D, K, P, path):
    """The shapes with three and two epilogue groups, odd and even numbers of search accumulators and of stages, at sizes
    where a thread block works through dozens of tiles and several runs (the small cases above leave most blocks with one
    tile or none)."""
    lockstep(N, D, K, P, iters=2, seed=900 + K + D, path=path)


@pytest.mark.parametrize("N,D,K,P", [(300001, 64, 9, 4), (400003, 8, 5, 3), (250001, 128, 4, 2), (200003, 12, 6, 5),
                                     (350001, 4, 3, 7), (300007, 32, 300, 6)])
def test_lockstep_at_that_size_on_the_fp32_kernels(N, D, K, P):
    """Shapes outside the tensor-core kernels (other D, more than 256 centroids), many tiles per block."""
    lockstep(N, D, K, P, iters=2, seed=700 + K + D)


def test_exact_ties_take_the_lowest_index():
    pts = np.zeros((300, 4), dtype=np.float32)
    cents = np.array([[1, 0, 0, 0], [0, 1, 0, 0], [-1, 0, 0, 0], [0, 0, 0, 0.5]], dtype=np.float32)
    cents = np.concatenate([cents[:3], cents[:3], cents[3:]])          # duplicates: exact ties
    km = ec.KMeans(to_dev(pts), cents.shape[0], 1, to_dev(cents))
    lab = torch.empty(300, dtype=torch.int32, device="cuda")
    km.assign(to_dev(cents), lab)
    assert (to_host(lab) == 6).all()
    cents[6] = [0, 0, 0, 1]                                             # now seven centroids at distance 1
    km.assign(to_dev(cents), lab)
    assert (to_host(lab) == 0).all()
    km.destroy()


def test_free_running_config5_reduced():
    """Both sides run their own trajectory for 20 iterations from the one-centroid-per-component start."""
    N, D, K, P, iters = 1 << 17, 32, 64, 64, 20
    points, comp, _ = inputs.kmeans_mixture(1005, N, D, K)
    cents0 = inputs.kmeans_first_of_component(points, comp, K)
    masks = inputs.kmeans_masks(2005, iters, P, K, 0.75)
    km = ec.KMeans(to_dev(points), K, P, to_dev(cents0))
    d_masks = [to_dev(m) for m in masks]
    for t in range(iters):
        km.iterate(d_masks[t])
    d_cent = torch.empty(K, D, device="cuda")
    d_labels = torch.empty(N, dtype=torch.int32, device="cuda")
    km.get(d_cent, d_labels)
    torch.cuda.synchronize()
    cents = cents0
    for t in range(iters):
        prev = cents
        cents, labels, _, _ = oracle.kmeans_iterate(points, cents, P, masks[t], 8)
    assert rows_close(to_host(d_cent), cents)
    # labels of the last iteration were taken against the centroids before the last update
    check_labels(to_host(d_labels), points, prev)
    km.destroy()


def test_full_size_config5_one_iteration_sampled():
    """N = 2^22 in the launch configuration the benchmark times; the checker labels a sample of points one by one."""
    N, D, K, P = 1 << 22, 32, 64, 64
    points, comp, _ = inputs.kmeans_mixture(1005, N, D, K)
    cents = inputs.kmeans_first_of_component(points, comp, K)
    mask = inputs.kmeans_masks(2005, 1, P, K, 0.75)[0]
    km = ec.KMeans(to_dev(points), K, P, to_dev(cents))
    km.iterate(to_dev(mask))
    d_cent = torch.empty(K, D, device="cuda")
    d_labels = torch.empty(N, dtype=torch.int32, device="cuda")
    d_red = torch.empty(K, D + 4, device="cuda")
    d_cnt = torch.empty(K, dtype=torch.int32, device="cuda")
    km.get(d_cent, d_labels, d_red, d_cnt)
    torch.cuda.synchronize()
    g_labels = to_host(d_labels)
    idx = np.random.default_rng(0).choice(N, size=1 << 16, replace=False)
    idx.sort()
    c_lab, d1, d2, second = oracle.kmeans_assign(points[idx], cents, 8)
    diff = np.nonzero(g_labels[idx] != c_lab)[0]
    assert ((d2[diff] - d1[diff]) <= 1e-5 * d2[diff]).all()
    # properties that hold at any size: counts of arrived cells add up, centroids are means of labelled points
    arrived = ((mask[:, 0][None, :] >> np.arange(P, dtype=np.uint64)[:, None]) & np.uint64(1)).astype(bool)   # [P][K]
    assert np.array_equal(to_host(d_cnt).view(np.uint32), arrived.sum(0).astype(np.uint32))
    shard = N // P
    onehot_counts = np.stack([np.bincount(g_labels[r * shard:(r + 1) * shard], minlength=K) for r in range(P)])
    assert np.array_equal(to_host(d_red)[:, D], (onehot_counts * arrived).sum(0).astype(np.float32))
    k = int(np.argmax(arrived.sum(0)))
    sel = np.zeros(N, dtype=bool)
    for r in range(P):
        if arrived[r, k]:
            sel[r * shard:(r + 1) * shard] = g_labels[r * shard:(r + 1) * shard] == k
    mean = points[sel].astype(np.float64).mean(0)
    assert np.linalg.norm(to_host(d_cent)[k] - mean) <= 1e-4 * np.linalg.norm(mean)
    km.destroy()


def test_iteration_with_two_rounds_matches_checker():
    """Late rows of round 1 are folded in by round 2 of the same iteration, before the centroid update."""
    N, D, K, P = 1 << 15, 32, 64, 64
    points, comp, _ = inputs.kmeans_mixture(1005, N, D, K)
    cents = inputs.kmeans_first_of_component(points, comp, K)
    rounds = inputs.arrival_rounds(77, P, K, 0.75, last_round=2)             # [P][K] -> 1 or 2
    masks = inputs.cumulative_masks(rounds)
    km = ec.KMeans(to_dev(points), K, P, to_dev(cents))
    km.iterate_rounds([to_dev(m) for m in masks])
    d_cent = torch.empty(K, D, device="cuda")
    d_red = torch.empty(K, D + 4, device="cuda")
    d_cnt = torch.empty(K, dtype=torch.int32, device="cuda")
    km.get(d_cent, None, d_red, d_cnt)
    torch.cuda.synchronize()
    new, labels, c_red, c_cnt = oracle.kmeans_iterate(points, cents, P, masks, 8)
    assert (c_cnt == P).all() and np.array_equal(to_host(d_cnt).view(np.uint32), c_cnt)
    assert np.array_equal(to_host(d_red)[:, D], c_red[:, D])
    assert rows_close(to_host(d_cent), new)
    # with both rounds every point counts: the centroids are the plain cluster means
    means = np.stack([points[labels == k].astype(np.float64).mean(0) for k in range(K)])
    assert rows_close(to_host(d_cent), means.astype(np.float32))
    km.destroy()


@pytest.mark.parametrize("N,D,K,P,iters", [(30000, 32, 16, 8, 40), (20011, 16, 200, 5, 8), (25000, 32, 64, 64, 8),
                                           (26000, 32, 100, 4, 8), (24001, 16, 90, 3, 8)])
def test_running_sums_follow_label_changes_over_many_iterations(N, D, K, P, iters):
    """The tensor-core path sums only what changed since the previous iteration (+x into the cluster a point joins,
    -x out of the one it leaves) and sums everything afresh every 32nd iteration.  With overlapping clusters and
    centroids that are pushed around before every iteration many points change hands each time; after each of 40
    iterations the reduced sums and counts must still be those of the labels (counts exactly)."""
    points, comp, _ = inputs.kmeans_mixture(77, N, D, K, sigma=6.0)          # heavily overlapping components
    cents = inputs.kmeans_first_of_component(points, comp, K)
    rng = np.random.default_rng(78)
    km = ec.KMeans(to_dev(points), K, P, to_dev(cents))
    full = ec.KMeans(to_dev(points), K, P, to_dev(cents))
    full.set_refresh(1)                                                         # sums all points in every iteration
    d_labels = torch.empty(N, dtype=torch.int32, device="cuda")
    d_red = torch.empty(K, D + 4, device="cuda")
    d_red_full = torch.empty(K, D + 4, device="cuda")
    prev = None
    moved = 0
    for t in range(iters):
        cents = (cents + rng.normal(0.0, 0.8, size=cents.shape)).astype(np.float32)
        km.set_centroids(to_dev(cents))
        km.iterate(None)
        km.get(labels=d_labels, reduced=d_red)
        full.set_centroids(to_dev(cents))
        full.iterate(None)
        full.get(reduced=d_red_full)
        torch.cuda.synchronize()
        assert torch.equal(d_red[:, D], d_red_full[:, D])                       # counts: running = summed afresh
        assert rows_close(to_host(d_red)[:, :D], to_host(d_red_full)[:, :D], rel=1e-5)
        g_labels = to_host(d_labels)
        check_labels(g_labels, points, cents)
        if prev is not None:
            moved += int((g_labels != prev).sum())
        prev = g_labels.copy()
        want = oracle.kmeans_partials(points, g_labels, K, P, 4).astype(np.float64).sum(axis=0)      # [K][D+4]
        got = to_host(d_red)
        assert np.array_equal(got[:, D], want[:, D].astype(np.float32)), f"iteration {t}: counts"
        assert rows_close(got[:, :D], want[:, :D]), f"iteration {t}: sums"
    assert moved > (iters // 2) * N // 10                                         # the test did exercise the changes
    km.destroy()
    full.destroy()


@pytest.mark.parametrize("N,D,K,P", [(40000 + 77, 32, 16, 5),
                                     # every block takes many tiles and several runs; four, three and two epilogue groups
                                     (900001, 32, 64, 64), (700011, 32, 90, 7), (600013, 16, 128, 6)])
def test_distance_bounds_change_nothing_but_the_time(N, D, K, P):
    """The same iterations with and without the distance bounds: labels, counts and centroids must be the same,
    whether tiles are skipped (separated clusters), searched again (two clusters that overlap and keep
    exchanging points) or the centroids are replaced from outside (two of them swapped: every bound is void)."""
    iters = 12
    rng = np.random.default_rng(31)
    centres = rng.uniform(-10, 10, size=(K, D)).astype(np.float32)
    centres[1] = centres[0] + 0.3                                       # clusters 0 and 1 overlap almost entirely
    comp = rng.integers(0, K, size=N)
    points = (centres[comp] + rng.standard_normal((N, D))).astype(np.float32)
    init = (centres + 0.5 * rng.standard_normal((K, D))).astype(np.float32)
    masks = [to_dev(np.ascontiguousarray(m).view(np.int64)) for m in inputs.kmeans_masks(77, iters, P, K, 0.8)]
    d_points = to_dev(points)
    out = []
    for use_bounds in (True, False):
        km = ec.KMeans(d_points, K, P, to_dev(init))
        km.set_bounds(use_bounds)
        trace = []
        for t in range(iters):
            if t == 7:                                                  # swap two centroids behind the driver's back
                c = torch.empty(K, D, device="cuda")
                km.get(c)
                c[[2, 3]] = c[[3, 2]]
                km.set_centroids(c.contiguous())
            km.iterate(masks[t])
            c = torch.empty(K, D, device="cuda")
            lab = torch.empty(N, dtype=torch.int32, device="cuda")
            red = torch.empty(K, D + 4, device="cuda")
            km.get(c, lab, red)
            trace.append((to_host(c), to_host(lab), to_host(red)))
        assert km.tc_status() == 0
        km.destroy()
        out.append(trace)
    changed = 0
    for t in range(iters):
        (c1, l1, r1), (c0, l0, r0) = out[0][t], out[1][t]
        assert np.array_equal(l1, l0), f"labels differ in iteration {t}"
        # the same tiles issue the same sums in the same order either way: not a bit may differ
        assert np.array_equal(r1, r0), f"reduced sums differ in iteration {t}"
        assert np.array_equal(c1, c0), f"centroids differ in iteration {t}"
        if t:
            changed += int((out[1][t][1] != out[1][t - 1][1]).sum())
    assert changed > 100                                                # the overlapping clusters did keep moving points
    # and the labels are the checker's for the centroids the last iteration started from
    c_prev = out[0][iters - 2][0]
    check_labels(out[0][iters - 1][1], points, c_prev)


def test_many_runs_per_block_with_churn():
    """More runs than resident blocks, so that a block works through several runs, on clusters that keep exchanging
    points: with the bounds, without them, and with every iteration summing all points afresh the labels and counts
    must agree, the first two to the bit, the running sums with the fresh ones to rounding."""
    N, D, K, P, iters = (1 << 21) + 1234, 32, 64, 64, 6
    g = torch.Generator(device="cuda").manual_seed(99)
    centres = (torch.rand(K, D, device="cuda", generator=g) - 0.5) * 4.0          # sigma 1 around centres 4 wide: heavy overlap
    comp = torch.randint(0, K, (N,), device="cuda", generator=g)
    points = (centres[comp] + torch.randn(N, D, device="cuda", generator=g)).contiguous()
    init = points[torch.randperm(N, device="cuda", generator=g)[:K]].contiguous()
    masks = [to_dev(np.ascontiguousarray(m).view(np.int64)) for m in inputs.kmeans_masks(123, iters, P, K, 0.8)]
    traces = []
    for mode in ("bounds", "no bounds", "fresh sums"):
        km = ec.KMeans(points, K, P, init)
        km.set_bounds(mode == "bounds")
        if mode == "fresh sums":
            km.set_refresh(1)
        tr = []
        for t in range(iters):
            km.iterate(masks[t])
            c = torch.empty(K, D, device="cuda")
            lab = torch.empty(N, dtype=torch.int32, device="cuda")
            red = torch.empty(K, D + 4, device="cuda")
            km.get(c, lab, red)
            tr.append((c.clone(), lab.clone(), red.clone()))
        assert km.tc_status() == 0
        km.destroy()
        traces.append(tr)
    moved = 0
    for t in range(iters):
        (c1, l1, r1), (c0, l0, r0), (cf, lf, rf) = traces[0][t], traces[1][t], traces[2][t]
        assert torch.equal(l1, l0) and torch.equal(r1, r0) and torch.equal(c1, c0), f"bounds on / off differ in iteration {t}"
        # fresh sums: the centroids of the iteration before differ by rounding, so a few near-tie labels may differ
        same = (l1 == lf).float().mean().item()
        assert same > 0.9999, f"labels of running and fresh sums: {same}"
        err = (r1[:, :D].double() - rf[:, :D].double()).norm(dim=1) / rf[:, :D].double().norm(dim=1).clamp_min(1e-30)
        assert float(err.max()) < 2e-4, f"running sums drifted from fresh ones in iteration {t}: {float(err.max())}"
        if t:
            moved += int((l0 != traces[1][t - 1][1]).sum())
    assert moved > 10000


def test_two_contexts_on_two_streams_do_not_disturb_each_other():
    """Contexts are independent (ec.h): two of them iterate at the same time on two streams, on different data and
    shapes (one per tensor-core kernel layout), and each ends where it ends when it runs alone."""
    shapes = [(300001, 32, 64, 16, 11), (260003, 16, 128, 4, 12)]
    data = []
    for N, D, K, P, seed in shapes:
        points, comp, _ = inputs.kmeans_mixture(seed, N, D, K, sigma=1.0, box=2.5)      # overlapping: labels keep moving
        init = points[np.random.default_rng(seed).choice(N, K, replace=False)].copy()
        masks = [to_dev(np.ascontiguousarray(m).view(np.int64)) for m in inputs.kmeans_masks(seed + 1, 6, P, K, 0.8)]
        data.append((to_dev(points), to_dev(init), masks, N, D, K, P))

    def run(order):
        kms = [ec.KMeans(d[0], d[5], d[6], d[1]) for d in data]
        streams = [torch.cuda.Stream(), torch.cuda.Stream()] if order == "together" else [None, None]
        torch.cuda.synchronize()
        for t in range(6):
            for i, km in enumerate(kms):
                km.iterate(data[i][2][t], stream=streams[i])
            if order == "alone":
                torch.cuda.synchronize()
        torch.cuda.synchronize()
        out = []
        for i, km in enumerate(kms):
            N, D, K = data[i][3], data[i][4], data[i][5]
            c = torch.empty(K, D, device="cuda")
            lab = torch.empty(N, dtype=torch.int32, device="cuda")
            km.get(c, lab)
            torch.cuda.synchronize()
            assert km.tc_status() == 0
            out.append((to_host(c), to_host(lab)))
            km.destroy()
        return out

    alone, together = run("alone"), run("together")
    for (c0, l0), (c1, l1) in zip(alone, together):
        assert np.array_equal(l0, l1) and np.array_equal(c0, c1)
