"""Pins for the CPU checker's K-means: a scikit-learn Lloyd step (library special
case with one rank and every contribution present), the monotone inertia of Lloyd's
iteration, and bookkeeping identities of the partial sums."""
import numpy as np
import pytest

import oracle
from paper_2203_17063_b200 import inputs


def small_problem(N=4096, D=8, K=6, seed=21):
    pts, comp, _ = inputs.kmeans_mixture(seed, N, D, K)
    init = inputs.kmeans_first_of_component(pts, comp, K)
    return pts, comp, init


def test_assign_matches_numpy_argmin():
    pts, _, init = small_problem()
    labels, best, second, second_label = oracle.kmeans_assign(pts, init)
    d2 = ((pts.astype(np.float64)[:, None, :] - init.astype(np.float64)[None, :, :]) ** 2).sum(-1)
    assert np.array_equal(labels, d2.argmin(1))
    srt = np.sort(d2, axis=1)
    assert np.allclose(best, srt[:, 0], rtol=1e-13) and np.allclose(second, srt[:, 1], rtol=1e-13)
    assert np.array_equal(second_label, np.argsort(d2, axis=1, kind="stable")[:, 1])


def test_exact_tie_goes_to_lowest_index():
    pts = np.array([[0.0, 0.0], [1.0, 1.0]], dtype=np.float32)
    cents = np.array([[1.0, 0.0], [0.0, 1.0], [-1.0, 0.0]], dtype=np.float32)   # all at distance 1 from the origin
    labels, best, second, second_label = oracle.kmeans_assign(pts, cents)
    assert labels.tolist() == [0, 0] and best[0] == 1.0 and second[0] == 1.0 and second_label[0] == 1


def test_one_rank_is_a_textbook_lloyd_step():
    from sklearn.cluster import KMeans

    pts, _, init = small_problem()
    K = init.shape[0]
    new, labels, reduced, count = oracle.kmeans_iterate(pts, init, 1, None)
    km = KMeans(n_clusters=K, init=init.astype(np.float64), n_init=1, max_iter=1, algorithm="lloyd", tol=0.0)
    km.fit(pts.astype(np.float64))
    # after max_iter=1 sklearn's centres are the means of the points assigned to the initial centres
    assert np.allclose(new, km.cluster_centers_, rtol=1e-5, atol=1e-5)
    assert (count == 1).all()
    # and the labels of the step are the nearest initial centre
    means = np.stack([pts[labels == k].astype(np.float64).mean(0) for k in range(K)])
    assert np.allclose(new, means, rtol=1e-5, atol=1e-5)


def test_inertia_never_increases_when_everything_arrives():
    pts, _, _ = small_problem(N=3000, D=5, K=7, seed=22)
    cents = pts[:7].copy()                        # a poor start, so that several iterations move
    prev = np.inf
    for _ in range(8):
        labels, best, _, _ = oracle.kmeans_assign(pts, cents)
        inertia = best.sum()
        assert inertia <= prev * (1 + 1e-6)       # partial sums travel through fp32: allow its rounding
        prev = inertia
        cents, _, _, _ = oracle.kmeans_iterate(pts, cents, 4, None)


def test_partials_bookkeeping_and_masked_update():
    N, D, K, P = 4096, 8, 6, 8
    pts, comp, init = small_problem(N, D, K)
    labels, _, _, _ = oracle.kmeans_assign(pts, init)
    part = oracle.kmeans_partials(pts, labels, K, P)
    assert part.shape == (P, K, D + 4) and (part[:, :, D + 1:] == 0).all()
    shard = N // P
    for r in (0, 3, 7):
        lab = labels[r * shard:(r + 1) * shard]
        x = pts[r * shard:(r + 1) * shard].astype(np.float64)
        for k in range(K):
            assert part[r, k, D] == (lab == k).sum()
            assert np.allclose(part[r, k, :D], x[lab == k].sum(0), rtol=1e-6, atol=1e-6)
    assert part[:, :, D].sum() == N
    # masked combine: each centroid is the mean of exactly the points of the arrived (rank, centroid) cells
    arrived = np.random.default_rng(1).random((P, K)) < 0.6
    arrived[:, 2] = False                         # nobody reports centroid 2: it must stay where it was
    mask = inputs.pack_mask(arrived)
    new, labels2, reduced, count = oracle.kmeans_iterate(pts, init, P, mask)
    assert np.array_equal(labels, labels2)
    assert count.tolist() == arrived.sum(0).tolist()
    for k in range(K):
        sel = np.zeros(N, dtype=bool)
        for r in range(P):
            if arrived[r, k]:
                sel[r * shard:(r + 1) * shard] = labels[r * shard:(r + 1) * shard] == k
        assert reduced[k, D] == sel.sum()
        if sel.any():
            assert np.allclose(new[k], pts[sel].astype(np.float64).mean(0), rtol=1e-5, atol=1e-5)
        else:
            assert np.array_equal(new[k], init[k])
    assert np.array_equal(new[2], init[2])


def test_ragged_shards():
    N, D, K, P = 1000, 3, 4, 7                    # 1000 / 7 is not an integer
    pts, comp, init = small_problem(N, D, K, seed=23)
    labels, _, _, _ = oracle.kmeans_assign(pts, init)
    part = oracle.kmeans_partials(pts, labels, K, P)
    assert part[:, :, D].sum() == N
    for r in range(P):
        assert part[r, :, D].sum() == (r + 1) * N // P - r * N // P
