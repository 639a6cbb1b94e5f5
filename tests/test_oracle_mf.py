"""The checker's matrix-factorisation iteration against what the mathematics fixes."""
import numpy as np
import pytest

import oracle
from paper_2203_17063_b200 import inputs


def _small(P=4, U=24, I=10, k=4, nnz=160, seed=11, lr=0.02, lam=0.05, seg=3):
    d = inputs.mf_ratings(seed, U, I, 3, nnz, P)
    pu, qi = inputs.mf_init_factors(seed, U, I, k, 0.3)
    return d, pu, qi, oracle.MatrixFactorization(d, pu, qi, lr, lam, seg)


def test_both_storage_orders_hold_the_same_ratings():
    d, *_ = _small()
    a = sorted(zip(np.repeat(np.arange(24), np.diff(d["user_ptr"])).tolist(), d["user_item"].tolist(), d["user_val"].tolist()))
    b = []
    for r in range(4):
        for i in range(10):
            for j in range(int(d["rank_item_ptr"][r, i]), int(d["rank_item_ptr"][r, i + 1])):
                u = int(d["item_user"][j])
                assert r * 24 // 4 <= u < (r + 1) * 24 // 4                # a rank holds only its own users
                b.append((u, i, float(d["item_val"][j])))
    assert a == sorted(b)


def test_steps_follow_the_gradient_of_the_loss():
    """Finite differences of loss(): d/dp_u = -(g_u - lam p_u), d/dq_i = -(sum_r G_r[i] - lam q_i)."""
    d, pu, qi, mf = _small()
    g_user, _ = mf.user_gradient()
    g_item = sum(mf.rank_item_gradient(r) for r in range(4))
    h = 1e-6
    for (u, c) in [(0, 0), (7, 3), (23, 1)]:
        mf.pu[u, c] += h; up = mf.loss(); mf.pu[u, c] -= 2 * h; dn = mf.loss(); mf.pu[u, c] += h
        assert np.isclose((up - dn) / (2 * h), -(g_user[u, c] - mf.lam * mf.pu[u, c]), rtol=1e-5, atol=1e-7)
    for (i, c) in [(0, 0), (4, 2), (9, 3)]:
        mf.qi[i, c] += h; up = mf.loss(); mf.qi[i, c] -= 2 * h; dn = mf.loss(); mf.qi[i, c] += h
        assert np.isclose((up - dn) / (2 * h), -(g_item[i, c] - mf.lam * mf.qi[i, c]), rtol=1e-5, atol=1e-7)


def test_fresh_iterations_are_plain_gradient_descent_and_the_error_falls():
    d, pu, qi, mf = _small()
    dense = np.zeros((24, 10)); cnt = np.zeros((24, 10))
    users = np.repeat(np.arange(24), np.diff(d["user_ptr"]))
    # the same step written with dense matrices: E = mask * (R - P Q^T) summed over repeated observations
    p, q = pu.astype(np.float64), qi.astype(np.float64)
    sses = []
    for it in range(30):
        E = np.zeros((24, 10))
        for u, i, v in zip(users, d["user_item"], d["user_val"]):
            E[u, i] += float(v) - p[u] @ q[i]
        sse, seg_clock, refreshed = mf.iterate(None, 0)
        sses.append(sse)
        p, q = p + 0.02 * (E @ q - 0.05 * p), q + 0.02 * (E.T @ p - 0.05 * q)
        assert np.allclose(mf.pu, p, rtol=1e-12, atol=1e-14) and np.allclose(mf.qi, q, rtol=1e-12, atol=1e-14)
        assert refreshed.all() and (seg_clock == it + 1).all()
    assert sses[-1] < 0.5 * sses[0] and all(b <= a * (1 + 1e-12) for a, b in zip(sses, sses[1:]))


def test_the_number_of_ranks_does_not_matter_when_everything_is_fresh():
    d1 = inputs.mf_ratings(3, 24, 10, 3, 160, 1)
    d4 = inputs.mf_ratings(3, 24, 10, 3, 160, 4)
    pu, qi = inputs.mf_init_factors(3, 24, 10, 4, 0.3)
    a = oracle.MatrixFactorization(d1, pu, qi, 0.02, 0.05, 3)
    b = oracle.MatrixFactorization(d4, pu, qi, 0.02, 0.05, 3)
    for _ in range(5):
        a.iterate(None, 0); b.iterate(None, 2)
    assert np.allclose(a.pu, b.pu, rtol=1e-12) and np.allclose(a.qi, b.qi, rtol=1e-12)


def test_stale_contributions_are_reused_until_they_are_too_old():
    """Slack 2: a contribution that is never delivered fresh is recomputed every third iteration (clock 1, 4, 7):
    the wait of Algorithm 1.  In between the rank's buffer is what it was."""
    d, pu, qi, mf = _small()
    never = np.zeros((4, 4), dtype=bool)
    never[0] = True                                         # rank 0 always fresh, the others never
    clocks = []
    for it in range(7):
        before = mf.grad[2].copy()
        sse, seg_clock, refreshed = mf.iterate(never, 2)
        clocks.append(int(mf.notif_clock[1, 2]))
        assert refreshed[0].all()
        if not refreshed[2].any():
            assert np.array_equal(mf.grad[2], before)
        assert (seg_clock == mf.notif_clock.min(axis=1)).all() and (mf.clock - seg_clock <= 2).all()
    assert clocks == [1, 1, 1, 4, 4, 4, 7]


def test_slack_zero_is_synchronous_whatever_the_refresh_pattern():
    d, pu, qi, a = _small()
    _, _, _, b = _small()
    rng = np.random.default_rng(0)
    for _ in range(4):
        a.iterate(None, 0)
        b.iterate(rng.random((4, 4)) < 0.3, 0)
    assert np.array_equal(a.pu, b.pu) and np.array_equal(a.qi, b.qi)
