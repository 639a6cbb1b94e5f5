"""The tensor-core candidate search on data built against its rounding, checked with the fp64 CPU checker.

The search multiplies points and centroids at reduced precision (bf16: 8 significant bits, tf32: 11) and may only
propose: whenever its two best scores are closer than its error bound the point is decided again by the exact fp32
form.  The data below puts every coordinate next to a rounding midpoint (or just below the next representable
number, for hardware that truncates), with the signs chosen so that all roundings push the inner product x.c the
same way, and sets the true inner product so that the nearer of two opposite centroids wins by a relative gap only
just above the near-tie limit of 1e-5.  A search that trusted its scores, or a bound a factor of two too small, gets
most of these points wrong; the test asks for none.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle
from tests.gpu_util import ec, to_dev, to_host


@pytest.fixture(autouse=True)
def _need_gpu(cuda_device):
    yield


def reduced_precision(a, bits, truncate):
    """a (fp64 array of fp32 values) kept to `bits` significant bits, rounded to nearest even or truncated."""
    m, e = np.frexp(a)                        # a = m 2^e, 0.5 <= |m| < 1
    s = np.ldexp(m, bits)
    s = np.trunc(s) if truncate else np.rint(s)
    return np.ldexp(s, e - bits)


def adversarial_pair(D, bits, truncate, n_points, seed, gap_lo=3e-5, gap_hi=3e-4, extra_pairs=0):
    """Centroids c_0 and c_1 = -c_0 (plus `extra_pairs` far pairs) and n_points points x with |x| close to |c_0|,
    x.c_0 = +-g tiny, built so that reduced precision shifts the computed x.c_0 by nearly 2^(1-bits) |x||c_0|
    against the truth.  Returns (points fp32, centroids fp32)."""
    rng = np.random.default_rng(seed)
    half = D // 2
    # magnitudes: numbers with `bits` significant bits in [1, 1.25) and [2, 2.5), where half a unit in the last place is
    # largest relative to the number; coordinate d of the first half and d + half share one
    base = np.ldexp(rng.integers(1 << (bits - 1), 5 << (bits - 3), size=half).astype(np.float64), -(bits - 1)) * rng.choice([1.0, 2.0], size=half)
    ulp = np.ldexp(1.0, np.floor(np.log2(base)).astype(int) - (bits - 1))          # spacing of the reduced format at base
    def below(eta):        # just under the point where the value would go up: comes down to base
        return base + (ulp * (1.0 - eta) if truncate else 0.5 * ulp * (1.0 - eta))
    def above(eta):        # just over the midpoint: goes up to base + ulp (truncation cannot go up: stays exact)
        return base + (0.0 if truncate else 0.5 * ulp * (1.0 + eta))
    eta_c = 2.0 ** -6
    sign = rng.choice([-1.0, 1.0], size=D)
    c0 = np.concatenate([below(eta_c), above(eta_c)]) * sign      # first half loses magnitude, second half gains
    c0[half - 1] = base[half - 1] * sign[half - 1]                # the tuning coordinate's centroid entry is exact
    pts = np.empty((n_points, D))
    for j in range(n_points):
        eta = 2.0 ** -rng.integers(5, 9)
        x = np.concatenate([below(eta), -above(eta)]) * sign       # products: + (underestimated), - (overestimated)
        g = rng.uniform(gap_lo, gap_hi) * (x @ x + c0 @ c0) / 4.0  # d_1^2 - d_0^2 = 4 x.c_0 = relative gap * d^2
        rest = x @ c0 - x[half - 1] * c0[half - 1]
        x[half - 1] = (g - rest) / c0[half - 1]                    # sets x.c_0 = g exactly (up to fp32 rounding of x)
        if j % 2:
            x = -x                                                 # mirrored: truth is c_1, the search prefers c_0
        pts[j] = x
    cents = [c0, -c0]
    for q in range(extra_pairs):                                   # far pairs: never the nearest, but they widen tau
        v = rng.standard_normal(D)
        v *= 3.0 * np.linalg.norm(c0) / np.linalg.norm(v)
        cents += [v, -v]
    return pts.astype(np.float32), np.asarray(cents, dtype=np.float32)


def plain_search_labels(points, cents, bits, truncate):
    """What a search at reduced precision would answer if nobody checked it (test bookkeeping: shows the data bites)."""
    xr = reduced_precision(points.astype(np.float64), bits, truncate)
    cr = reduced_precision(cents.astype(np.float64), bits, False)
    v = (cents.astype(np.float64) ** 2).sum(1)[None, :] - 2.0 * xr @ cr.T
    return v.argmin(1)


@pytest.mark.parametrize("D", [16, 32])
@pytest.mark.parametrize("bits,truncate", [(8, False), (11, False), (11, True)])
@pytest.mark.parametrize("extra_pairs", [0, 31])
def test_search_never_decides_inside_its_error(D, bits, truncate, extra_pairs):
    n = 128 * 6 + 37
    points, cents = adversarial_pair(D, bits, truncate, n, seed=100 * D + bits + (7 if truncate else 0), extra_pairs=extra_pairs)
    K = cents.shape[0]
    c_labels, d1, d2, second = oracle.kmeans_assign(points, cents, 4)
    rel_gap = (d2 - d1) / d2
    assert (rel_gap > 2e-5).all() and (rel_gap < 1e-3).all()       # decided, but barely
    assert set(np.unique(c_labels)) == {0, 1}
    fooled = (plain_search_labels(points, cents, bits, truncate) != c_labels).mean()
    assert fooled > 0.9                                             # an unchecked search gets nearly all of them wrong
    d_points = to_dev(points)
    km = ec.KMeans(d_points, K, 1, to_dev(cents))
    km.set_path(2)                                                  # the tensor-core path
    lab = torch.empty(n, dtype=torch.int32, device="cuda")
    km.assign(to_dev(cents), lab)
    torch.cuda.synchronize()
    assert np.array_equal(to_host(lab), c_labels), "stand-alone assignment"
    km.iterate(None)                                                # the fused pass (search + sums), first iteration
    km.get(labels=lab)
    torch.cuda.synchronize()
    assert np.array_equal(to_host(lab), c_labels), "fused pass, all points summed"
    km.set_centroids(to_dev(cents))
    km.iterate(None)                                                # the fused pass that sums only changes
    km.get(labels=lab)
    torch.cuda.synchronize()
    assert np.array_equal(to_host(lab), c_labels), "fused pass, changes only"
    assert km.tc_status() == 0
    km.destroy()


def test_norms_that_differ_by_orders_of_magnitude_inside_a_tile():
    """The error bound of a point scales with its own squared norm.  Points of norm 100 and of norm 0.01 alternate
    inside every tile, around centroids of norm 1: a bound taken from a neighbour's norm would let the search decide
    large points it cannot separate."""
    D, K, n = 32, 24, 128 * 40 + 5
    rng = np.random.default_rng(5)
    cents = rng.standard_normal((K, D))
    cents /= np.linalg.norm(cents, axis=1, keepdims=True)
    direction = rng.standard_normal((n, D))
    direction /= np.linalg.norm(direction, axis=1, keepdims=True)
    scale = np.where(rng.random(n) < 0.5, 100.0, 0.01)
    points = (direction * scale[:, None]).astype(np.float32)
    cents = cents.astype(np.float32)
    c_labels, d1, d2, second = oracle.kmeans_assign(points, cents, 4)
    for P in (1, 3):
        km = ec.KMeans(to_dev(points), K, P, to_dev(cents))
        km.set_path(2)
        lab = torch.empty(n, dtype=torch.int32, device="cuda")
        for _ in range(3):                                         # the race this guards against was timing dependent
            km.assign(to_dev(cents), lab)
            torch.cuda.synchronize()
            g = to_host(lab)
            diff = np.nonzero(g != c_labels)[0]
            assert ((d2[diff] - d1[diff]) <= 1e-5 * d2[diff]).all()
            assert np.array_equal(g[diff], second[diff])
        km.destroy()
