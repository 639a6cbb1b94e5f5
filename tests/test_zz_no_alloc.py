"""ec_kmeans_partials_static: the partial sums for callers that cannot allocate device memory.

Collected last on purpose (a run that stops at the first failure has then already run
everything else).  The entry point keeps its per-block sums in one fixed array inside the
library, shared by all calls, so the test makes two calls in a row with different labels
and checks both against the workspace-based ec_kmeans_partials: nothing may leak from the
first call into the second.  Same kernels and order of additions: the bits must agree."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2203_17063_b200 import binding as ec
from paper_2203_17063_b200 import inputs


def test_static_partials_match_workspace_partials_twice(cuda_device):
    N, D, K, P = 1 << 16, 32, 64, 64
    pts, comp, _ = inputs.kmeans_mixture(31, N, D, K)
    d_pts = torch.from_numpy(pts).cuda()
    rng = np.random.default_rng(32)
    label_sets = [torch.from_numpy(comp.astype(np.int32)).cuda(),
                  torch.from_numpy(rng.integers(0, K, size=N, dtype=np.int32)).cuda()]
    km = ec.KMeans(d_pts, K, P, torch.from_numpy(pts[:K].copy()).cuda())
    expect = []
    for lab in label_sets:
        out = torch.empty(P, K, D + 4, device="cuda")
        km.partials(lab, out)
        expect.append(out)
    torch.cuda.synchronize()
    assert not torch.equal(expect[0], expect[1])
    for lab, want in zip(label_sets, expect):                       # two calls in a row on the shared array
        got = torch.full((P, K, D + 4), float("nan"), device="cuda")
        ec.kmeans_partials_static(d_pts, lab, K, P, got)
        torch.cuda.synchronize()
        assert torch.equal(got[:, :, D], want[:, :, D])             # counts exact
        num = torch.linalg.norm(got[:, :, :D].double() - want[:, :, :D].double(), dim=-1)
        den = torch.linalg.norm(want[:, :, :D].double(), dim=-1)
        assert bool((num <= 1e-4 * den + 1e-30).all())              # the tolerance of the K-means parity tests
        assert torch.equal(got, want)                               # and in fact the same bits
    km.destroy()


def test_static_partials_reject_shapes_beyond_the_fixed_array(cuda_device):
    # 64 ranks x 2 blocks per rank x 1024 centroids x 36 floats = 18.9 MB of per-block sums: above 8 MiB
    N, D, K, P = 1 << 16, 32, 1024, 64
    pts = torch.zeros(N, D, device="cuda")
    lab = torch.zeros(N, dtype=torch.int32, device="cuda")
    out = torch.empty(P, K, D + 4, device="cuda")
    with pytest.raises(ec.EcError) as err:
        ec.kmeans_partials_static(pts, lab, K, P, out)
    assert err.value.code == ec.ERR_CAPACITY
    with pytest.raises(ec.EcError):
        ec.kmeans_partials_static(pts, lab, K, 0, out)              # invalid P
