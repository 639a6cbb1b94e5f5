"""Broadcast with a data threshold (Sec. III-B): the checker against what the paper and the
mathematics fix, and the CUDA path against the checker."""
import numpy as np
import pytest
import torch

import oracle
from paper_2203_17063_b200 import inputs


# ---------------------------------------------------------------------------
# the checker
# ---------------------------------------------------------------------------
def _case(P, n, seed):
    rng = np.random.default_rng(seed)
    src = rng.standard_normal(n).astype(np.float32)
    dsts = [np.full(n, -7.0, dtype=np.float32) for _ in range(P)]
    return src, dsts


def test_full_threshold_is_a_plain_broadcast():
    src, dsts = _case(5, 1000, 1)
    words = oracle.bcast(src, dsts, 2, 64, 1.0)
    for d in dsts:
        assert np.array_equal(d, np.broadcast_to(src, d.shape))      # every receiver holds the root's vector
    assert np.array_equal(words, oracle.data_fraction_mask(5, 16, 1.0))


@pytest.mark.parametrize("fraction,segments", [(0.0, 0), (0.25, 4), (0.26, 5), (0.5, 8), (0.75, 12), (1.0, 16)])
def test_a_quarter_half_three_quarters_of_the_data(fraction, segments):
    """The thresholds of the paper's Broadcast experiment: that share of the segments, rounded up, is shipped."""
    n, seg, P = 1000, 64, 4                                # 16 segments, the last one short (40 elements)
    src, dsts = _case(P, n, 2)
    words = oracle.bcast(src, dsts, 0, seg, fraction)
    cut = min(n, segments * seg)
    for d in dsts:
        assert np.array_equal(d[:cut], src[:cut])
        assert (d[cut:] == -7.0).all()                     # beyond the threshold the receiver keeps what it had
    arrived = np.zeros((P, 16), dtype=bool)
    arrived[:, :segments] = True
    assert np.array_equal(words, inputs.pack_mask(arrived))


def test_absent_receivers_and_root_in_place():
    n, seg, P, root = 300, 50, 70, 65                      # two notification words per segment
    src, dsts = _case(P, n, 3)
    dsts[root] = src                                       # the root broadcasts from its own buffer
    dsts[3] = None
    dsts[64] = None
    before = src.copy()
    words = oracle.bcast(src, dsts, root, seg, 0.5)
    assert np.array_equal(src, before)
    arrived = np.zeros((P, 6), dtype=bool)
    arrived[:, :3] = True
    arrived[3] = False
    arrived[64] = False
    assert np.array_equal(words, inputs.pack_mask(arrived))
    for r, d in enumerate(dsts):
        if d is not None and r != root:
            assert np.array_equal(d[:150], src[:150]) and (d[150:] == -7.0).all()


def test_broadcast_then_reduce_of_the_delivered_part():
    """The words a broadcast returns are a valid arrival mask: reducing the receive buffers under them
    gives P times the delivered prefix and the identity elsewhere."""
    n, seg, P = 256, 32, 4
    src = np.arange(n, dtype=np.float32)
    dsts = [np.full(n, np.nan, dtype=np.float32) for _ in range(P)]     # never-received data is poison
    words = oracle.bcast(src, dsts, 1, seg, 0.5)
    ar = oracle.Allreduce(P, n, oracle.F32, oracle.SUM, seg)
    res = np.full(n, np.nan, dtype=np.float32)
    cnt = np.zeros(n // seg, dtype=np.uint32)
    ar.apply(dsts, words, res, cnt)
    assert np.array_equal(res[:128], P * src[:128]) and (res[128:] == 0.0).all()
    assert cnt.tolist() == [P] * 4 + [0] * 4


# ---------------------------------------------------------------------------
# the CUDA path
# ---------------------------------------------------------------------------
@pytest.mark.gpu
@pytest.mark.parametrize("P,n,seg,fraction,dtype_name", [
    (4, 1000, 64, 0.5, "f32"), (16, (1 << 18) + 5, 4096, 0.75, "f32"), (70, 30000, 1000, 0.26, "bf16"),
    (256, 8191, 512, 1.0, "i64"), (3, 100, 7, 0.0, "f64"), (1, 64, 64, 1.0, "f32"), (5, 12289, 4096, 0.7, "bf16")])
@pytest.mark.parametrize("misalign", [0, 1])
def test_gpu_bcast_matches_checker(cuda_device, P, n, seg, fraction, dtype_name, misalign):
    from tests.gpu_util import ec, to_dev, to_host
    dt = {"f32": (ec.F32, np.float32), "bf16": (ec.BF16, np.uint16), "i64": (ec.I64, np.int64), "f64": (ec.F64, np.float64)}[dtype_name]
    rng = np.random.default_rng(7 + P)
    src = rng.integers(-30000, 30000, size=n).astype(dt[1])
    S = (n + seg - 1) // seg
    W = (P + 63) // 64
    root = P // 2
    h_dsts = [np.full(n, 77, dtype=dt[1]) for _ in range(P)]
    if P > 2:
        h_dsts[1] = None
    want = [None if d is None else d.copy() for d in h_dsts]
    if not misalign:                                       # aligned run: the root broadcasts in place;
        want[root] = src                                   # misaligned run: it has a receive buffer of its own
        h_dsts[root] = src
    want_words = oracle.bcast(src, want, root, seg, fraction)
    d_src = to_dev(src, misalign)
    d_dsts = [None if d is None else (d_src if d is src else to_dev(d, misalign)) for d in h_dsts]
    words = torch.full((S, W), -1, dtype=torch.int64, device="cuda")
    ec.bcast(d_src, d_dsts, root, dt[0], seg, fraction, words)
    torch.cuda.synchronize()
    assert np.array_equal(words.cpu().numpy().view(np.uint64), want_words)
    for r in range(P):
        if d_dsts[r] is None:
            continue
        assert np.array_equal(to_host(d_dsts[r]), want[r]), f"rank {r}"


@pytest.mark.gpu
def test_gpu_bcast_argument_errors(cuda_device):
    from tests.gpu_util import ec
    src = torch.zeros(1024, device="cuda")
    dsts = [torch.zeros(1024, device="cuda") for _ in range(3)]
    with pytest.raises(ec.EcError):
        ec.bcast(src, dsts, 3, ec.F32, 64, 0.5)            # root out of range
    with pytest.raises(ec.EcError):
        ec.bcast(src, dsts, 0, ec.F32, 64, 1.5)            # threshold beyond 1
    with pytest.raises(ec.EcError):
        ec.bcast(src, [src[8:], dsts[1]], 1, ec.F32, 64, 0.5)   # a receive buffer overlapping the source
