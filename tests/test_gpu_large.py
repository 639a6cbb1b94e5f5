"""Sizes beyond 2^31 elements and 2^32 bytes: the index arithmetic of the kernels.

The vectors are too long for the CPU checker to walk in a test, so the inputs are a pattern
generated on the device with plain tensor operations, and the checker is run on whole sampled
segments (copied back to the host) as small problems of their own: the first segments, the last
(short) one, and those that straddle the 2^31-element and the 2^32- and 2^33-byte marks."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle
from paper_2203_17063_b200 import inputs
from tests.gpu_util import bits, ec


def _pattern(n, r, dtype):
    """buf_r[i] = ((i * (2r + 3) + 17r) mod 65521) / 256 - 100: exact in fp32, different for every rank."""
    out = torch.empty(n, dtype=dtype, device="cuda")
    step = 1 << 26
    for lo in range(0, n, step):
        hi = min(n, lo + step)
        i = torch.arange(lo, hi, dtype=torch.int64, device="cuda")
        out[lo:hi] = (((i * (2 * r + 3) + 17 * r) % 65521).to(torch.float32) / 256.0 - 100.0).to(dtype)
    return out


def test_allreduce_beyond_2_31_elements(cuda_device):
    free, _ = torch.cuda.mem_get_info()
    P, seg = 3, (1 << 22) + 64
    n = (1 << 31) + 12345 * 4 + 3                       # last segment short, ends inside a vector
    if free < (P + 1) * n * 4 + (4 << 30):
        pytest.skip("not enough free device memory")
    S = (n + seg - 1) // seg
    bufs = [_pattern(n, r, torch.float32) for r in range(P)]
    rounds = inputs.arrival_rounds(4100, P, S, 0.5)
    masks = inputs.cumulative_masks(rounds)
    res = torch.full((n,), float("nan"), device="cuda")
    cnt = torch.zeros(S, dtype=torch.int32, device="cuda")
    ar = ec.Allreduce(P, n, ec.F32, ec.SUM, seg)
    marks = sorted({0, 1, S - 2, S - 1, (1 << 30) // seg, (1 << 30) // seg + 1, (1 << 31) // seg, (1 << 31) // seg - 1})
    for t, m in enumerate(masks):
        d_mask = torch.from_numpy(np.ascontiguousarray(m, dtype=np.uint64).view(np.int64)).cuda()
        ar.apply(bufs, d_mask, res, cnt)
        torch.cuda.synchronize()
        want_cnt = (rounds <= t + 1).sum(axis=0).astype(np.uint32)
        assert np.array_equal(cnt.cpu().numpy().view(np.uint32), want_cnt)
    # whole sampled segments against the checker, replaying the three rounds on the slice
    for s in marks:
        lo, hi = s * seg, min(n, (s + 1) * seg)
        h = [b[lo:hi].cpu().numpy() for b in bufs]
        ref = oracle.Allreduce(P, hi - lo, oracle.F32, oracle.SUM, hi - lo)
        c_res = np.full(hi - lo, np.nan, dtype=np.float32)
        c_cnt = np.zeros(1, dtype=np.uint32)
        for m in masks:
            ref.apply(h, np.ascontiguousarray(m[s:s + 1]), c_res, c_cnt)
        got = res[lo:hi].cpu().numpy()
        assert np.array_equal(bits(got), bits(c_res)), f"segment {s}"
    # and a closed form everywhere: all three ranks are in, the values are exact multiples of 2^-8
    step = 1 << 26
    for lo in range(0, n, step):
        hi = min(n, lo + step)
        want = sum(b[lo:hi].double() for b in bufs)
        assert bool((res[lo:hi].double() == want).all())
    ar.destroy()


def test_allgatherv_beyond_2_32_bytes(cuda_device):
    free, _ = torch.cuda.mem_get_info()
    counts = np.array([(1 << 29) + 5, 7, 0, (1 << 28) + 11, 3], dtype=np.int64)      # 6.4 GB of int64 in all
    total = int(counts.sum())
    if free < 2 * total * 8 + (4 << 30):
        pytest.skip("not enough free device memory")
    P = len(counts)
    bufs = []
    for r, c in enumerate(counts):
        t = torch.empty(int(c), dtype=torch.int64, device="cuda")
        step = 1 << 26
        for lo in range(0, int(c), step):
            hi = min(int(c), lo + step)
            t[lo:hi] = torch.arange(lo, hi, dtype=torch.int64, device="cuda") * 1000003 + (r + 1) * (1 << 56)
        bufs.append(t)
    arrived = np.array([True, True, True, True, False])
    d_mask = torch.from_numpy(inputs.pack_mask(arrived[:, None]).reshape(-1).view(np.int64)).cuda()
    d_counts = torch.from_numpy(counts).cuda()
    displs = torch.empty(P + 1, dtype=torch.int64, device="cuda")
    out = torch.full((total + 16,), -7, dtype=torch.int64, device="cuda")
    status = torch.ones(1, dtype=torch.int32, device="cuda")
    ec.allgatherv(bufs, d_counts, ec.I64, d_mask, displs, out[8:8 + total], status, out_capacity_elems=total)
    torch.cuda.synchronize()
    d = displs.cpu().numpy()
    assert np.array_equal(d, np.concatenate([[0], np.cumsum(counts)]))                   # the checker's definition of displs
    assert int(status.item()) == 0
    assert bool((out[:8] == -7).all()) and bool((out[8 + total:] == -7).all())          # guard words
    for r in range(P):
        slot = out[8 + int(d[r]): 8 + int(d[r + 1])]
        if arrived[r]:
            assert torch.equal(slot, bufs[r]), f"rank {r}"
        else:
            assert bool((slot == -7).all())


def _byte_pattern(nbytes, salt):
    """bytes[i] = low byte of (i * 2654435761 + salt) >> 11, filled on the device in pieces."""
    out = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    step = 1 << 27
    for lo in range(0, nbytes, step):
        hi = min(nbytes, lo + step)
        i = torch.arange(lo, hi, dtype=torch.int64, device="cuda")
        out[lo:hi] = (((i * 2654435761 + salt) >> 11) & 255).to(torch.uint8)
    return out


def test_alltoall_rank_buffers_beyond_2_32_bytes(cuda_device):
    free, _ = torch.cuda.mem_get_info()
    P = 3
    block = (3 << 29) + 48                                # 1.5 GiB blocks: a rank's buffer is 4.5 GiB
    if free < 2 * P * P * block + (6 << 30):
        pytest.skip("not enough free device memory")
    send = [_byte_pattern(P * block, 1000003 * (s + 1)) for s in range(P)]
    recv = [torch.full((P * block,), 0xA5, dtype=torch.uint8, device="cuda") for _ in range(P)]
    arrived = np.ones((P, P), dtype=bool)
    arrived[2, 0] = False                                 # the block from rank 0 to rank 2 is late
    words = np.zeros((P, 1), dtype=np.uint64)
    for d in range(P):
        for s in range(P):
            if arrived[d, s]:
                words[d, 0] |= np.uint64(1) << np.uint64(s)
    d_mask = torch.from_numpy(words.view(np.int64)).cuda()
    cnt = torch.zeros(P, dtype=torch.int32, device="cuda")
    ec.alltoall(send, recv, block, d_mask, cnt)
    torch.cuda.synchronize()
    assert cnt.cpu().tolist() == [3, 3, 2]
    for d in range(P):
        for s in range(P):
            slot = recv[d][s * block:(s + 1) * block]
            if arrived[d, s]:
                assert torch.equal(slot, send[s][d * block:(d + 1) * block]), f"block {s} -> {d}"   # the transpose rule of Sec. IV-B
            else:
                assert bool((slot == 0xA5).all())


def test_bcast_prefix_beyond_2_32_bytes(cuda_device):
    free, _ = torch.cuda.mem_get_info()
    n = (3 << 29) + 5                                     # 6.4 GB of fp32; three quarters of it are delivered
    seg = (1 << 22) + 64
    if free < 3 * n * 4 + (6 << 30):
        pytest.skip("not enough free device memory")
    S = (n + seg - 1) // seg
    keep = -(-3 * S // 4)                                 # ceil(0.75 S) segments
    src = _byte_pattern(n * 4, 77).view(torch.float32)
    dst = [src, torch.full((n,), -3.0, device="cuda"), torch.full((n,), -3.0, device="cuda")]   # the root receives in place
    notify = torch.zeros(S, dtype=torch.int64, device="cuda")
    ec.bcast(src, dst, 0, ec.F32, seg, 0.75, notify)
    torch.cuda.synchronize()
    got = notify.cpu().numpy().view(np.uint64)
    assert (got[:keep] == 7).all() and (got[keep:] == 0).all()
    edge = min(n, keep * seg)
    assert edge * 4 > 1 << 32
    for r in (1, 2):
        assert torch.equal(dst[r][:edge].view(torch.int32), src[:edge].view(torch.int32)), f"receiver {r}"
        assert bool((dst[r][edge:] == -3.0).all())


def test_kmeans_points_beyond_2_31_elements(cuda_device):
    """N * D > 2^31: point j sits within 0.5 of centre j mod K (centres 20 apart), so the labels, the counts and,
    to rounding, the centroids of one iteration are known in closed form at any size."""
    free, _ = torch.cuda.mem_get_info()
    N, D, K, P = (1 << 26) + 777, 32, 8, 3
    if free < N * D * 4 + (8 << 30):
        pytest.skip("not enough free device memory")
    g = torch.Generator(device="cuda").manual_seed(4242)
    centres = torch.zeros(K, D, device="cuda")
    centres[torch.arange(K), torch.arange(K)] = 20.0                      # centre k = 20 e_k
    pts = torch.empty(N, D, device="cuda")
    sums = torch.zeros(K, D, dtype=torch.float64, device="cuda")
    step = 1 << 22
    for lo in range(0, N, step):
        hi = min(N, lo + step)
        lab = torch.arange(lo, hi, device="cuda") % K
        blockp = centres[lab] + (torch.rand(hi - lo, D, device="cuda", generator=g) - 0.5)
        pts[lo:hi] = blockp
        sums.index_add_(0, lab, blockp.double())
    init = centres + 0.25                                                 # start off the centres: still the nearest by far
    km = ec.KMeans(pts, K, P, init.contiguous())
    km.iterate(None)
    cents = torch.empty(K, D, device="cuda")
    labels = torch.empty(N, dtype=torch.int32, device="cuda")
    reduced = torch.empty(K, D + 4, device="cuda")
    contrib = torch.empty(K, dtype=torch.int32, device="cuda")
    km.get(cents, labels, reduced, contrib)
    torch.cuda.synchronize()
    for lo in range(0, N, step):
        hi = min(N, lo + step)
        assert torch.equal(labels[lo:hi].long(), torch.arange(lo, hi, device="cuda") % K), f"labels of points {lo}..{hi}"
    counts = torch.tensor([(N - k + K - 1) // K for k in range(K)], dtype=torch.float64, device="cuda")
    assert torch.equal(reduced[:, D].double(), counts)                    # counts are exact
    assert bool((contrib == P).all())
    want = sums / counts[:, None]
    assert float((cents.double() - want).abs().max()) < 1e-4 * 20.0
    assert km.tc_status() == 0
    km.destroy()
