"""GPU parity of ec_allgatherv against the CPU checker (bit-exact), through the C ABI."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle
from paper_2203_17063_b200 import inputs
from tests.gpu_util import ec, to_dev, to_host

SENT = -0x0123456789ABCDEF
NP = {ec.F32: np.float32, ec.BF16: np.uint16, ec.I64: np.int64, ec.F64: np.float64}


@pytest.fixture(autouse=True)
def _need_gpu(cuda_device):
    yield


def gather_both(bufs, counts, dtype, arrived, capacity=None, guard=8, offset=0):
    """Run GPU and CPU on the same inputs; `out` is pre-filled with a sentinel and
    surrounded by guard words.  Returns (gpu_out, gpu_displs, gpu_status, cpu_out, cpu_displs, cpu_status)."""
    P = len(bufs)
    total = int(np.sum(counts))
    cap = total if capacity is None else capacity
    npdt = NP[dtype]
    sent = np.array([SENT], dtype=np.int64).view(npdt)[0] if npdt != np.uint16 else np.uint16(0xBEEF)
    mask = None if arrived is None else inputs.pack_mask(np.asarray(arrived)[:, None]).reshape(-1)
    c_out = np.full(cap, sent, dtype=npdt)
    c_displs, c_status = oracle.allgatherv(bufs, counts, mask, c_out)
    whole = np.full(cap + 2 * guard + offset, sent, dtype=npdt)
    d_whole = to_dev(whole)
    d_out = d_whole[guard + offset: guard + offset + cap]
    d_bufs = [to_dev(b) if (arrived is None or arrived[r]) else None for r, b in enumerate(bufs)]
    d_bufs = [b if b is not None else torch.empty(0, device="cuda") for b in d_bufs]
    d_counts = to_dev(np.asarray(counts, dtype=np.int64))
    d_displs = torch.full((P + 1,), -1, dtype=torch.int64, device="cuda")
    d_status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    d_mask = None if mask is None else to_dev(mask)
    ptrs = [b.data_ptr() if b.numel() else 0 for b in d_bufs]
    if arrived is None:
        ptrs = [b.data_ptr() for b in d_bufs]
    ec.allgatherv(ptrs, d_counts, dtype, d_mask, d_displs, d_out, d_status, out_capacity_elems=cap)
    torch.cuda.synchronize()
    g_whole = to_host(d_whole)
    lo, hi = guard + offset, guard + offset + cap
    assert (g_whole[:lo] == sent).all() and (g_whole[hi:] == sent).all(), "guard words overwritten"
    return g_whole[lo:hi], d_displs.cpu().numpy(), int(d_status.item()), c_out, c_displs, c_status


def test_config4_gather():
    P = 256
    counts = inputs.gather_counts(1004, P)
    bufs = inputs.gather_buffers(1004, counts)
    arrived = inputs.bernoulli_mask(2004, 0, P, 1, 0.8)[:, 0]
    g, gd, gs, c, cd, cs = gather_both(bufs, counts, ec.I64, arrived)
    assert gs == 0 and cs == 0
    assert np.array_equal(gd, cd) and gd[0] == 0 and np.array_equal(gd[1:], np.cumsum(counts))
    assert np.array_equal(g, c)
    # the late ranks arrive: one more call with only their bits completes the concatenation
    total = int(counts.sum())
    d_out = to_dev(g.copy())
    d_bufs = [to_dev(b) for b in bufs]
    d_displs = torch.empty(P + 1, dtype=torch.int64, device="cuda")
    d_status = torch.empty(1, dtype=torch.int32, device="cuda")
    late = inputs.pack_mask((~arrived)[:, None]).reshape(-1)
    ec.allgatherv(d_bufs, to_dev(counts), ec.I64, to_dev(late), d_displs, d_out, d_status)
    torch.cuda.synchronize()
    assert np.array_equal(to_host(d_out), np.concatenate(bufs)) and total == d_out.numel()


@pytest.mark.parametrize("P", [1, 2, 63, 64, 65, 255, 256, 1024])
def test_rank_counts_and_all_arrived(P):
    rng = np.random.default_rng(P)
    counts = rng.integers(0, 300, size=P).astype(np.int64)      # zero-length contributions included
    bufs = [rng.integers(-2 ** 63, 2 ** 63 - 1, size=int(c), dtype=np.int64) for c in counts]
    if counts.sum() == 0:
        counts[0] = 5
        bufs[0] = np.arange(5, dtype=np.int64)
    g, gd, gs, c, cd, cs = gather_both(bufs, counts, ec.I64, None)
    assert gs == 0 and np.array_equal(gd, cd) and np.array_equal(g, c)
    assert np.array_equal(g, np.concatenate(bufs))
    arrived = rng.random(P) < 0.5
    g, gd, gs, c, cd, cs = gather_both(bufs, counts, ec.I64, arrived, offset=1)
    assert gs == 0 and np.array_equal(gd, cd) and np.array_equal(g, c)


@pytest.mark.parametrize("dtype", [ec.F32, ec.BF16, ec.I64, ec.F64])
def test_element_sizes_and_odd_offsets(dtype):
    P = 40
    rng = np.random.default_rng(3)
    counts = rng.integers(1, 5000, size=P).astype(np.int64)
    counts[::3] |= 1                                             # odd counts: slots start at every phase modulo 16 bytes
    npdt = NP[dtype]
    if npdt == np.uint16:
        bufs = [rng.integers(0, 65535, size=int(c)).astype(np.uint16) for c in counts]
    elif npdt == np.int64:
        bufs = [rng.integers(-2 ** 63, 2 ** 63 - 1, size=int(c), dtype=np.int64) for c in counts]
    else:
        bufs = [rng.standard_normal(int(c)).astype(npdt) for c in counts]
    arrived = rng.random(P) < 0.7
    for off in (0, 1, 3):
        g, gd, gs, c, cd, cs = gather_both(bufs, counts, dtype, arrived, offset=off)
        assert gs == 0 and np.array_equal(gd, cd)
        assert np.array_equal(g.view(np.uint8), c.view(np.uint8))


def test_capacity_exceeded_writes_nothing():
    counts = np.array([500, 600, 700], dtype=np.int64)
    bufs = [np.arange(int(c), dtype=np.int64) for c in counts]
    g, gd, gs, c, cd, cs = gather_both(bufs, counts, ec.I64, None, capacity=1799)
    assert gs != 0 and cs != 0
    assert np.array_equal(gd, cd)
    assert (g == SENT).all()
    # exactly enough is fine
    g, gd, gs, c, cd, cs = gather_both(bufs, counts, ec.I64, None, capacity=1800)
    assert gs == 0 and np.array_equal(g, c)


def test_large_contributions_span_many_chunks():
    counts = np.array([1 << 20, 3, (1 << 19) + 5], dtype=np.int64)
    bufs = inputs.gather_buffers(9, counts)
    g, gd, gs, c, cd, cs = gather_both(bufs, counts, ec.I64, [True, False, True])
    assert gs == 0 and np.array_equal(g, c)


@pytest.mark.parametrize("P", [3, 64, 200])
def test_compact_variant_matches_checker(P):
    rng = np.random.default_rng(40 + P)
    counts = rng.integers(0, 3000, size=P).astype(np.int64)
    bufs = [rng.integers(-2 ** 63, 2 ** 63 - 1, size=int(c), dtype=np.int64) for c in counts]
    arrived = rng.random(P) < 0.6
    mask = inputs.pack_mask(arrived[:, None]).reshape(-1)
    cap = int(counts.sum())
    c_out = np.full(cap, SENT, dtype=np.int64)
    c_displs, c_status = oracle.allgatherv(bufs, counts, mask, c_out, compact=True)
    d_out = to_dev(np.full(cap, SENT, dtype=np.int64))
    d_displs = torch.empty(P + 1, dtype=torch.int64, device="cuda")
    d_status = torch.empty(1, dtype=torch.int32, device="cuda")
    ec.allgatherv([to_dev(b) for b in bufs], to_dev(counts), ec.I64, to_dev(mask), d_displs, d_out, d_status, compact=True)
    torch.cuda.synchronize()
    assert int(d_status.item()) == 0 == c_status
    assert np.array_equal(d_displs.cpu().numpy(), c_displs)
    assert np.array_equal(to_host(d_out), c_out)
