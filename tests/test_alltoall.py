"""AlltoAll (Sec. IV-B): checker pinned to numpy's transpose and to sentinels (no GPU), then the GPU
kernel against the checker, byte for byte, through the C ABI."""
import numpy as np
import pytest

import oracle


def make(P, B, seed):
    rng = np.random.default_rng(seed)
    send = [rng.integers(0, 256, size=P * B, dtype=np.uint8) for _ in range(P)]
    return send


def words(arrived):          # arrived[d][s]
    P = len(arrived)
    out = np.zeros((P, (P + 63) // 64), dtype=np.uint64)
    for d in range(P):
        for s in range(P):
            if arrived[d][s]:
                out[d, s // 64] |= np.uint64(1 << (s % 64))
    return out


@pytest.mark.parametrize("P,B", [(1, 7), (4, 16), (8, 1), (65, 24), (16, 1000)])
def test_checker_all_arrived_is_a_block_transpose(P, B):
    send = make(P, B, P * 31 + B)
    recv = [np.full(P * B, 0xEE, dtype=np.uint8) for _ in range(P)]
    cnt = oracle.alltoall(send, recv, B, None)
    cube = np.stack(send).reshape(P, P, B)                     # [source][destination][byte]
    assert np.array_equal(np.stack(recv).reshape(P, P, B), np.swapaxes(cube, 0, 1))
    assert (cnt == P).all()


def test_checker_missing_blocks_keep_their_slots():
    P, B = 70, 12
    send = make(P, B, 5)
    rng = np.random.default_rng(6)
    arrived = rng.random((P, P)) < 0.6
    recv = [np.full(P * B, 0xEE, dtype=np.uint8) for _ in range(P)]
    cnt = oracle.alltoall(send, recv, B, words(arrived))
    for d in range(P):
        assert cnt[d] == arrived[d].sum()
        for s in range(P):
            slot = recv[d][s * B:(s + 1) * B]
            if arrived[d, s]:
                assert np.array_equal(slot, send[s][d * B:(d + 1) * B])
            else:
                assert (slot == 0xEE).all()
    # the late blocks complete it
    oracle.alltoall(send, recv, B, words(~arrived))
    assert np.array_equal(np.stack(recv).reshape(P, P, B), np.swapaxes(np.stack(send).reshape(P, P, B), 0, 1))


@pytest.mark.gpu
@pytest.mark.parametrize("P,B,off", [(4, 32768, 0), (16, 32768, 0), (64, 4096, 0), (65, 48, 0), (8, 1, 0), (8, 24, 0),
                                     (16, 1024, 8), (200, 256, 0), (1, 100, 0)])
def test_gpu_matches_checker(cuda_device, P, B, off):
    """Message sizes from the paper's sweep (1 byte to 32 KiB), 4 to 64 ranks and beyond; `off` misaligns the buffers."""
    import torch

    from paper_2203_17063_b200 import binding as ec

    send = make(P, B, 100 + P + B)
    rng = np.random.default_rng(7)
    arrived = rng.random((P, P)) < 0.7
    for mask in (None, words(arrived)):
        recv = [np.full(P * B, 0xEE, dtype=np.uint8) for _ in range(P)]
        cnt = oracle.alltoall(send, recv, B, mask)
        d_send, d_recv = [], []
        for s in send:
            t = torch.empty(P * B + off, dtype=torch.uint8, device="cuda")
            t[off:].copy_(torch.from_numpy(s))
            d_send.append(t[off:])
        for _ in range(P):
            t = torch.full((P * B + off + 16,), 0xEE, dtype=torch.uint8, device="cuda")
            d_recv.append(t)
        d_cnt = torch.full((P,), -1, dtype=torch.int32, device="cuda")
        d_mask = None if mask is None else torch.from_numpy(mask.view(np.int64)).cuda()
        ec.alltoall(d_send, [t[off:off + P * B] for t in d_recv], B, d_mask, d_cnt)
        torch.cuda.synchronize()
        for d in range(P):
            whole = d_recv[d].cpu().numpy()
            assert np.array_equal(whole[off:off + P * B], recv[d])
            assert (whole[:off] == 0xEE).all() and (whole[off + P * B:] == 0xEE).all()      # guards intact
        assert np.array_equal(d_cnt.cpu().numpy().view(np.uint32), cnt)


@pytest.mark.gpu
def test_gpu_argument_errors(cuda_device):
    import torch

    from paper_2203_17063_b200 import binding as ec

    a = [torch.zeros(64, dtype=torch.uint8, device="cuda") for _ in range(2)]
    with pytest.raises(ec.EcError):
        ec.alltoall(a, a, 32)                                   # in place is not allowed
    with pytest.raises(ec.EcError):
        ec.alltoall(a, [torch.zeros(64, dtype=torch.uint8, device="cuda") for _ in range(2)], 0)
