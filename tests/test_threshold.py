"""Threshold variants of Reduce / Broadcast (Sec. III-B): pins of the plain statement in the
checker against what the paper says about the binomial spanning tree, then the library's host
generators against the checker (no GPU), then the status-threshold kernel (GPU)."""
import numpy as np
import pytest

import oracle


def test_binomial_tree_shape_as_the_paper_describes_it():
    # rank 0 is the root; with eight processes it sends to 1, 2 and 4 (the children of p are p + 2^i)
    assert [r for r in range(8) if oracle.bst_parent(r) == 0 and r] == [1, 2, 4]
    assert [oracle.bst_parent(r) for r in range(1, 8)] == [0, 0, 1, 0, 1, 2, 3]
    # the tree works in stages doubling the number of involved processes
    for P in (8, 16, 64):
        involved = [sum(1 for r in range(P) if oracle.bst_stage_of_rank(r) <= k) for k in range(-1, P.bit_length() - 1)]
        assert involved == [1 << i for i in range(P.bit_length())]
        # half of all processes are added on the last stage ...
        last = P.bit_length() - 2
        assert sum(1 for r in range(P) if oracle.bst_stage_of_rank(r) == last) == P // 2
        # ... so a threshold of 75 % behaves exactly like 100 %
        assert oracle.process_threshold_ranks(P, 0.75) == oracle.process_threshold_ranks(P, 1.0) == P
        assert oracle.process_threshold_ranks(P, 0.5) == P // 2
        assert oracle.process_threshold_ranks(P, 0.25) == P // 4
    assert oracle.process_threshold_ranks(8, 0.0) == 0
    assert oracle.process_threshold_ranks(12, 0.6) == 8 and oracle.process_threshold_ranks(12, 0.7) == 12   # P not a power of two


@pytest.mark.parametrize("P,S", [(8, 5), (64, 3), (65, 4), (200, 2), (12, 7)])
@pytest.mark.parametrize("fraction", [0.0, 0.1, 0.25, 0.5, 0.75, 1.0])
def test_library_generators_match_the_checker(P, S, fraction):
    from paper_2203_17063_b200 import binding as ec

    words, ranks = ec.mask_process_threshold(P, S, fraction)
    assert ranks == oracle.process_threshold_ranks(P, fraction)
    assert np.array_equal(words, oracle.process_threshold_mask(P, S, fraction))
    assert np.array_equal(ec.mask_data_fraction(P, S, fraction), oracle.data_fraction_mask(P, S, fraction))


def test_generator_argument_errors():
    from paper_2203_17063_b200 import binding as ec

    for bad in (-0.1, 1.5, float("nan")):
        with pytest.raises(ec.EcError):
            ec.mask_data_fraction(8, 4, bad)
        with pytest.raises(ec.EcError):
            ec.mask_process_threshold(8, 4, bad)


@pytest.mark.gpu
def test_threshold_reduce_on_the_gpu(cuda_device):
    """Reduce with a process threshold and with a data fraction: results and status counts match the
    checker, and the threshold kernel counts the segments that reached it."""
    import torch

    from paper_2203_17063_b200 import binding as ec
    from paper_2203_17063_b200 import inputs
    from tests.gpu_util import bits, to_dev, to_host

    P, n, seg = 16, 100000, 4096
    S = (n + seg - 1) // seg
    bufs = inputs.rank_buffers("normal_f32", 3, P, n)
    d_bufs = [to_dev(b) for b in bufs]
    for words in (ec.mask_process_threshold(P, S, 0.5)[0], ec.mask_data_fraction(P, S, 0.25),
                  ec.mask_process_threshold(P, S, 0.75)[0]):
        ar = ec.Allreduce(P, n, ec.F32, ec.SUM, seg)
        d_res = torch.empty(n, device="cuda")
        d_cnt = torch.empty(S, dtype=torch.int32, device="cuda")
        ar.apply(d_bufs, to_dev(words), d_res, d_cnt)
        ready = torch.full((1,), 99, dtype=torch.int32, device="cuda")
        ref = oracle.Allreduce(P, n, oracle.F32, oracle.SUM, seg)
        c = np.empty(n, dtype=np.float32)
        cc = np.empty(S, dtype=np.uint32)
        ref.apply(bufs, words, c, cc)
        torch.cuda.synchronize()
        assert np.array_equal(bits(to_host(d_res)), bits(c))
        assert np.array_equal(to_host(d_cnt).view(np.uint32), cc)
        for need in (1, P // 2, P):
            ec.threshold_segments(d_cnt, need, ready)
            torch.cuda.synchronize()
            assert int(ready.item()) == oracle.threshold_segments(cc, need)
        ar.destroy()
