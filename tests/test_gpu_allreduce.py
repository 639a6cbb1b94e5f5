"""GPU parity of ec_allreduce_* against the CPU checker, element by element, through the C ABI."""
import math

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle
from paper_2203_17063_b200 import inputs
from tests.gpu_util import NP_OUT, bits, ec, run_schedule, sentinel, to_dev, to_host


@pytest.fixture(autouse=True)
def _need_gpu(cuda_device):
    yield


def _bufs(kind, seed, P, n, **kw):
    return inputs.rank_buffers(kind, seed, P, n, **kw)


# ---------------------------------------------------------------------------
# the five workloads, reduced (several tiles, a ragged tail) and at full size
# ---------------------------------------------------------------------------
def test_config1_all_arrived_fixed_order_bit_exact():
    P, n, seg = 4, 1 << 20, 16384
    bufs = _bufs("uniform_f32", 1001, P, n)
    (g, gc, c, cc), = run_schedule(P, n, seg, ec.F32, ec.SUM, bufs, [None])
    assert (gc == P).all()
    # all arrived: the result is the plain rank-order sum
    acc = np.zeros(n, dtype=np.float32)
    for b in bufs:
        acc = acc + b
    assert np.array_equal(bits(g), bits(acc))
    # and the same with an explicit all-ones mask
    S = n // seg
    run_schedule(P, n, seg, ec.F32, ec.SUM, bufs, [np.full((S, 1), 0xF, dtype=np.uint64)])


@pytest.mark.parametrize("n,seg", [((1 << 20) + 37, 65536), (1 << 24, 65536)], ids=["reduced", "full"])
def test_config2_three_rounds(n, seg):
    P = 16
    S = (n + seg - 1) // seg
    bufs = _bufs("normal_f32", 1002, P, n)
    rounds = inputs.arrival_rounds(2002, P, S, 0.7)
    masks = inputs.cumulative_masks(rounds)
    outs = run_schedule(P, n, seg, ec.F32, ec.SUM, bufs, masks, oracle_threads=8)
    g, gc, _, _ = outs[-1]
    assert (gc == P).all()
    # final result equals the one-shot fold in canonical order (round of arrival, rank)
    order = np.argsort(rounds.T.astype(np.int32) * 1024 + np.arange(P)[None, :], axis=1, kind="stable").astype(np.int32)
    one = oracle.allreduce_oneshot(bufs, oracle.F32, oracle.SUM, seg, order)
    assert np.array_equal(bits(g), bits(one))
    # and sits within the sequential-summation bound of the double sum
    if n <= (1 << 21):
        ref, mag = oracle.allreduce_ref64(bufs, oracle.F32, seg, None)
        assert (np.abs(g.astype(np.float64) - ref) <= (P - 1) * 2.0 ** -24 * mag * 1.01).all()


@pytest.mark.parametrize("n,seg", [((1 << 21) + 8 * 13, 131072), (1 << 25, 131072)], ids=["reduced", "full"])
def test_config3_bf16_fixed_and_pairwise(n, seg):
    P = 32
    S = (n + seg - 1) // seg
    bufs = _bufs("normal_bf16", 1003, P, n, sigma=1e-3)
    rounds = inputs.arrival_rounds(2003, P, S, 0.9)
    masks = inputs.cumulative_masks(rounds)
    outs = run_schedule(P, n, seg, ec.BF16, ec.SUM, bufs, masks, oracle_threads=8)
    assert (outs[-1][1] == P).all()
    # pairwise variant: tolerance gate against the double-precision sum, on the round-1 subset and all-at-once
    for m in (masks[0], None):
        (g, gc, c, cc), = run_schedule(P, n, seg, ec.BF16, ec.SUM, bufs, [m], order=ec.ORDER_PAIRWISE,
                                       oracle_threads=8, compare=False)
        assert np.array_equal(gc, cc)
        ref, mag = oracle.allreduce_ref64(bufs, oracle.BF16, seg, m)
        tol = 1e-5 * math.log2(P) * mag
        assert (np.abs(g.astype(np.float64) - ref) <= tol).all()
        assert np.abs(g - ref).max() <= 1e-5 * math.log2(P) * np.abs(ref).max()
        # the tree is the checker's tree: same bits
        assert np.array_equal(bits(g), bits(c))


@pytest.mark.parametrize("op", [ec.SUM, ec.MAX])
def test_config4_int64_reductions(op):
    P, n, seg = 256, 1 << 20, 8192
    S = n // seg
    bufs = _bufs("int64_below", 1004, P, n, bound=1 << 20)
    rounds = inputs.arrival_rounds(2004, P, S, 0.8, last_round=2)
    masks = inputs.cumulative_masks(rounds)
    outs = run_schedule(P, n, seg, ec.I64, op, bufs, masks, oracle_threads=8)
    g = outs[-1][0]
    stack = np.stack(bufs)
    assert np.array_equal(g, stack.sum(0) if op == ec.SUM else stack.max(0))


def test_int64_full_range_wraps():
    P, n, seg = 7, 50000, 4096
    bufs = _bufs("int64_full", 5, P, n)
    S = (n + seg - 1) // seg
    masks = inputs.cumulative_masks(inputs.arrival_rounds(6, P, S, 0.5))
    for op in (ec.SUM, ec.MAX, ec.MIN):
        run_schedule(P, n, seg, ec.I64, op, bufs, masks)


# ---------------------------------------------------------------------------
# edge cases
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("P", [1, 2, 63, 64, 65, 128, 255, 256, 1024])
def test_rank_counts_at_word_boundaries(P):
    n, seg = 3000, 256
    S = (n + seg - 1) // seg
    bufs = _bufs("normal_f32", 100 + P, P, n)
    rounds = inputs.arrival_rounds(200 + P, P, S, 0.6)
    masks = inputs.cumulative_masks(rounds)
    # garbage above bit P-1 must change nothing
    if P % 64:
        junk = np.uint64(((1 << 64) - 1) ^ ((1 << (P % 64)) - 1))
        masks = [m.copy() for m in masks]
        for m in masks:
            m[:, -1] |= junk
    poison = [rounds > t for t in (1, 2, 3)]
    run_schedule(P, n, seg, ec.F32, ec.SUM, bufs, masks, poison=poison)


@pytest.mark.parametrize("dtype,kind", [(ec.F32, "normal_f32"), (ec.BF16, "normal_bf16"), (ec.I64, "int64_full"),
                                        (ec.F64, "f64")])
@pytest.mark.parametrize("op", [ec.SUM, ec.MAX, ec.MIN])
def test_every_dtype_and_op(dtype, kind, op):
    P, n, seg = 5, 10000, 1024
    S = (n + seg - 1) // seg
    if kind == "f64":
        bufs = [np.random.default_rng(r).standard_normal(n) for r in range(P)]
    else:
        bufs = _bufs(kind, 300, P, n)
    rounds = inputs.arrival_rounds(301, P, S, 0.5)
    rounds[:, 2] = 3                                   # a segment that is empty until the last round
    masks = inputs.cumulative_masks(rounds)
    run_schedule(P, n, seg, dtype, op, bufs, masks, poison=[rounds > t for t in (1, 2, 3)])


@pytest.mark.parametrize("n,seg,off,roff", [
    (1000, 64, 0, 0),        # aligned, vector path, n % seg != 0
    (1000, 63, 0, 0),        # segment size not a multiple of the vector width: element-wise path
    (1000, 64, 1, 0),        # rank buffers one element off 16-byte alignment
    (1000, 64, 0, 1),        # result one element off
    (50, 64, 0, 0),          # n < seg: a single short segment
    (1001, 1, 0, 0),         # one element per segment
    (4099, 4096, 0, 0),      # short last segment of 3 elements
    (4103, 4100, 0, 0),      # vector path with a ragged tail inside every segment? (4100 % 4 == 0)
])
@pytest.mark.parametrize("dtype,kind", [(ec.F32, "normal_f32"), (ec.BF16, "normal_bf16"), (ec.I64, "int64_full")])
def test_alignment_and_ragged_shapes(n, seg, off, roff, dtype, kind):
    P = 6
    S = (n + seg - 1) // seg
    bufs = _bufs(kind, 400, P, n)
    rounds = inputs.arrival_rounds(401 + n, P, S, 0.5)
    masks = inputs.cumulative_masks(rounds)
    run_schedule(P, n, seg, dtype, ec.SUM, bufs, masks, offset_elems=off, result_offset=roff)
    run_schedule(P, n, seg, dtype, ec.SUM, bufs, masks, offset_elems=off, result_offset=roff, tile=(64, 96))


@pytest.mark.parametrize("tile", [(64, 4), (128, 1000), (256, 1 << 16), (256, 12)])
def test_tile_shapes_do_not_change_results(tile):
    P, n, seg = 9, 70001, 9000
    S = (n + seg - 1) // seg
    bufs = _bufs("normal_f32", 500, P, n)
    masks = inputs.cumulative_masks(inputs.arrival_rounds(501, P, S, 0.4))
    run_schedule(P, n, seg, ec.F32, ec.SUM, bufs, masks, tile=tile)
    run_schedule(P, n, seg, ec.F32, ec.SUM, bufs, masks[:1], tile=tile, order=ec.ORDER_PAIRWISE)


@pytest.mark.parametrize("P", [1, 2, 3, 4, 5, 8, 9, 16, 31, 64, 100, 300])
def test_pairwise_tree_matches_checker_bits(P):
    n, seg = 2100, 512
    S = (n + seg - 1) // seg
    bufs = _bufs("normal_f32", 600 + P, P, n)
    masks = inputs.cumulative_masks(inputs.arrival_rounds(601 + P, P, S, 0.6))
    outs = run_schedule(P, n, seg, ec.F32, ec.SUM, bufs, masks, order=ec.ORDER_PAIRWISE)
    ref, mag = oracle.allreduce_ref64(bufs, oracle.F32, seg, None)
    g = outs[-1][0]
    # three rounds, each a tree plus one add: error below (ceil(log2 P) + 3) rounding units of sum|x|
    assert (np.abs(g - ref) <= (math.ceil(math.log2(max(P, 2))) + 3) * 2.0 ** -24 * mag * 1.01).all()
    # bf16 and fp64 inputs through the same tree
    b16 = _bufs("normal_bf16", 700 + P, P, n, sigma=1.0)
    run_schedule(P, n, seg, ec.BF16, ec.SUM, b16, masks, order=ec.ORDER_PAIRWISE)
    f64 = [np.random.default_rng(P * 10 + r).standard_normal(n) for r in range(P)]
    run_schedule(P, n, seg, ec.F64, ec.SUM, f64, masks, order=ec.ORDER_PAIRWISE)
    if P <= 64:
        # up to 64 ranks the tree is walked out of bulk-staged tiles by default; the direct-load kernel must give the same bits
        run_schedule(P, n, seg, ec.F32, ec.SUM, bufs, masks, order=ec.ORDER_PAIRWISE, path=0)
        run_schedule(P, n, seg, ec.BF16, ec.SUM, b16, masks, order=ec.ORDER_PAIRWISE, path=0)
        # ... and a misaligned call (element-wise tree) and a tile with a ragged tail of single elements
        run_schedule(P, n, seg, ec.F32, ec.SUM, bufs, masks, order=ec.ORDER_PAIRWISE, offset_elems=1)
        run_schedule(P, n - 3, seg - 1, ec.F32, ec.SUM, [b[:n - 3] for b in bufs], masks, order=ec.ORDER_PAIRWISE)


def test_signed_zero_and_identity_rules():
    n, seg = 64, 16
    z = np.full(n, -0.0, dtype=np.float32)
    outs = run_schedule(2, n, seg, ec.F32, ec.SUM, [z, z], [None])
    assert not np.signbit(outs[0][0]).any()            # +0.0 + (-0.0) = +0.0
    outs = run_schedule(2, n, seg, ec.F32, ec.MAX, [z, z], [None])
    assert np.signbit(outs[0][0]).all()                # -0.0 > -inf
    outs = run_schedule(2, n, seg, ec.F32, ec.SUM, [z, z], [None], order=ec.ORDER_PAIRWISE)
    assert np.signbit(outs[0][0]).all()                # the tree adds -0.0 + -0.0 and nothing else
    # nothing arrives in the first apply: identities everywhere, counts zero
    none = np.zeros((4, 1), dtype=np.uint64)
    for op, ident in ((ec.SUM, 0.0), (ec.MAX, -np.inf), (ec.MIN, np.inf)):
        (g, gc, c, cc), = run_schedule(2, n, seg, ec.F32, op, [z, z], [none])
        assert (g == ident).all() and (gc == 0).all()
    (g, gc, _, _), = run_schedule(2, n, seg, ec.I64, ec.MAX, [np.zeros(n, np.int64)] * 2, [none])
    assert (g == np.iinfo(np.int64).min).all()


def test_idempotence_regress_reset_and_untouched_segments():
    P, n, seg = 10, 5000, 500
    S = 10
    bufs = _bufs("normal_f32", 800, P, n)
    rounds = inputs.arrival_rounds(801, P, S, 0.5)
    rounds[:, 4] = 1                                   # segment 4 complete after round 1: idle afterwards
    masks = inputs.cumulative_masks(rounds)
    ar = ec.Allreduce(P, n, ec.F32, ec.SUM, seg)
    d_bufs = [to_dev(b) for b in bufs]
    d_res = to_dev(sentinel(np.float32, n))
    d_cnt = torch.zeros(S, dtype=torch.int32, device="cuda")
    d_masks = [to_dev(m) for m in masks]
    ar.apply(d_bufs, d_masks[0], d_res, d_cnt)
    first = to_host(d_res).copy()
    assert not np.isnan(first).any()
    # same mask again: not a byte changes
    ar.apply(d_bufs, d_masks[0], d_res, d_cnt)
    assert np.array_equal(bits(to_host(d_res)), bits(first))
    # scribble into the idle segment: later applies must neither read nor write it
    d_res[4 * seg:5 * seg] = 12345.0
    ar.apply(d_bufs, d_masks[1], d_res, d_cnt)
    assert (to_host(d_res)[4 * seg:5 * seg] == 12345.0).all()
    # a mask with bits cleared (regress) un-applies nothing
    before = to_host(d_res).copy()
    cnt_before = d_cnt.cpu().numpy().copy()
    ar.apply(d_bufs, to_dev(np.zeros_like(masks[0])), d_res, d_cnt)
    assert np.array_equal(bits(to_host(d_res)), bits(before))
    assert np.array_equal(d_cnt.cpu().numpy(), cnt_before)
    ar.apply(d_bufs, d_masks[2], d_res, None)          # contrib_count may be NULL
    # new epoch: the same schedule reproduces the same bits
    runs = []
    for _ in range(2):
        ar.reset()
        d_res.copy_(to_dev(sentinel(np.float32, n)))
        for m in d_masks:
            ar.apply(d_bufs, m, d_res, d_cnt)
        runs.append(to_host(d_res).copy())
    assert np.array_equal(bits(runs[0]), bits(runs[1]))
    ref = oracle.Allreduce(P, n, oracle.F32, oracle.SUM, seg)
    c = sentinel(np.float32, n)
    for m in masks:
        ref.apply(bufs, m, c, None)
    assert np.array_equal(bits(runs[0]), bits(c))
    ar.destroy()


def test_argument_errors_on_device():
    n, seg, P = 1000, 100, 3
    ar = ec.Allreduce(P, n, ec.F32, ec.SUM, seg)
    bufs = [torch.zeros(n, device="cuda") for _ in range(P)]
    res = torch.zeros(n, device="cuda")
    L = ec.lib()
    tbl = (ec.C.c_void_p * P)(*[b.data_ptr() for b in bufs])
    st = torch.cuda.current_stream().cuda_stream
    assert L.ec_allreduce_apply(ar._h, tbl, P + 1, n, ec.F32, ec.SUM, seg, None, res.data_ptr(), None, st) == ec.ERR_INVALID
    assert L.ec_allreduce_apply(ar._h, tbl, P, n, ec.I64, ec.SUM, seg, None, res.data_ptr(), None, st) == ec.ERR_INVALID
    assert L.ec_allreduce_apply(ar._h, tbl, P, n, ec.F32, ec.SUM, seg, None, bufs[1].data_ptr(), None, st) == ec.ERR_INVALID
    assert L.ec_allreduce_apply(ar._h, tbl, P, n, ec.F32, ec.SUM, seg, None, None, None, st) == ec.ERR_INVALID
    assert L.ec_allreduce_apply(ar._h, tbl, P, n, ec.F32, ec.SUM, seg, None, res.data_ptr(), None, st) == ec.OK
    torch.cuda.synchronize()
    with pytest.raises(ec.EcError):
        ec.Allreduce(P, n, ec.I64, ec.SUM, seg, ec.ORDER_PAIRWISE)
    ar.destroy()


def test_library_allocated_workspace():
    """init with workspace = NULL lets the library allocate; results are the same."""
    import ctypes as C
    L = ec.lib()
    P, n, seg = 4, 4096, 512
    bufs = _bufs("normal_f32", 900, P, n)
    d_bufs = [to_dev(b) for b in bufs]
    h = C.c_void_p()
    assert L.ec_allreduce_init(C.byref(h), P, n, ec.F32, ec.SUM, seg, ec.ORDER_FIXED, None, 0) == ec.OK
    res = torch.empty(n, device="cuda")
    tbl = (C.c_void_p * P)(*[b.data_ptr() for b in d_bufs])
    assert L.ec_allreduce_apply(h, tbl, P, n, ec.F32, ec.SUM, seg, None, res.data_ptr(), None,
                                torch.cuda.current_stream().cuda_stream) == ec.OK
    torch.cuda.synchronize()
    ref = oracle.Allreduce(P, n, oracle.F32, oracle.SUM, seg)
    c = np.empty(n, dtype=np.float32)
    ref.apply(bufs, None, c, None)
    assert np.array_equal(bits(to_host(res)), bits(c))
    assert L.ec_allreduce_destroy(h) == ec.OK


@pytest.mark.parametrize("P,n,seg", [(4, 1 << 16, 1024), (16, 1 << 20, 4096), (70, 70 * 3000, 1000), (5, 100, 10), (256, 256 * 512, 512)])
def test_ring_order_matches_checker_bits(P, n, seg):
    """EC_ORDER_RING: chunk c of the vector is folded over the ranks c, c+1, ..., c-1 (Scatter-Reduce of the ring)."""
    S = (n + seg - 1) // seg
    bufs = _bufs("normal_f32", 950 + P, P, n)
    masks = inputs.cumulative_masks(inputs.arrival_rounds(951 + P, P, S, 0.6))
    run_schedule(P, n, seg, ec.F32, ec.SUM, bufs, masks, order=ec.ORDER_RING)
    run_schedule(P, n, seg, ec.F32, ec.SUM, bufs, [None], order=ec.ORDER_RING, tile=(64, 96))
    b16 = _bufs("normal_bf16", 960 + P, P, n, sigma=1.0)
    run_schedule(P, n, seg, ec.BF16, ec.SUM, b16, masks, order=ec.ORDER_RING)


def test_ring_order_needs_segments_inside_chunks():
    with pytest.raises(ec.EcError) as err:
        ec.Allreduce(4, 1000, ec.F32, ec.SUM, 64, ec.ORDER_RING)        # ceil(1000/4) = 250 is not a multiple of 64
    assert err.value.code == ec.ERR_INVALID


# ---------------------------------------------------------------------------
# the whole epoch from host memory in one call (uploads, reset, applies, read-back)
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("dtype,kind,kw", [(ec.F32, "normal_f32", {}), (ec.BF16, "normal_bf16", {"sigma": 1.0})],
                         ids=["f32", "bf16"])
def test_epoch_from_host_buffers_matches_round_by_round_checker(dtype, kind, kw):
    P, n, seg = 16, (1 << 18) + 24, 8192
    S = (n + seg - 1) // seg
    bufs = _bufs(kind, 1010, P, n, **kw)
    rounds = inputs.arrival_rounds(2010, P, S, 0.6)
    masks = inputs.cumulative_masks(rounds)
    ref = oracle.Allreduce(P, n, dtype, ec.SUM, seg)
    c_res = sentinel(NP_OUT[dtype], n)
    c_cnt = np.zeros(S, dtype=np.uint32)
    for m in masks:
        ref.apply(bufs, m, c_res, c_cnt)
    ar = ec.Allreduce(P, n, dtype, ec.SUM, seg)
    h_bufs = [torch.from_numpy(b.view(np.int16) if b.dtype == np.uint16 else b).pin_memory() for b in bufs]
    h_masks = [torch.from_numpy(np.ascontiguousarray(m, dtype=np.uint64).view(np.int64)).pin_memory() for m in masks]
    h_res = torch.from_numpy(sentinel(NP_OUT[dtype], n)).pin_memory()
    h_cnt = torch.full((S,), -1, dtype=torch.int32).pin_memory()
    staging = torch.empty(ar.host_staging_bytes(len(masks)), dtype=torch.uint8, device="cuda")
    for _ in range(2):                                   # a second epoch on the same context and staging area
        h_res.fill_(float("nan"))
        ar.epoch_host(h_bufs, h_masks, h_res, h_cnt, staging)
        torch.cuda.synchronize()
        assert np.array_equal(h_cnt.numpy().view(np.uint32), c_cnt)
        assert np.array_equal(bits(h_res.numpy()), bits(c_res))
    small = torch.empty(ar.host_staging_bytes(len(masks)) - 256, dtype=torch.uint8, device="cuda")
    with pytest.raises(ec.EcError) as err:
        ar.epoch_host(h_bufs, h_masks, h_res, h_cnt, small)
    assert err.value.code == ec.ERR_CAPACITY
    ar.destroy()


# ---------------------------------------------------------------------------
# short segments with many ranks: one block per segment, contributions staged in shared memory
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("P,seg_vectors", [(5, 1), (8, 9), (64, 9), (64, 32), (48, 25), (200, 64), (200, 3), (1024, 2)])
@pytest.mark.parametrize("dtype,kind,kw", [(ec.F32, "normal_f32", {}), (ec.BF16, "normal_bf16", {"sigma": 1.0}),
                                           (ec.I64, "int64_full", {}), (ec.F64, "normal_f64", {})],
                         ids=["f32", "bf16", "i64", "f64"])
def test_short_segments_many_ranks(P, seg_vectors, dtype, kind, kw):
    per_vec = {ec.F32: 4, ec.BF16: 8, ec.I64: 2, ec.F64: 2}[dtype]
    seg = seg_vectors * per_vec
    S = 37
    n = (S - 1) * seg + max(1, seg - per_vec - 1)        # the last segment is short and ends inside a vector
    if kind == "normal_f64":
        bufs = [b.astype(np.float64) * (1.0 + 2.0 ** -30) for b in _bufs("normal_f32", 3000 + P, P, n)]
    else:
        bufs = _bufs(kind, 3000 + P, P, n, **kw)
    rounds = inputs.arrival_rounds(3100 + P + seg_vectors, P, S, 0.5)
    masks = inputs.cumulative_masks(rounds)
    poison = [rounds > t for t in (1, 2, 3)]
    run_schedule(P, n, seg, dtype, ec.SUM, bufs, masks, poison=poison)
    if dtype != ec.BF16:
        run_schedule(P, n, seg, dtype, ec.MAX, bufs, [masks[0], None])


def test_short_segments_ring_order_and_untouched_rows():
    P, seg, S = 16, 36, 64                                # one centroid-like row of 36 floats per segment
    n = seg * S                                           # ceil(n / P) = 144 = 4 segments per ring chunk
    bufs = _bufs("normal_f32", 3200, P, n)
    rounds = inputs.arrival_rounds(3201, P, S, 0.4)
    rounds[:, 5] = 3                                      # a segment nobody reaches before the last round
    rounds[:, 6] = 1                                      # and one that is complete at once
    masks = inputs.cumulative_masks(rounds)
    run_schedule(P, n, seg, ec.F32, ec.SUM, bufs, masks, order=ec.ORDER_RING)
    outs = run_schedule(P, n, seg, ec.F32, ec.SUM, bufs, masks + [masks[-1]])
    assert np.array_equal(bits(outs[-1][0]), bits(outs[-2][0]))          # nothing new: nothing changes


# ---------------------------------------------------------------------------
# the optional path that stages the rank tiles through shared memory with bulk asynchronous copies
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("dtype,kind,kw", [(ec.F32, "normal_f32", {}), (ec.BF16, "normal_bf16", {"sigma": 1.0}),
                                           (ec.I64, "int64_full", {})], ids=["f32", "bf16", "i64"])
@pytest.mark.parametrize("P,n,seg", [(16, (1 << 18) + 37 * 8, 65536), (3, 9000, 3000), (64, 1 << 16, 4096), (7, 20000, 20000)])
def test_bulk_copy_path_matches_checker(dtype, kind, kw, P, n, seg):
    S = (n + seg - 1) // seg
    bufs = _bufs(kind, 4000 + P, P, n, **kw)
    rounds = inputs.arrival_rounds(4100 + P, P, S, 0.6)
    masks = inputs.cumulative_masks(rounds)
    poison = [rounds > t for t in (1, 2, 3)]
    run_schedule(P, n, seg, dtype, ec.SUM, bufs, masks, poison=poison, path=1)
    run_schedule(P, n, seg, dtype, ec.MAX if dtype != ec.BF16 else ec.SUM, bufs, [masks[0], None], path=1)


def test_bulk_copy_path_ring_order_misaligned_and_limits():
    P, n, seg = 16, 1 << 16, 1024
    bufs = _bufs("normal_f32", 4200, P, n)
    masks = inputs.cumulative_masks(inputs.arrival_rounds(4201, P, n // seg, 0.5))
    run_schedule(P, n, seg, ec.F32, ec.SUM, bufs, masks, order=ec.ORDER_RING, path=1)
    run_schedule(P, n, seg, ec.F32, ec.SUM, bufs, masks, offset_elems=1, path=1)      # not 16-byte aligned: default kernel
    ar = ec.Allreduce(100, 4096, ec.F32, ec.SUM, 1024)
    with pytest.raises(ec.EcError) as err:
        ar.set_path(1)                                                                  # more than 64 ranks
    assert err.value.code == ec.ERR_UNSUPPORTED
    ar.destroy()
    ar = ec.Allreduce(8, 4096, ec.F32, ec.SUM, 1024, ec.ORDER_PAIRWISE)
    ar.set_path(0)                                                                      # the pairwise tree has both forms
    ar.set_path(1)
    ar.destroy()
