"""Helpers shared by the GPU parity tests: run the same schedule through the CUDA
library (via its C ABI binding) and through the CPU checker, compare bit for bit."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2203_17063_b200 import binding as ec
from paper_2203_17063_b200 import inputs

NP_IN = {ec.F32: np.float32, ec.BF16: np.uint16, ec.I64: np.int64, ec.F64: np.float64}
NP_OUT = {ec.F32: np.float32, ec.BF16: np.float32, ec.I64: np.int64, ec.F64: np.float64}
BITS = {np.dtype(np.float32): np.uint32, np.dtype(np.float64): np.uint64, np.dtype(np.int64): np.int64}


def bits(a: np.ndarray) -> np.ndarray:
    return a.view(BITS[a.dtype])


def to_dev(a: np.ndarray, offset_elems: int = 0) -> torch.Tensor:
    """Upload a numpy array; with offset_elems > 0 the tensor starts that many
    elements into a fresh allocation (to misalign it on purpose)."""
    if a.dtype == np.uint16:
        t = torch.from_numpy(a.view(np.int16)).view(torch.bfloat16)
    elif a.dtype == np.uint64:
        t = torch.from_numpy(a.view(np.int64))
    elif a.dtype == np.uint32:
        t = torch.from_numpy(a.view(np.int32))
    else:
        t = torch.from_numpy(a)
    if offset_elems == 0:
        return t.cuda()
    big = torch.empty(t.numel() + offset_elems, dtype=t.dtype, device="cuda")
    view = big[offset_elems:]
    view.copy_(t)
    return view


def to_host(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    return t.cpu().numpy()


def sentinel(dtype_out, n):
    if dtype_out == np.int64:
        return np.full(n, -0x0123456789ABCDEF, dtype=np.int64)
    return np.full(n, np.nan, dtype=dtype_out)


GUARD = 64          # guard elements on either side of an output (256 or 512 bytes: alignment is kept)
GUARD_COUNT = 0x5EA1ED


def guarded(values: np.ndarray, offset_elems: int = 0):
    """Upload `values` with GUARD sentinel elements before and after it (compute-sanitizer's stand-in: a kernel that
    writes outside its output is caught by check_guards).  Returns (whole allocation, view of the values)."""
    t = torch.from_numpy(values)
    lead = GUARD + offset_elems
    big = torch.empty(lead + t.numel() + GUARD, dtype=t.dtype, device="cuda")
    fill = GUARD_COUNT if not t.dtype.is_floating_point else float("inf")
    big.fill_(fill)
    view = big[lead:lead + t.numel()]
    view.copy_(t)
    return big, view


def check_guards(big: torch.Tensor, view: torch.Tensor, what: str) -> None:
    lead = view.storage_offset() - big.storage_offset()
    fill = GUARD_COUNT if not big.dtype.is_floating_point else float("inf")
    ok = bool((big[:lead] == fill).all()) and bool((big[lead + view.numel():] == fill).all())
    assert ok, f"{what}: bytes outside the output were written"


def run_schedule(P, n, seg, dtype, op, bufs, masks, order=ec.ORDER_FIXED, offset_elems=0, result_offset=0,
                 tile=None, poison=None, oracle_threads=4, compare=True, path=None):
    """Apply the cumulative masks one round after the other on GPU and CPU.

    masks: list of uint64 [S][W] arrays (or None = everything arrived).
    poison: optional boolean [P][S] per round list; where True the GPU's copy of
    that (rank, segment) is overwritten with NaN / a byte pattern before the round.
    Returns the list of (gpu_result, gpu_count, cpu_result, cpu_count) per round.
    """
    S = (n + seg - 1) // seg
    ar = ec.Allreduce(P, n, dtype, op, seg, order)
    if tile is not None:
        ar.set_tile(*tile)
    if path is not None:
        ar.set_path(path)
    ref = oracle.Allreduce(P, n, dtype, op, seg)
    d_bufs = [to_dev(b, offset_elems) for b in bufs]
    res_np = sentinel(NP_OUT[dtype], n)
    res_all, d_res = guarded(res_np.copy(), result_offset)
    cnt_all, d_cnt = guarded(np.full(S, 0xFFFFFFF, dtype=np.int32))
    c_res = res_np.copy()
    c_cnt = np.full(S, 0xFFFFFFF, dtype=np.uint32)
    out = []
    for t, m in enumerate(masks):
        if poison is not None:
            for r in range(P):
                pb = bufs[r].copy()
                sel = np.repeat(poison[t][r], seg)[:n]
                if pb.dtype == np.int64:
                    pb[sel] = 0x5A5A5A5A5A5A5A5A
                elif pb.dtype == np.uint16:
                    pb[sel] = 0x7FC0                      # bf16 NaN
                else:
                    pb[sel] = np.nan
                d_bufs[r].copy_(to_dev(pb))
        d_mask = None if m is None else to_dev(np.ascontiguousarray(m, dtype=np.uint64))
        ar.apply(d_bufs, d_mask, d_res, d_cnt)
        torch.cuda.synchronize()
        check_guards(res_all, d_res, f"round {t}: result")
        check_guards(cnt_all, d_cnt, f"round {t}: contrib_count")
        ref.apply(bufs, m, c_res, c_cnt, order=order, threads=oracle_threads)
        g_res = to_host(d_res)
        g_cnt = d_cnt.cpu().numpy().view(np.uint32)
        if compare:
            assert np.array_equal(g_cnt, c_cnt), f"round {t}: contributor counts differ"
            same = bits(g_res) == bits(c_res)
            if not same.all():
                bad = np.nonzero(~same)[0]
                raise AssertionError(f"round {t}: {bad.size} of {n} elements differ, first at {bad[0]}: "
                                     f"gpu {g_res[bad[0]]!r} cpu {c_res[bad[0]]!r}")
        out.append((g_res.copy(), g_cnt.copy(), c_res.copy(), c_cnt.copy()))
    ar.destroy()
    return out


def random_rounds(seed, P, S, p_first, last_round=3):
    return inputs.arrival_rounds(seed, P, S, p_first, last_round)
