"""Thin ctypes binding of ``libec_b200.so`` (the C ABI of ``include/ec.h``).

Argument marshalling only: every step of the collectives runs in the CUDA
kernels of the library.  PyTorch supplies device memory and streams.  There is
no CPU fallback: if the library cannot be loaded, importing a symbol raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libec_b200.so")

F32, BF16, I64, F64 = 0, 1, 2, 3
SUM, MAX, MIN = 0, 1, 2
ORDER_FIXED, ORDER_PAIRWISE, ORDER_RING = 0, 1, 2
MAX_RANKS = 1024

OK, ERR_INVALID, ERR_UNSUPPORTED, ERR_CUDA, ERR_STATE, ERR_CAPACITY = 0, -1, -2, -3, -4, -5

IN_TORCH = {F32: torch.float32, BF16: torch.bfloat16, I64: torch.int64, F64: torch.float64}
OUT_TORCH = {F32: torch.float32, BF16: torch.float32, I64: torch.int64, F64: torch.float64}

# every symbol include/ec.h declares: (restype, argtypes)
_vp, _sz, _i, _u64 = C.c_void_p, C.c_size_t, C.c_int, C.c_uint64
SYMBOLS = {
    "ec_allreduce_workspace_bytes": (_sz, [_i, _sz, _sz]),
    "ec_allreduce_init": (_i, [C.POINTER(_vp), _i, _sz, _i, _i, _sz, _i, _vp, _sz]),
    "ec_allreduce_apply": (_i, [_vp, _vp, _i, _sz, _i, _i, _sz, _vp, _vp, _vp, _vp]),
    "ec_allreduce_ssp_apply": (_i, [_vp, _vp, _i, _sz, _i, _i, _sz, _vp, C.c_uint32, C.c_uint32, _vp, _vp, _vp, _vp, _vp]),
    "ec_allreduce_reset": (_i, [_vp, _vp]),
    "ec_allreduce_host_staging_bytes": (_sz, [_vp, _i]),
    "ec_allreduce_epoch_host": (_i, [_vp, _vp, _vp, _i, _vp, _vp, _vp, _sz, _vp]),
    "ec_allreduce_set_tile": (_i, [_vp, _i, _sz]),
    "ec_allreduce_set_path": (_i, [_vp, _i]),
    "ec_allreduce_destroy": (_i, [_vp]),
    "ec_allgatherv": (_i, [_vp, _vp, _i, _i, _vp, _vp, _vp, _sz, _vp, _vp]),
    "ec_kmeans_workspace_bytes": (_sz, [_sz, _i, _i, _i]),
    "ec_kmeans_init": (_i, [C.POINTER(_vp), _vp, _sz, _i, _i, _i, _vp, _vp, _sz]),
    "ec_kmeans_assign": (_i, [_vp, _vp, _vp, _vp]),
    "ec_kmeans_partials": (_i, [_vp, _vp, _vp, _vp]),
    "ec_kmeans_iterate": (_i, [_vp, _vp, _vp]),
    "ec_kmeans_iterate_rounds": (_i, [_vp, _vp, _i, _vp]),
    "ec_kmeans_set_centroids": (_i, [_vp, _vp, _vp]),
    "ec_kmeans_get": (_i, [_vp, _vp, _vp, _vp, _vp, _vp]),
    "ec_kmeans_set_path": (_i, [_vp, _i]),
    "ec_kmeans_set_refresh": (_i, [_vp, _i]),
    "ec_kmeans_set_bounds": (_i, [_vp, _i]),
    "ec_kmeans_tc_status": (_i, [_vp, _vp, _vp]),
    "ec_kmeans_destroy": (_i, [_vp]),
    "ec_kmeans_partials_static": (_i, [_vp, _vp, _sz, _i, _i, _i, _vp, _vp]),
    "ec_allgatherv_compact": (_i, [_vp, _vp, _i, _i, _vp, _vp, _vp, _sz, _vp, _vp]),
    "ec_alltoall": (_i, [_vp, _vp, _i, _sz, _vp, _vp, _vp]),
    "ec_mf_workspace_bytes": (_sz, [_i, _i, _i, _i, _sz]),
    "ec_mf_init": (_i, [C.POINTER(_vp), _i, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, C.c_float, C.c_float, _sz, _vp, _sz]),
    "ec_mf_iterate": (_i, [_vp, _vp, C.c_uint32, _vp]),
    "ec_mf_set_factors": (_i, [_vp, _vp, _vp, _vp]),
    "ec_mf_get": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "ec_mf_destroy": (_i, [_vp]),
    "ec_bcast": (_i, [_vp, _vp, _i, _i, _sz, _i, _sz, C.c_double, _vp, _vp]),
    "ec_mask_data_fraction": (_i, [_i, _sz, C.c_double, _vp]),
    "ec_mask_process_threshold": (_i, [_i, _sz, C.c_double, _vp, C.POINTER(_i)]),
    "ec_threshold_segments": (_i, [_vp, _sz, C.c_uint32, _vp, _vp]),
    "ec_strerror": (C.c_char_p, [_i]),
    "ec_last_cuda_error": (_i, []),
    "ec_version": (_i, []),
}

_lib = None


def lib() -> C.CDLL:
    """Load the CUDA library; raises if it was not built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2203_17063_b200.build` "
                "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        for name, (res, args) in SYMBOLS.items():
            fn = getattr(L, name)
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


class EcError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().ec_strerror(code).decode()
        if code == ERR_CUDA:
            msg += f" [cudaError {lib().ec_last_cuda_error()}]"
        super().__init__(f"{where}: {msg} ({code})")


def _check(code: int, where: str) -> None:
    if code != OK:
        raise EcError(code, where)


def _ptr(t) -> int | None:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _table(bufs):
    return (C.c_void_p * len(bufs))(*[_ptr(b) for b in bufs])


class Allreduce:
    """ec_allreduce_init / apply / reset / destroy for one (P, n, dtype, op, segment_size)."""

    def __init__(self, P: int, n: int, dtype: int, op: int, segment_size: int, order: int = ORDER_FIXED,
                 device="cuda"):
        L = lib()
        self.P, self.n, self.dtype, self.op, self.seg, self.order = P, n, dtype, op, segment_size, order
        self.S = (n + segment_size - 1) // segment_size if segment_size else 0
        self.W = (P + 63) // 64
        need = L.ec_allreduce_workspace_bytes(P, n, segment_size)
        self._ws = torch.empty(max(need, 256), dtype=torch.uint8, device=device) if need else None
        h = C.c_void_p()
        _check(L.ec_allreduce_init(C.byref(h), P, n, dtype, op, segment_size, order,
                                   _ptr(self._ws), need), "ec_allreduce_init")
        self._h = h

    def apply(self, rank_bufs, arrival_mask, result, contrib_count=None, stream=None) -> None:
        _check(lib().ec_allreduce_apply(self._h, _table(rank_bufs), len(rank_bufs), self.n, self.dtype, self.op,
                                        self.seg, _ptr(arrival_mask), _ptr(result), _ptr(contrib_count),
                                        _stream(stream)), "ec_allreduce_apply")

    def apply_raw(self, table, arrival_mask_ptr, result_ptr, count_ptr, stream_ptr) -> int:
        """Same call with pre-marshalled arguments (for timing loops); returns the status code."""
        return lib().ec_allreduce_apply(self._h, table, self.P, self.n, self.dtype, self.op, self.seg,
                                        arrival_mask_ptr, result_ptr, count_ptr, stream_ptr)

    def ssp_apply(self, rank_bufs, notif_clock, clock: int, slack: int, result, contrib_count=None, seg_clock=None,
                  wait_count=None, stream=None) -> None:
        """ec_allreduce_ssp_apply: stale-synchronous apply; notif_clock is a device uint32 [S][P] tensor."""
        _check(lib().ec_allreduce_ssp_apply(self._h, _table(rank_bufs), len(rank_bufs), self.n, self.dtype, self.op,
                                            self.seg, _ptr(notif_clock), clock, slack, _ptr(result),
                                            _ptr(contrib_count), _ptr(seg_clock), _ptr(wait_count), _stream(stream)),
               "ec_allreduce_ssp_apply")

    def reset(self, stream=None) -> None:
        _check(lib().ec_allreduce_reset(self._h, _stream(stream)), "ec_allreduce_reset")

    def host_staging_bytes(self, rounds: int) -> int:
        return lib().ec_allreduce_host_staging_bytes(self._h, rounds)

    def epoch_host(self, host_rank_bufs, host_masks, host_result, host_contrib_count, staging, stream=None) -> None:
        """ec_allreduce_epoch_host: a whole epoch from host tensors (pinned for asynchronous copies);
        `staging` is a device uint8 tensor of at least host_staging_bytes(len(host_masks)) bytes."""
        _check(lib().ec_allreduce_epoch_host(self._h, _table(host_rank_bufs), _table(host_masks), len(host_masks),
                                             _ptr(host_result), _ptr(host_contrib_count), _ptr(staging),
                                             staging.numel() * staging.element_size(), _stream(stream)),
               "ec_allreduce_epoch_host")

    def epoch_host_raw(self, buf_table, mask_table, rounds, result_ptr, count_ptr, staging_ptr, staging_bytes,
                       stream_ptr) -> int:
        """Same call with pre-marshalled arguments (for timing loops); returns the status code."""
        return lib().ec_allreduce_epoch_host(self._h, buf_table, mask_table, rounds, result_ptr, count_ptr,
                                             staging_ptr, staging_bytes, stream_ptr)

    def set_tile(self, threads: int = 0, tile_elems: int = 0) -> None:
        _check(lib().ec_allreduce_set_tile(self._h, threads, tile_elems), "ec_allreduce_set_tile")

    def set_path(self, path: int) -> None:
        _check(lib().ec_allreduce_set_path(self._h, path), "ec_allreduce_set_path")

    def destroy(self) -> None:
        if getattr(self, "_h", None):
            lib().ec_allreduce_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def allgatherv(bufs, counts, dtype: int, arrival_mask, displs, out, status, stream=None,
               out_capacity_elems: int | None = None, compact: bool = False) -> None:
    """ec_allgatherv (fixed slots) or ec_allgatherv_compact (only arrived ranks get a slot):
    counts/displs/out/status are device tensors, bufs a list of device tensors (or None)."""
    cap = out.numel() if out_capacity_elems is None else out_capacity_elems
    fn = lib().ec_allgatherv_compact if compact else lib().ec_allgatherv
    _check(fn(_table(bufs), _ptr(counts), len(bufs), dtype, _ptr(arrival_mask), _ptr(displs),
                               _ptr(out), cap, _ptr(status), _stream(stream)), "ec_allgatherv")


def bcast(src, dst_bufs, root: int, dtype: int, segment_size: int, data_fraction: float, notify=None,
          stream=None) -> None:
    """ec_bcast: src and the entries of dst_bufs are device tensors (entries may be None)."""
    _check(lib().ec_bcast(_ptr(src), _table(dst_bufs), len(dst_bufs), root, src.numel(), dtype, segment_size,
                          data_fraction, _ptr(notify), _stream(stream)), "ec_bcast")


class KMeans:
    """ec_kmeans_* on device tensors: points fp32 [N][D], centroids fp32 [K][D]."""

    def __init__(self, points: torch.Tensor, K: int, P: int, init_centroids: torch.Tensor):
        L = lib()
        assert points.is_cuda and points.dtype == torch.float32 and points.is_contiguous()
        assert init_centroids.is_cuda and init_centroids.dtype == torch.float32 and init_centroids.is_contiguous()
        self.N, self.D = points.shape
        self.K, self.P = K, P
        self.points = points                      # keep alive: the library does not copy them
        need = L.ec_kmeans_workspace_bytes(self.N, self.D, K, P)
        self._ws = torch.empty(max(need, 256), dtype=torch.uint8, device=points.device) if need else None
        h = C.c_void_p()
        _check(L.ec_kmeans_init(C.byref(h), _ptr(points), self.N, self.D, K, P, _ptr(init_centroids),
                                _ptr(self._ws), need), "ec_kmeans_init")
        self._h = h

    def assign(self, centroids, labels, stream=None) -> None:
        _check(lib().ec_kmeans_assign(self._h, _ptr(centroids), _ptr(labels), _stream(stream)), "ec_kmeans_assign")

    def partials(self, labels, partials, stream=None) -> None:
        _check(lib().ec_kmeans_partials(self._h, _ptr(labels), _ptr(partials), _stream(stream)), "ec_kmeans_partials")

    def iterate(self, arrival_mask=None, stream=None) -> None:
        _check(lib().ec_kmeans_iterate(self._h, _ptr(arrival_mask), _stream(stream)), "ec_kmeans_iterate")

    def iterate_rounds(self, arrival_masks, stream=None) -> None:
        """One iteration whose allreduce epoch has len(arrival_masks) applies (cumulative device masks)."""
        _check(lib().ec_kmeans_iterate_rounds(self._h, _table(arrival_masks), len(arrival_masks), _stream(stream)),
               "ec_kmeans_iterate_rounds")

    def iterate_raw(self, mask_ptr, stream_ptr) -> int:
        return lib().ec_kmeans_iterate(self._h, mask_ptr, stream_ptr)

    def set_centroids(self, centroids, stream=None) -> None:
        _check(lib().ec_kmeans_set_centroids(self._h, _ptr(centroids), _stream(stream)), "ec_kmeans_set_centroids")

    def get(self, centroids=None, labels=None, reduced=None, contrib_count=None, stream=None) -> None:
        _check(lib().ec_kmeans_get(self._h, _ptr(centroids), _ptr(labels), _ptr(reduced), _ptr(contrib_count),
                                   _stream(stream)), "ec_kmeans_get")

    def set_refresh(self, every: int) -> None:
        """Every `every`-th iteration sums all points afresh (1 = each one does; default 32)."""
        _check(lib().ec_kmeans_set_refresh(self._h, every), "ec_kmeans_set_refresh")

    def set_bounds(self, enable: bool) -> None:
        """Distance bounds that let an iteration skip tiles whose labels cannot change (on by default)."""
        _check(lib().ec_kmeans_set_bounds(self._h, 1 if enable else 0), "ec_kmeans_set_bounds")

    def set_path(self, path: int) -> None:
        """0 automatic, 1 fp32 fused kernel, 2 tensor-core fused kernel."""
        _check(lib().ec_kmeans_set_path(self._h, path), "ec_kmeans_set_path")

    def tc_status(self, stream=None) -> int:
        out = torch.zeros(1, dtype=torch.int32, device=self.points.device)
        _check(lib().ec_kmeans_tc_status(self._h, _ptr(out), _stream(stream)), "ec_kmeans_tc_status")
        return int(out.item())

    def destroy(self) -> None:
        if getattr(self, "_h", None):
            lib().ec_kmeans_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def kmeans_partials_static(points: torch.Tensor, labels: torch.Tensor, K: int, P: int, partials: torch.Tensor,
                           stream=None) -> None:
    """ec_kmeans_partials_static: the per-rank partial sums without a workspace, for callers that
    must not allocate device memory (the per-block sums go to a fixed array inside the library)."""
    N, D = points.shape
    _check(lib().ec_kmeans_partials_static(_ptr(points), _ptr(labels), N, D, K, P, _ptr(partials), _stream(stream)),
           "ec_kmeans_partials_static")


def mask_data_fraction(P: int, S: int, fraction: float):
    """ec_mask_data_fraction: host notification words (numpy uint64 [S][W]) with the first ceil(fraction*S) segments set."""
    import numpy as np
    out = np.zeros((S, (P + 63) // 64), dtype=np.uint64)
    _check(lib().ec_mask_data_fraction(P, S, fraction, out.ctypes.data), "ec_mask_data_fraction")
    return out


def mask_process_threshold(P: int, S: int, fraction: float):
    """ec_mask_process_threshold: (host notification words, number of ranks the binomial-tree stages bring in)."""
    import numpy as np
    out = np.zeros((S, (P + 63) // 64), dtype=np.uint64)
    n = C.c_int(0)
    _check(lib().ec_mask_process_threshold(P, S, fraction, out.ctypes.data, C.byref(n)), "ec_mask_process_threshold")
    return out, n.value


def threshold_segments(contrib_count, need: int, ready, stream=None) -> None:
    """ec_threshold_segments: ready[0] = number of segments whose contributor count is at least `need` (device tensors)."""
    _check(lib().ec_threshold_segments(_ptr(contrib_count), contrib_count.numel(), need, _ptr(ready), _stream(stream)),
           "ec_threshold_segments")


def alltoall(send_bufs, recv_bufs, block_bytes: int, arrival_mask=None, recv_count=None, stream=None) -> None:
    """ec_alltoall: recv[d] block s <- send[s] block d for every notified (d, s); device tensors."""
    _check(lib().ec_alltoall(_table(send_bufs), _table(recv_bufs), len(send_bufs), block_bytes, _ptr(arrival_mask),
                             _ptr(recv_count), _stream(stream)), "ec_alltoall")


class MatrixFactorization:
    """ec_mf_*: data is a dict of device tensors (user_ptr, user_item, user_val, rank_item_ptr, item_user,
    item_val) laid out as inputs.mf_ratings describes; the factors are device fp32 tensors."""

    def __init__(self, data: dict, n_users: int, n_items: int, P: int, user_factors: torch.Tensor,
                 item_factors: torch.Tensor, lr: float, lam: float, segment_rows: int):
        L = lib()
        self.data = data                                   # keep alive: the library does not copy the ratings
        self.U, self.I, self.P, self.k = n_users, n_items, P, user_factors.shape[1]
        self.S = (n_items + segment_rows - 1) // segment_rows
        need = L.ec_mf_workspace_bytes(n_users, n_items, self.k, P, segment_rows)
        self._ws = torch.empty(max(need, 256), dtype=torch.uint8, device=user_factors.device)
        h = C.c_void_p()
        _check(L.ec_mf_init(C.byref(h), n_users, n_items, self.k, P, _ptr(data["user_ptr"]), _ptr(data["user_item"]),
                            _ptr(data["user_val"]), _ptr(data["rank_item_ptr"]), _ptr(data["item_user"]),
                            _ptr(data["item_val"]), _ptr(user_factors), _ptr(item_factors), lr, lam, segment_rows,
                            _ptr(self._ws), need), "ec_mf_init")
        self._h = h

    def iterate(self, refresh_mask=None, slack: int = 0, stream=None) -> None:
        _check(lib().ec_mf_iterate(self._h, _ptr(refresh_mask), slack, _stream(stream)), "ec_mf_iterate")

    def set_factors(self, user_factors, item_factors, stream=None) -> None:
        _check(lib().ec_mf_set_factors(self._h, _ptr(user_factors), _ptr(item_factors), _stream(stream)), "ec_mf_set_factors")

    def get(self, user_factors=None, item_factors=None, sse=None, seg_clock=None, notif_clock=None, wait_count=None,
            stream=None) -> None:
        _check(lib().ec_mf_get(self._h, _ptr(user_factors), _ptr(item_factors), _ptr(sse), _ptr(seg_clock),
                               _ptr(notif_clock), _ptr(wait_count), _stream(stream)), "ec_mf_get")

    def destroy(self) -> None:
        if getattr(self, "_h", None):
            lib().ec_mf_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass
