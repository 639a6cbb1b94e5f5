"""ctypes front end of the CPU checker (``ec_oracle.cpp``).  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the GPU library and its Python binding never do.  All arguments
are numpy arrays in host memory.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ec_oracle.cpp")
_LIB = os.path.join(_HERE, "libec_oracle.so")

F32, BF16, I64, F64 = 0, 1, 2, 3
SUM, MAX, MIN = 0, 1, 2
ORDER_FIXED, ORDER_PAIRWISE, ORDER_RING = 0, 1, 2

_IN_NP = {F32: np.float32, BF16: np.uint16, I64: np.int64, F64: np.float64}
_OUT_NP = {F32: np.float32, BF16: np.float32, I64: np.int64, F64: np.float64}

CXXFLAGS = ["-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-fPIC", "-shared", "-std=c++17"]


def build(force: bool = False) -> str:
    """Compile the checker with g++ (plain -O2, no contraction, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["g++", *CXXFLAGS, "-o", _LIB, _SRC])
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.oracle_allreduce_new.restype = C.c_void_p
        L.oracle_allreduce_new.argtypes = [C.c_int, C.c_size_t, C.c_int, C.c_int, C.c_size_t]
        L.oracle_allreduce_free.argtypes = [C.c_void_p]
        L.oracle_allreduce_reset.argtypes = [C.c_void_p]
        L.oracle_allreduce_apply.restype = C.c_int
        L.oracle_allreduce_apply.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                             C.c_int, C.c_int]
        L.oracle_allreduce_applied.argtypes = [C.c_void_p, C.c_void_p]
        L.oracle_allreduce_oneshot.restype = C.c_int
        L.oracle_allreduce_oneshot.argtypes = [C.c_int, C.c_size_t, C.c_int, C.c_int, C.c_size_t,
                                               C.c_void_p, C.c_void_p, C.c_void_p]
        L.oracle_allreduce_ref64.restype = C.c_int
        L.oracle_allreduce_ref64.argtypes = [C.c_int, C.c_size_t, C.c_int, C.c_size_t, C.c_void_p,
                                             C.c_void_p, C.c_void_p, C.c_void_p]
        L.oracle_allreduce_ssp.restype = C.c_int
        L.oracle_allreduce_ssp.argtypes = [C.c_int, C.c_size_t, C.c_int, C.c_int, C.c_size_t, C.c_void_p, C.c_void_p,
                                           C.c_uint32, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.oracle_allgatherv_compact.restype = C.c_int
        L.oracle_allgatherv_compact.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_size_t, C.c_void_p,
                                                C.c_void_p, C.c_void_p, C.c_size_t]
        L.oracle_alltoall.restype = C.c_int
        L.oracle_alltoall.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_size_t, C.c_void_p, C.c_void_p]
        L.oracle_allgatherv.restype = C.c_int
        L.oracle_allgatherv.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_size_t, C.c_void_p,
                                        C.c_void_p, C.c_void_p, C.c_size_t]
        L.oracle_kmeans_assign.argtypes = [C.c_void_p, C.c_size_t, C.c_int, C.c_void_p, C.c_int,
                                           C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int]
        L.oracle_kmeans_partials.argtypes = [C.c_void_p, C.c_size_t, C.c_int, C.c_int, C.c_int,
                                             C.c_void_p, C.c_void_p, C.c_int]
        L.oracle_kmeans_update.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
        L.oracle_max_threads.restype = C.c_int
        _lib = L
    return _lib


def max_threads() -> int:
    return int(lib().oracle_max_threads())


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _ptr_table(bufs, dtype_np):
    keep = [np.ascontiguousarray(b, dtype=dtype_np) for b in bufs]
    table = (C.c_void_p * len(keep))(*[b.ctypes.data for b in keep])
    return keep, table


class Allreduce:
    """State of one eventually consistent allreduce (which contributions are
    already folded into ``result``) plus the apply/reset calls."""

    def __init__(self, P: int, n: int, dtype: int, op: int, segment_size: int):
        self.P, self.n, self.dtype, self.op, self.seg = P, n, dtype, op, segment_size
        self.S = (n + segment_size - 1) // segment_size
        self.W = (P + 63) // 64
        self._h = lib().oracle_allreduce_new(P, n, dtype, op, segment_size)
        if not self._h:
            raise ValueError("bad allreduce parameters")

    def __del__(self):
        if getattr(self, "_h", None):
            lib().oracle_allreduce_free(self._h)
            self._h = None

    def reset(self) -> None:
        lib().oracle_allreduce_reset(self._h)

    def apply(self, bufs, arrival_mask, result: np.ndarray, contrib_count: np.ndarray | None = None,
              order: int = ORDER_FIXED, threads: int = 1) -> None:
        """Fold the newly notified contributions into ``result`` (in place)."""
        assert len(bufs) == self.P
        keep, table = _ptr_table(bufs, _IN_NP[self.dtype])
        for b in keep:
            assert b.size >= self.n
        assert result.dtype == _OUT_NP[self.dtype] and result.flags.c_contiguous and result.size >= self.n
        if arrival_mask is not None:
            arrival_mask = np.ascontiguousarray(arrival_mask, dtype=np.uint64)
            assert arrival_mask.size == self.S * self.W
        if contrib_count is not None:
            assert contrib_count.dtype == np.uint32 and contrib_count.size >= self.S
        rc = lib().oracle_allreduce_apply(self._h, table, _ptr(arrival_mask), _ptr(result),
                                          _ptr(contrib_count), order, threads)
        if rc != 0:
            raise RuntimeError("oracle_allreduce_apply failed")

    def applied(self) -> np.ndarray:
        out = np.zeros((self.P, self.S), dtype=np.uint8)
        lib().oracle_allreduce_applied(self._h, _ptr(out))
        return out.astype(bool)


def allreduce_oneshot(bufs, dtype: int, op: int, segment_size: int, order: np.ndarray) -> np.ndarray:
    """Fold each segment once, left to right through ``order`` (int32 [S][P], -1 ends a row)."""
    P = len(bufs)
    keep, table = _ptr_table(bufs, _IN_NP[dtype])
    n = keep[0].size
    order = np.ascontiguousarray(order, dtype=np.int32)
    result = np.empty(n, dtype=_OUT_NP[dtype])
    rc = lib().oracle_allreduce_oneshot(P, n, dtype, op, segment_size, table, _ptr(order), _ptr(result))
    if rc != 0:
        raise RuntimeError("oracle_allreduce_oneshot failed")
    return result


def allreduce_ref64(bufs, dtype: int, segment_size: int, arrival_mask=None):
    """(double-precision sum over notified ranks, sum of magnitudes) per element."""
    P = len(bufs)
    keep, table = _ptr_table(bufs, _IN_NP[dtype])
    n = keep[0].size
    if arrival_mask is not None:
        arrival_mask = np.ascontiguousarray(arrival_mask, dtype=np.uint64)
    ref = np.empty(n, dtype=np.float64)
    mag = np.empty(n, dtype=np.float64)
    rc = lib().oracle_allreduce_ref64(P, n, dtype, segment_size, table, _ptr(arrival_mask), _ptr(ref), _ptr(mag))
    if rc != 0:
        raise RuntimeError("oracle_allreduce_ref64 failed")
    return ref, mag


def allreduce_ssp(bufs, dtype: int, op: int, segment_size: int, notif_clock: np.ndarray, clock: int, slack: int):
    """Stale-synchronous allreduce: returns (result, contrib_count, seg_clock, wait_count).
    notif_clock is uint32 [S][P]: the clock of the contribution each rank buffer holds, 0 = none."""
    P = len(bufs)
    keep, table = _ptr_table(bufs, _IN_NP[dtype])
    n = keep[0].size
    S = (n + segment_size - 1) // segment_size
    notif_clock = np.ascontiguousarray(notif_clock, dtype=np.uint32)
    assert notif_clock.shape == (S, P)
    result = np.empty(n, dtype=_OUT_NP[dtype])
    count = np.empty(S, dtype=np.uint32)
    seg_clock = np.empty(S, dtype=np.uint32)
    wait = np.empty(S, dtype=np.uint32)
    rc = lib().oracle_allreduce_ssp(P, n, dtype, op, segment_size, table, _ptr(notif_clock), clock, slack,
                                    _ptr(result), _ptr(count), _ptr(seg_clock), _ptr(wait))
    if rc != 0:
        raise RuntimeError("oracle_allreduce_ssp failed")
    return result, count, seg_clock, wait


def allgatherv(bufs, counts: np.ndarray, arrival_mask, out: np.ndarray, compact: bool = False):
    """Returns (displs int64 [P+1], status); copies notified ranks into ``out`` in place.
    compact=False: fixed slots from the counts of all ranks; compact=True: only notified ranks get a slot."""
    P = len(bufs)
    counts = np.ascontiguousarray(counts, dtype=np.int64)
    keep = [np.ascontiguousarray(b) for b in bufs]
    for r, b in enumerate(keep):
        assert b.dtype == out.dtype and b.size >= counts[r]
    table = (C.c_void_p * P)(*[b.ctypes.data for b in keep])
    if arrival_mask is not None:
        arrival_mask = np.ascontiguousarray(arrival_mask, dtype=np.uint64)
    displs = np.empty(P + 1, dtype=np.int64)
    assert out.flags.c_contiguous
    fn = lib().oracle_allgatherv_compact if compact else lib().oracle_allgatherv
    status = fn(table, _ptr(counts), P, out.dtype.itemsize, _ptr(arrival_mask), _ptr(displs), _ptr(out), out.size)
    return displs, int(status)


def alltoall(send_bufs, recv_bufs, block_bytes: int, arrival_mask=None) -> np.ndarray:
    """recv_bufs[d] block s <- send_bufs[s] block d for every notified (d, s), in place (uint8 arrays of
    P * block_bytes bytes); returns recv_count uint32 [P]."""
    P = len(send_bufs)
    for b in list(send_bufs) + list(recv_bufs):
        assert b.dtype == np.uint8 and b.flags.c_contiguous and b.size >= P * block_bytes
    st = (C.c_void_p * P)(*[b.ctypes.data for b in send_bufs])
    rt = (C.c_void_p * P)(*[b.ctypes.data for b in recv_bufs])
    if arrival_mask is not None:
        arrival_mask = np.ascontiguousarray(arrival_mask, dtype=np.uint64)
    count = np.empty(P, dtype=np.uint32)
    rc = lib().oracle_alltoall(st, rt, P, block_bytes, _ptr(arrival_mask), _ptr(count))
    if rc != 0:
        raise RuntimeError("oracle_alltoall failed")
    return count


def kmeans_assign(points: np.ndarray, centroids: np.ndarray, threads: int = 1):
    """Returns (labels int32, best d^2, second-best d^2, second-best label)."""
    points = np.ascontiguousarray(points, dtype=np.float32)
    centroids = np.ascontiguousarray(centroids, dtype=np.float32)
    N, D = points.shape
    K = centroids.shape[0]
    labels = np.empty(N, dtype=np.int32)
    best = np.empty(N, dtype=np.float64)
    second = np.empty(N, dtype=np.float64)
    second_label = np.empty(N, dtype=np.int32)
    lib().oracle_kmeans_assign(_ptr(points), N, D, _ptr(centroids), K, _ptr(labels), _ptr(best),
                               _ptr(second), _ptr(second_label), threads)
    return labels, best, second, second_label


def kmeans_partials(points: np.ndarray, labels: np.ndarray, K: int, P: int, threads: int = 1) -> np.ndarray:
    """fp32 [P][K][D+4]: per rank and centroid the coordinate sums, the point count, three zeros."""
    points = np.ascontiguousarray(points, dtype=np.float32)
    labels = np.ascontiguousarray(labels, dtype=np.int32)
    N, D = points.shape
    out = np.empty((P, K, D + 4), dtype=np.float32)
    lib().oracle_kmeans_partials(_ptr(points), N, D, K, P, _ptr(labels), _ptr(out), threads)
    return out


def kmeans_update(reduced: np.ndarray, old_centroids: np.ndarray) -> np.ndarray:
    reduced = np.ascontiguousarray(reduced, dtype=np.float32)
    old_centroids = np.ascontiguousarray(old_centroids, dtype=np.float32)
    K, D = old_centroids.shape
    assert reduced.shape == (K, D + 4)
    new = np.empty_like(old_centroids)
    lib().oracle_kmeans_update(_ptr(reduced), D, K, _ptr(old_centroids), _ptr(new))
    return new


def kmeans_iterate(points: np.ndarray, centroids: np.ndarray, P: int, arrival_mask, threads: int = 1):
    """One Lloyd iteration whose combine step is one eventually consistent
    allreduce epoch with one segment per centroid row: assignment, per-rank
    partials, a single apply with this iteration's notifications (late rows are
    dropped; the next iteration supersedes them), centroid update.
    Returns (new centroids, labels, reduced [K][D+4], contrib_count [K])."""
    K, D = centroids.shape
    labels, _, _, _ = kmeans_assign(points, centroids, threads)
    partials = kmeans_partials(points, labels, K, P, threads)
    n = K * (D + 4)
    ar = Allreduce(P, n, F32, SUM, D + 4)
    reduced = np.empty(n, dtype=np.float32)
    count = np.empty(K, dtype=np.uint32)
    masks = arrival_mask if isinstance(arrival_mask, (list, tuple)) else [arrival_mask]
    for m in masks:                       # several cumulative masks = several rounds of one epoch before the update
        ar.apply([partials[r].reshape(-1) for r in range(P)], m, reduced, count)
    reduced = reduced.reshape(K, D + 4)
    return kmeans_update(reduced, centroids), labels, reduced, count


# ---------------------------------------------------------------------------
# Threshold variants of Reduce / Broadcast (Sec. III-B), written out plainly.
# ---------------------------------------------------------------------------
def bst_stage_of_rank(rank: int) -> int:
    """Stage of the binomial spanning tree in which a rank receives its data (root: -1).
    The tree works in stages that double the number of involved processes: after stage k the
    ranks 0 .. 2^(k+1)-1 are involved, so rank r > 0 joins in stage floor(log2 r)."""
    if rank == 0:
        return -1
    stage = 0
    while (1 << (stage + 1)) <= rank:
        stage += 1
    return stage


def bst_parent(rank: int) -> int:
    """Parent in the binomial tree: the children of p are p + 2^i for the stages i after p joined
    (-1 for the root)."""
    if rank == 0:
        return -1
    return rank - (1 << bst_stage_of_rank(rank))


def process_threshold_ranks(P: int, fraction: float) -> int:
    """Number of ranks involved when whole stages are added until at least fraction*P take part."""
    involved = 1 if fraction > 0 else 0
    stage = 0
    while 0 < involved < P and involved < fraction * P:
        involved = min(P, sum(1 for r in range(P) if bst_stage_of_rank(r) <= stage))
        stage += 1
    return involved


def process_threshold_mask(P: int, S: int, fraction: float) -> np.ndarray:
    arrived = np.zeros((P, S), dtype=bool)
    arrived[:process_threshold_ranks(P, fraction)] = True
    return _pack_words(arrived)


def data_fraction_mask(P: int, S: int, fraction: float) -> np.ndarray:
    import math
    arrived = np.zeros((P, S), dtype=bool)
    arrived[:, :min(S, math.ceil(fraction * S))] = True
    return _pack_words(arrived)


def bcast(src: np.ndarray, dst_bufs, root: int, segment_size: int, data_fraction: float):
    """Broadcast with a data threshold (Sec. III-B): the first ceil(fraction * S) segments of the root's
    vector are written into every receive buffer that exists (entries of dst_bufs may be None, and the
    root's own entry may be the source itself); nothing else is touched.  Works in place on dst_bufs and
    returns the notification words uint64 [S][W]: bit r of segment s = rank r now holds segment s."""
    import math
    n, P = src.size, len(dst_bufs)
    S = (n + segment_size - 1) // segment_size
    keep = min(S, math.ceil(data_fraction * S))
    holds = np.zeros((P, S), dtype=bool)
    for r in range(P):
        if dst_bufs[r] is None and r != root:
            continue
        for s in range(keep):
            lo, hi = s * segment_size, min(n, (s + 1) * segment_size)
            if dst_bufs[r] is not None and dst_bufs[r] is not src:
                for i in range(lo, hi):
                    dst_bufs[r][i] = src[i]
            holds[r, s] = True
    return _pack_words(holds)


def _pack_words(arrived: np.ndarray) -> np.ndarray:
    P, S = arrived.shape
    out = np.zeros((S, (P + 63) // 64), dtype=np.uint64)
    for s in range(S):
        for r in range(P):
            if arrived[r, s]:
                out[s, r // 64] |= np.uint64(1 << (r % 64))
    return out


def threshold_segments(contrib_count: np.ndarray, need: int) -> int:
    return int(sum(1 for c in contrib_count if c >= need))


# ---------------------------------------------------------------------------------------------
# Matrix factorisation trained by gradient steps whose item gradients go through the
# stale-synchronous allreduce (the paper's experiment with allreduce_SSP, Sec. V; the paper names the
# model and the collective, not the update rule: what follows is the textbook rule).
#
#   model      r_ui ~ <p_u, q_i>;  e_ui = r_ui - <p_u, q_i>
#   rank r     owns the users [r*U/P, (r+1)*U/P) with all their ratings; user factors are local
#   shared     the item factors; every rank contributes G_r[i] = sum over its ratings of e_ui * p_u
#   one iteration at clock t (all errors e are taken at the factors the iteration starts from)
#     1. contribution (r, s) - s an item segment of `segment_rows` rows - is recomputed if its bit in
#        `refresh` is set, if it was never computed, or if it is older than t - slack (Algorithm 1:
#        a contribution that is too stale is waited for); then its clock becomes t.  Otherwise the
#        rank's buffer keeps the gradient it delivered earlier.
#     2. R = sum over ranks of G_r in rank order (all clocks are now >= t - slack);
#        seg_clock[s] = min over ranks of the clocks (the age of the result, Sec. III-A)
#     3. p_u += lr * (sum_i e_ui * q_i - lam * p_u)        for every user
#     4. q_i += lr * (R_i - lam * q_i)                       for every item
#   sse = sum of e_ui^2 over all ratings at the start of the iteration.
# ---------------------------------------------------------------------------------------------
class MatrixFactorization:
    def __init__(self, data: dict, user_factors: np.ndarray, item_factors: np.ndarray, lr: float, lam: float,
                 segment_rows: int):
        self.d = data
        self.U, self.I, self.P = data["n_users"], data["n_items"], data["P"]
        self.k = user_factors.shape[1]
        self.pu = user_factors.astype(np.float64)
        self.qi = item_factors.astype(np.float64)
        self.lr, self.lam, self.seg = float(lr), float(lam), int(segment_rows)
        self.S = (self.I + self.seg - 1) // self.seg
        self.clock = 0
        self.grad = np.zeros((self.P, self.I, self.k), dtype=np.float64)      # what each rank delivered last
        self.notif_clock = np.zeros((self.S, self.P), dtype=np.uint32)

    def rank_item_gradient(self, r: int) -> np.ndarray:
        """G_r[i] = sum over rank r's ratings (u, i) of e_ui * p_u, at the current factors."""
        d = self.d
        out = np.zeros((self.I, self.k), dtype=np.float64)
        for i in range(self.I):
            for j in range(int(d["rank_item_ptr"][r, i]), int(d["rank_item_ptr"][r, i + 1])):
                u = int(d["item_user"][j])
                e = float(d["item_val"][j]) - float(np.dot(self.pu[u], self.qi[i]))
                out[i] += e * self.pu[u]
        return out

    def user_gradient(self):
        """(g_u = sum_i e_ui * q_i for every user, sum of e^2), at the current factors."""
        d = self.d
        g = np.zeros((self.U, self.k), dtype=np.float64)
        sse = 0.0
        for u in range(self.U):
            for j in range(int(d["user_ptr"][u]), int(d["user_ptr"][u + 1])):
                i = int(d["user_item"][j])
                e = float(d["user_val"][j]) - float(np.dot(self.pu[u], self.qi[i]))
                g[u] += e * self.qi[i]
                sse += e * e
        return g, sse

    def iterate(self, refresh: np.ndarray | None, slack: int):
        """One iteration; refresh is bool [P][S] or None (= everything fresh).
        Returns (sse at the start of the iteration, seg_clock uint32 [S], refreshed bool [P][S])."""
        self.clock += 1
        t = self.clock
        min_ok = t - slack if t > slack else 1
        refreshed = np.zeros((self.P, self.S), dtype=bool)
        for r in range(self.P):
            fresh = None
            for s in range(self.S):
                want = refresh is None or bool(refresh[r, s])
                c = int(self.notif_clock[s, r])
                if want or c == 0 or c < min_ok:
                    if fresh is None:
                        fresh = self.rank_item_gradient(r)
                    lo, hi = s * self.seg, min(self.I, (s + 1) * self.seg)
                    self.grad[r, lo:hi] = fresh[lo:hi]
                    self.notif_clock[s, r] = t
                    refreshed[r, s] = True
        reduced = np.zeros((self.I, self.k), dtype=np.float64)
        for r in range(self.P):
            reduced += self.grad[r]
        seg_clock = self.notif_clock.min(axis=1).astype(np.uint32)
        g_user, sse = self.user_gradient()
        self.pu = self.pu + self.lr * (g_user - self.lam * self.pu)
        self.qi = self.qi + self.lr * (reduced - self.lam * self.qi)
        return sse, seg_clock, refreshed

    def loss(self) -> float:
        """0.5 * sum e^2 + 0.5 * lam * (|P|^2 + |Q|^2): the function whose gradient the steps follow."""
        _, sse = self.user_gradient()
        return 0.5 * sse + 0.5 * self.lam * (float((self.pu ** 2).sum()) + float((self.qi ** 2).sum()))
