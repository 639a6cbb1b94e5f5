"""Seeded synthetic inputs for the eventually consistent collectives.

This module only *draws* data: rank buffers, arrival schedules, gather counts
and K-means point clouds.  It performs none of the method's arithmetic (no
reduction, no scan, no distance) and is the single source of the bytes that
both the CUDA path and the CPU checker consume, so the two always see
identical inputs.  Everything is generated on the host with numpy's
counter-based Philox generator keyed by ``(seed, stream)``; a stream is a rank,
an iteration or a named purpose, so any buffer can be regenerated alone.

Shapes follow the workloads of the paper's experiments section: dense
per-process vectors of 10^4 .. 8,388,608 elements ("several kilobytes to
hundreds of megabytes") exchanged by 4-64 processes, and gradient-like vectors
exchanged every iteration of an ML solver.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
import os

import numpy as np

# Stream identifiers (second Philox key word) so that different purposes of one
# seed never share random numbers.
_STREAM_VALUES = 0            # + rank
_STREAM_SCHEDULE = 1 << 20
_STREAM_COUNTS = 2 << 20
_STREAM_KM_CENTRES = 3 << 20
_STREAM_KM_POINTS = 4 << 20   # + chunk
_STREAM_KM_MASK = 5 << 20     # + iteration
_STREAM_MF = 6 << 20          # + purpose / iteration


def _rng(seed: int, stream: int) -> np.random.Generator:
    key = np.array([seed & 0xFFFFFFFFFFFFFFFF, stream & 0xFFFFFFFFFFFFFFFF], dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def _pool_map(fn, items):
    workers = min(len(items), os.cpu_count() or 1, 16)
    if workers <= 1:
        return [fn(i) for i in items]
    with ThreadPoolExecutor(max_workers=workers) as ex:
        return list(ex.map(fn, items))


# --------------------------------------------------------------------------
# rank buffers
# --------------------------------------------------------------------------
def uniform_f32(seed: int, rank: int, n: int, out: np.ndarray | None = None) -> np.ndarray:
    """n fp32 values uniform in [-1, 1): k / 2^23 - 1 with k a 24-bit integer."""
    u = _rng(seed, _STREAM_VALUES + rank).random(n, dtype=np.float32)
    u *= np.float32(2.0)
    u -= np.float32(1.0)
    if out is not None:
        out[...] = u
        return out
    return u


def normal_f32(seed: int, rank: int, n: int, sigma: float = 1.0,
               out: np.ndarray | None = None) -> np.ndarray:
    """n fp32 values N(0, sigma^2)."""
    x = _rng(seed, _STREAM_VALUES + rank).standard_normal(n, dtype=np.float32)
    if sigma != 1.0:
        x *= np.float32(sigma)
    if out is not None:
        out[...] = x
        return out
    return x


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bfloat16 (round to nearest even); returns the raw uint16 bits."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of raw bfloat16 bits to fp32 (for test bookkeeping only)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bf16_bits(seed: int, rank: int, n: int, sigma: float,
                     out: np.ndarray | None = None) -> np.ndarray:
    """n gradient-like values N(0, sigma^2), rounded to bfloat16; raw uint16 bits."""
    b = f32_to_bf16_bits(normal_f32(seed, rank, n, sigma))
    if out is not None:
        out[...] = b
        return out
    return b


def int64_full_range(seed: int, rank: int, n: int) -> np.ndarray:
    """n int64 values uniform over the whole int64 range."""
    raw = _rng(seed, _STREAM_VALUES + rank).integers(0, 2 ** 64, size=n, dtype=np.uint64)
    return raw.view(np.int64)


def int64_below(seed: int, rank: int, n: int, bound: int = 1 << 20) -> np.ndarray:
    """n int64 values uniform in [0, bound)."""
    return _rng(seed, _STREAM_VALUES + rank).integers(0, bound, size=n, dtype=np.int64)


def rank_buffers(kind: str, seed: int, P: int, n: int, **kw) -> list[np.ndarray]:
    """All P rank buffers of one workload, generated in parallel.

    kind: "uniform_f32" | "normal_f32" | "normal_bf16" | "int64_full" | "int64_below".
    """
    fn = {
        "uniform_f32": lambda r: uniform_f32(seed, r, n),
        "normal_f32": lambda r: normal_f32(seed, r, n, kw.get("sigma", 1.0)),
        "normal_bf16": lambda r: normal_bf16_bits(seed, r, n, kw.get("sigma", 1e-3)),
        "int64_full": lambda r: int64_full_range(seed, r, n),
        "int64_below": lambda r: int64_below(seed, r, n, kw.get("bound", 1 << 20)),
    }[kind]
    return _pool_map(fn, list(range(P)))


# --------------------------------------------------------------------------
# arrival schedules (the notifications)
# --------------------------------------------------------------------------
def mask_words(P: int) -> int:
    """Number of 64-bit words that hold one bit per rank."""
    return (P + 63) // 64


def num_segments(n: int, segment_size: int) -> int:
    return (n + segment_size - 1) // segment_size


def arrival_rounds(seed: int, P: int, S: int, p_first: float, last_round: int = 3) -> np.ndarray:
    """Round (1-based) in which each (rank, segment) contribution arrives.

    Round 1 with probability p_first, otherwise uniformly one of rounds
    2..last_round.  With last_round = 3 every contribution has landed two
    rounds after the first one, i.e. the schedule respects a staleness bound
    (slack) of 2.  Returns int8 [P][S].
    """
    g = _rng(seed, _STREAM_SCHEDULE)
    u = g.random((P, S))
    late = g.integers(2, last_round + 1, size=(P, S)) if last_round >= 2 else np.ones((P, S), np.int64)
    rounds = np.where(u < p_first, 1, late).astype(np.int8)
    return rounds


def pack_mask(arrived: np.ndarray) -> np.ndarray:
    """Pack a boolean [P][S] "has arrived" table into uint64 [S][W] notification words.

    Bit (r % 64) of word [s][r // 64] is the notification of rank r for segment s.
    """
    arrived = np.asarray(arrived, dtype=bool)
    P, S = arrived.shape
    W = mask_words(P)
    out = np.zeros((S, W), dtype=np.uint64)
    for r in range(P):
        out[:, r // 64] |= arrived[r].astype(np.uint64) << np.uint64(r % 64)
    return out


def cumulative_masks(rounds: np.ndarray, last_round: int | None = None) -> list[np.ndarray]:
    """Packed notification words as they stand after round 1, 2, ... (cumulative)."""
    last = int(rounds.max()) if last_round is None else last_round
    return [pack_mask(rounds <= t) for t in range(1, last + 1)]


def bernoulli_mask(seed: int, stream: int, P: int, S: int, p: float) -> np.ndarray:
    """Boolean [P][S]: each contribution has arrived with probability p."""
    return _rng(seed, _STREAM_SCHEDULE + 1 + stream).random((P, S)) < p


# --------------------------------------------------------------------------
# allgatherv
# --------------------------------------------------------------------------
def gather_counts(seed: int, P: int, lo: int = 1024, hi: int = 65536) -> np.ndarray:
    """Per-rank element counts uniform in [lo, hi]; int64 [P]."""
    return _rng(seed, _STREAM_COUNTS).integers(lo, hi + 1, size=P, dtype=np.int64)


def gather_buffers(seed: int, counts: np.ndarray) -> list[np.ndarray]:
    """One int64 buffer per rank holding counts[r] full-range values."""
    return _pool_map(lambda r: int64_full_range(seed, r, int(counts[r])), list(range(len(counts))))


# --------------------------------------------------------------------------
# K-means point cloud
# --------------------------------------------------------------------------
def kmeans_mixture(seed: int, N: int, D: int, K: int, sigma: float = 1.0,
                   box: float = 10.0) -> tuple[np.ndarray, np.ndarray, np.ndarray]:
    """N points from a K-component isotropic Gaussian mixture.

    Centres uniform in [-box, box]^D, equal weights, standard deviation sigma.
    Returns (points fp32 [N][D], component int32 [N], centres fp32 [K][D]).
    """
    centres = _rng(seed, _STREAM_KM_CENTRES).uniform(-box, box, size=(K, D)).astype(np.float32)
    comp = _rng(seed, _STREAM_KM_CENTRES + 1).integers(0, K, size=N, dtype=np.int32)
    chunk = 1 << 18
    starts = list(range(0, N, chunk))
    points = np.empty((N, D), dtype=np.float32)

    def fill(i0: int) -> None:
        i1 = min(N, i0 + chunk)
        noise = _rng(seed, _STREAM_KM_POINTS + i0 // chunk).standard_normal((i1 - i0, D), dtype=np.float32)
        if sigma != 1.0:
            noise *= np.float32(sigma)
        np.add(noise, centres[comp[i0:i1]], out=points[i0:i1])

    _pool_map(fill, starts)
    return points, comp, centres


def kmeans_first_of_component(points: np.ndarray, comp: np.ndarray, K: int) -> np.ndarray:
    """Initial centroids: for each mixture component the first point (in index
    order) drawn from it.  One starting centroid per component keeps Lloyd's
    iteration away from decision boundaries that cut through dense data."""
    first = np.full(K, -1, dtype=np.int64)
    seen = 0
    for j, z in enumerate(comp):
        if first[z] < 0:
            first[z] = j
            seen += 1
            if seen == K:
                break
    if (first < 0).any():
        raise ValueError("a mixture component drew no point; enlarge N")
    return np.ascontiguousarray(points[first], dtype=np.float32)


def kmeans_masks(seed: int, iters: int, P: int, K: int, p: float) -> list[np.ndarray]:
    """Per iteration the packed notification words [K][W]: contribution
    (rank, centroid row) has arrived with probability p."""
    return [pack_mask(_rng(seed, _STREAM_KM_MASK + t).random((P, K)) < p) for t in range(iters)]


# --------------------------------------------------------------------------
# Matrix-factorisation ratings (stand-in for the paper's MovieLens experiment)
# --------------------------------------------------------------------------
def mf_ratings(seed: int, n_users: int, n_items: int, k_true: int, nnz: int, P: int, noise: float = 0.1) -> dict:
    """A sparse low-rank rating matrix, stored twice as such data usually is: by user
    (CSR over all users; rank r owns the users [r*U/P, (r+1)*U/P) and so a contiguous
    range of the ratings) and, inside every rank's share, by item.

    Users are drawn uniformly, items with a popularity that falls off like a power law
    (item = floor(I * x^1.5), x uniform: the most popular of 16384 items draws 0.15 % of the ratings), ratings are the inner product of two hidden
    factor vectors with N(0, 1/k_true) entries plus N(0, noise^2).  Returns a dict with
        user_ptr  int64 [U+1], user_item int32 [nnz], user_val fp32 [nnz]       (by user)
        rank_item_ptr int64 [P][I+1] (offsets into the next two), item_user int32 [nnz],
        item_val fp32 [nnz]                                                     (by rank, then item)
    """
    g = _rng(seed, _STREAM_MF)
    users = np.sort(g.integers(0, n_users, size=nnz, dtype=np.int64))
    items = np.minimum((n_items * g.random(nnz) ** 1.5).astype(np.int64), n_items - 1)
    a = _rng(seed, _STREAM_MF + 1).standard_normal((n_users, k_true)).astype(np.float32) / np.float32(np.sqrt(k_true))
    b = _rng(seed, _STREAM_MF + 2).standard_normal((n_items, k_true)).astype(np.float32) / np.float32(np.sqrt(k_true))
    val = np.empty(nnz, dtype=np.float32)
    chunk = 1 << 20
    for lo in range(0, nnz, chunk):
        hi = min(nnz, lo + chunk)
        clean = np.einsum("jk,jk->j", a[users[lo:hi]], b[items[lo:hi]])
        val[lo:hi] = clean + np.float32(noise) * _rng(seed, _STREAM_MF + 16 + lo // chunk).standard_normal(hi - lo, dtype=np.float32)
    # inside one user the ratings are ordered by item
    order = np.lexsort((items, users))
    users, items, val = users[order], items[order], val[order]
    user_ptr = np.zeros(n_users + 1, dtype=np.int64)
    np.cumsum(np.bincount(users, minlength=n_users), out=user_ptr[1:])
    rank_item_ptr = np.zeros((P, n_items + 1), dtype=np.int64)
    item_user = np.empty(nnz, dtype=np.int32)
    item_val = np.empty(nnz, dtype=np.float32)
    for r in range(P):
        lo, hi = int(user_ptr[r * n_users // P]), int(user_ptr[(r + 1) * n_users // P])
        by_item = np.argsort(items[lo:hi], kind="stable")
        item_user[lo:hi] = users[lo:hi][by_item]
        item_val[lo:hi] = val[lo:hi][by_item]
        rank_item_ptr[r, 0] = lo
        np.cumsum(np.bincount(items[lo:hi], minlength=n_items), out=rank_item_ptr[r, 1:])
        rank_item_ptr[r, 1:] += lo
    return {"user_ptr": user_ptr, "user_item": items.astype(np.int32), "user_val": val,
            "rank_item_ptr": rank_item_ptr, "item_user": item_user, "item_val": item_val,
            "n_users": n_users, "n_items": n_items, "nnz": nnz, "P": P}


def mf_init_factors(seed: int, n_users: int, n_items: int, k: int, scale: float = 0.1) -> tuple[np.ndarray, np.ndarray]:
    """Starting factors: small normal values, fp32 [U][k] and [I][k]."""
    pu = (scale * _rng(seed, _STREAM_MF + 3).standard_normal((n_users, k))).astype(np.float32)
    qi = (scale * _rng(seed, _STREAM_MF + 4).standard_normal((n_items, k))).astype(np.float32)
    return pu, qi


def mf_refresh_masks(seed: int, iters: int, P: int, S: int, p: float) -> list[np.ndarray]:
    """Per iteration the packed words [S][W]: the gradient of (rank, item segment) is delivered fresh
    with probability p (the others keep what they sent last)."""
    return [pack_mask(_rng(seed, _STREAM_MF + 1024 + t).random((P, S)) < p) for t in range(iters)]
