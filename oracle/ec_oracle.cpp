// CPU checker for the eventually consistent collectives.  TEST INFRASTRUCTURE ONLY.
//
// This file is the slow, plain statement of what the GPU library must compute.
// It is compiled on its own (g++ -O2 -ffp-contract=off, no fast-math), shares
// no header, helper, table or constant generator with the CUDA sources, and is
// called only by the tests, by the smoke check and by the benchmark's
// "cpu_baseline" leg.  The product never routes through it.
//
// Conventions (all pointers are HOST pointers):
//   P ranks, n elements per rank, seg elements per segment, S = ceil(n/seg);
//   segment s covers elements [s*seg, min(n,(s+1)*seg)).
//   Notification words: uint64 [S][W], W = ceil(P/64); the notification of rank
//   r for segment s is bit (r % 64) of word [s][r / 64]; bits >= P mean nothing.
//
// Passages followed:
//   * Sec. II (GASPI model): a contribution's bytes may be used only once its
//     notification is visible -> a buffer whose bit is 0 is never read.
//   * Sec. IV-A (segmented pipelined ring, Scatter-Reduce stage): every chunk
//     is reduced independently of the others; the operator is a global sum.
//     After the Allgather stage every node holds the complete reduction ->
//     once all bits are set the result is the plain allreduce.
//   * Sec. III (threshold and status parameters): the collective reports how
//     much took part -> contrib_count[s], the number of ranks folded in so far.
//   * Sec. IV-A Allgather stage / Sec. IV-B AlltoAll: every writer owns a fixed
//     slot and a notification of its own -> allgatherv slots come from the
//     counts of ALL ranks, whether they have arrived or not.
//
// Readings where the paper is silent (each also listed in the design notes):
//   order      one apply folds its newly arrived ranks in ascending rank order
//              onto what is already there;
//   start      a segment nobody has contributed to starts from the operator's
//              identity (+0.0, -inf/+inf, 0, INT64_MIN/MAX) and `result` is
//              not read; the first apply of an epoch writes the identity into
//              segments without contributors; later applies do not touch
//              segments without new arrivals;
//   int64 sum  wraps modulo 2^64;
//   float max  acc = (x > acc) ? x : acc   (min: x < acc);
//   bf16       raw bits widened exactly (bits << 16); arithmetic and output fp32;
//   ring       the vector is cut into P chunks of ceil(n/P) elements; chunk c is folded over the ranks
//              c, c+1, ..., c-1 (mod P), the order of the ring's Scatter-Reduce (Sec. IV-A);
//   pairwise   balanced binary tree over the rank index, P padded to a power of
//              two, absent ranks contribute the identity; a segment that already
//              holds a partial result gets the tree's root added onto it.
//
// Parity pins (tests/test_oracle_*.py, all run without a GPU): brute force over
// every mask on tiny inputs, integer-valued float data against exact integer
// sums, numpy/std library special cases for the scan and the concatenation,
// the rounding error bounds of sequential and pairwise summation, a
// scikit-learn Lloyd step for K-means with one rank.  The paper prints no
// numeric worked example for this path, so parity against absolute values of
// the paper is unpinned; everything above is pinned by mathematics.

#include <cstddef>
#include <cstdint>
#include <cstring>
#include <limits>
#include <new>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

enum { DT_F32 = 0, DT_BF16 = 1, DT_I64 = 2, DT_F64 = 3 };
enum { OP_SUM = 0, OP_MAX = 1, OP_MIN = 2 };
enum { ORDER_FIXED = 0, ORDER_PAIRWISE = 1, ORDER_RING = 2 };

inline bool notified(const uint64_t* mask, size_t W, size_t s, int r) {
    if (mask == nullptr) return true;  // no mask: every contribution has arrived
    const uint64_t word = mask[s * W + (size_t)(r / 64)];
    return ((word >> (r % 64)) & 1u) != 0;
}

inline float widen_bf16(uint16_t bits) {
    const uint32_t u = (uint32_t)bits << 16;
    float f;
    std::memcpy(&f, &u, sizeof f);
    return f;
}

// ---- element types: In = what a rank buffer holds, Acc = what result holds ----
struct F32 { typedef float In; typedef float Acc; static Acc widen(In x) { return x; } };
struct BF16 { typedef uint16_t In; typedef float Acc; static Acc widen(In x) { return widen_bf16(x); } };
struct F64 { typedef double In; typedef double Acc; static Acc widen(In x) { return x; } };
struct I64 { typedef int64_t In; typedef int64_t Acc; static Acc widen(In x) { return x; } };

template <class A> A identity_of(int op);
template <> float identity_of<float>(int op) {
    if (op == OP_SUM) return 0.0f;
    return op == OP_MAX ? -std::numeric_limits<float>::infinity() : std::numeric_limits<float>::infinity();
}
template <> double identity_of<double>(int op) {
    if (op == OP_SUM) return 0.0;
    return op == OP_MAX ? -std::numeric_limits<double>::infinity() : std::numeric_limits<double>::infinity();
}
template <> int64_t identity_of<int64_t>(int op) {
    if (op == OP_SUM) return 0;
    return op == OP_MAX ? std::numeric_limits<int64_t>::min() : std::numeric_limits<int64_t>::max();
}

inline float combine(int op, float a, float x) {
    if (op == OP_SUM) return a + x;
    if (op == OP_MAX) return (x > a) ? x : a;
    return (x < a) ? x : a;
}
inline double combine(int op, double a, double x) {
    if (op == OP_SUM) return a + x;
    if (op == OP_MAX) return (x > a) ? x : a;
    return (x < a) ? x : a;
}
inline int64_t combine(int op, int64_t a, int64_t x) {
    if (op == OP_SUM) return (int64_t)((uint64_t)a + (uint64_t)x);  // wraps; signed overflow would be undefined
    if (op == OP_MAX) return (x > a) ? x : a;
    return (x < a) ? x : a;
}

struct AllreduceState {
    int P; size_t n, seg, S, W; int dtype, op;
    std::vector<unsigned char> applied;  // [P][S]
    bool first_apply;
};

// Balanced tree over ranks [lo, hi) of element i; ranks not in `take` give the identity.
template <class T>
typename T::Acc tree_sum(const void* const* bufs, const unsigned char* take, int P, int lo, int hi,
                         size_t i, int op) {
    typedef typename T::Acc Acc;
    if (hi - lo == 1) {
        if (lo < P && take[lo]) return T::widen(((const typename T::In*)bufs[lo])[i]);
        return identity_of<Acc>(op);
    }
    const int mid = lo + (hi - lo) / 2;
    const Acc left = tree_sum<T>(bufs, take, P, lo, mid, i, op);
    const Acc right = tree_sum<T>(bufs, take, P, mid, hi, i, op);
    return combine(op, left, right);
}

template <class T>
void apply_typed(AllreduceState* st, const void* const* bufs, const uint64_t* mask, void* result_v,
                 uint32_t* contrib_count, int order, int threads) {
    typedef typename T::In In;
    typedef typename T::Acc Acc;
    Acc* result = (Acc*)result_v;
    const int P = st->P;
    const size_t S = st->S;
    int P2 = 1;
    while (P2 < P) P2 *= 2;
    (void)threads;
#pragma omp parallel for schedule(static) num_threads(threads)
    for (long long ss = 0; ss < (long long)S; ++ss) {
        const size_t s = (size_t)ss;
        const size_t lo = s * st->seg;
        const size_t hi = (lo + st->seg < st->n) ? lo + st->seg : st->n;
        // (1) what is the state of this segment?
        bool fresh = true, has_new = false;
        std::vector<unsigned char> take((size_t)P, 0);
        for (int r = 0; r < P; ++r) {
            const bool was = st->applied[(size_t)r * S + s] != 0;
            if (was) fresh = false;
            if (!was && notified(mask, st->W, s, r)) { take[(size_t)r] = 1; has_new = true; }
        }
        // (2) a segment nobody contributed to starts from the identity
        if (fresh && (has_new || st->first_apply)) {
            for (size_t i = lo; i < hi; ++i) result[i] = identity_of<Acc>(st->op);
        }
        // (3) fold the newly notified ranks
        if (has_new) {
            if (order == ORDER_RING) {
                // Scatter-Reduce of the segmented ring (Sec. IV-A): in step k node i sends chunk i-k and
                // receives chunk i-k-1, reducing it into its own data.  Chunk c therefore starts at node c
                // (step 0) and is reduced by nodes c+1, c+2, ... in turn: ranks c, c+1, ..., c-1 (mod P).
                const size_t chunk_len = (st->n + (size_t)P - 1) / (size_t)P;
                size_t c = lo / chunk_len;
                if (c > (size_t)(P - 1)) c = (size_t)(P - 1);
                for (int step = 0; step < P; ++step) {
                    const int r = (int)((c + (size_t)step) % (size_t)P);
                    if (!take[(size_t)r]) continue;
                    const In* buf = (const In*)bufs[r];
                    for (size_t i = lo; i < hi; ++i) result[i] = combine(st->op, result[i], T::widen(buf[i]));
                }
            } else if (order == ORDER_FIXED) {
                for (int r = 0; r < P; ++r) {
                    if (!take[(size_t)r]) continue;
                    const In* buf = (const In*)bufs[r];
                    for (size_t i = lo; i < hi; ++i) result[i] = combine(st->op, result[i], T::widen(buf[i]));
                }
            } else {
                for (size_t i = lo; i < hi; ++i) {
                    const Acc root = tree_sum<T>(bufs, take.data(), P, 0, P2, i, st->op);
                    result[i] = fresh ? root : combine(st->op, result[i], root);
                }
            }
            for (int r = 0; r < P; ++r)
                if (take[(size_t)r]) st->applied[(size_t)r * S + s] = 1;
        }
        // (4) status: how many ranks are in this segment's result now
        if (contrib_count != nullptr) {
            uint32_t c = 0;
            for (int r = 0; r < P; ++r)
                if (st->applied[(size_t)r * S + s]) ++c;
            contrib_count[s] = c;
        }
    }
    st->first_apply = false;
}

template <class T>
void oneshot_typed(int P, size_t n, size_t seg, int op, const void* const* bufs, const int32_t* order,
                   void* result_v) {
    typedef typename T::In In;
    typedef typename T::Acc Acc;
    Acc* result = (Acc*)result_v;
    const size_t S = (n + seg - 1) / seg;
    for (size_t s = 0; s < S; ++s) {
        const size_t lo = s * seg;
        const size_t hi = (lo + seg < n) ? lo + seg : n;
        for (size_t i = lo; i < hi; ++i) {
            Acc acc = identity_of<Acc>(op);
            for (int j = 0; j < P; ++j) {
                const int r = order[s * (size_t)P + (size_t)j];
                if (r < 0) break;
                acc = combine(op, acc, T::widen(((const In*)bufs[r])[i]));
            }
            result[i] = acc;
        }
    }
}

}  // namespace

extern "C" {

// ---------------------------------------------------------------------------
// allreduce
// ---------------------------------------------------------------------------
void* oracle_allreduce_new(int P, size_t n, int dtype, int op, size_t seg) {
    if (P < 1 || n == 0 || seg == 0 || dtype < 0 || dtype > 3 || op < 0 || op > 2) return nullptr;
    AllreduceState* st = new (std::nothrow) AllreduceState();
    if (!st) return nullptr;
    st->P = P; st->n = n; st->seg = seg; st->S = (n + seg - 1) / seg; st->W = (size_t)(P + 63) / 64;
    st->dtype = dtype; st->op = op;
    st->applied.assign((size_t)P * st->S, 0);
    st->first_apply = true;
    return st;
}

void oracle_allreduce_free(void* h) { delete (AllreduceState*)h; }

// New epoch: forget every notification that was consumed (Sec. II: notifications can be reset).
void oracle_allreduce_reset(void* h) {
    AllreduceState* st = (AllreduceState*)h;
    st->applied.assign(st->applied.size(), 0);
    st->first_apply = true;
}

// One apply: fold every contribution whose notification is set and that was not folded before.
// order: 0 = ascending rank order, 1 = pairwise tree.  Returns 0, or -1 on bad arguments.
int oracle_allreduce_apply(void* h, const void* const* bufs, const uint64_t* arrival_mask, void* result,
                           uint32_t* contrib_count, int order, int threads) {
    AllreduceState* st = (AllreduceState*)h;
    if (!st || !bufs || !result || threads < 1) return -1;
    switch (st->dtype) {
        case DT_F32: apply_typed<F32>(st, bufs, arrival_mask, result, contrib_count, order, threads); break;
        case DT_BF16: apply_typed<BF16>(st, bufs, arrival_mask, result, contrib_count, order, threads); break;
        case DT_I64: apply_typed<I64>(st, bufs, arrival_mask, result, contrib_count, order, threads); break;
        case DT_F64: apply_typed<F64>(st, bufs, arrival_mask, result, contrib_count, order, threads); break;
        default: return -1;
    }
    return 0;
}

// applied[r][s] as bytes, for tests.
void oracle_allreduce_applied(void* h, unsigned char* out) {
    AllreduceState* st = (AllreduceState*)h;
    std::memcpy(out, st->applied.data(), st->applied.size());
}

// One-shot fold of each segment in a given order: order is int32 [S][P], the ranks
// to fold for segment s from left to right, terminated by -1 if fewer than P.
int oracle_allreduce_oneshot(int P, size_t n, int dtype, int op, size_t seg, const void* const* bufs,
                             const int32_t* order, void* result) {
    if (P < 1 || n == 0 || seg == 0 || !bufs || !order || !result) return -1;
    switch (dtype) {
        case DT_F32: oneshot_typed<F32>(P, n, seg, op, bufs, order, result); break;
        case DT_BF16: oneshot_typed<BF16>(P, n, seg, op, bufs, order, result); break;
        case DT_I64: oneshot_typed<I64>(P, n, seg, op, bufs, order, result); break;
        case DT_F64: oneshot_typed<F64>(P, n, seg, op, bufs, order, result); break;
        default: return -1;
    }
    return 0;
}

// Double-precision sum of the notified contributions in rank order, plus the sum of
// their magnitudes (the scale of the rounding-error bound).  Floating dtypes only.
int oracle_allreduce_ref64(int P, size_t n, int dtype, size_t seg, const void* const* bufs,
                           const uint64_t* arrival_mask, double* ref, double* abs_sum) {
    if (P < 1 || n == 0 || seg == 0 || !bufs || !ref) return -1;
    if (dtype == DT_I64) return -1;
    const size_t W = (size_t)(P + 63) / 64;
    for (size_t i = 0; i < n; ++i) {
        const size_t s = i / seg;
        double acc = 0.0, mag = 0.0;
        for (int r = 0; r < P; ++r) {
            if (!notified(arrival_mask, W, s, r)) continue;
            double x;
            if (dtype == DT_F32) x = (double)((const float*)bufs[r])[i];
            else if (dtype == DT_BF16) x = (double)widen_bf16(((const uint16_t*)bufs[r])[i]);
            else x = ((const double*)bufs[r])[i];
            acc += x;
            mag += (x < 0 ? -x : x);
        }
        ref[i] = acc;
        if (abs_sum) abs_sum[i] = mag;
    }
    return 0;
}

// ---------------------------------------------------------------------------
// Stale-synchronous allreduce (Sec. III-A, Algorithm 1), stateless.
// Every rank buffer holds the last contribution that rank wrote for a segment, and
// notif_clock[s][r] is the clock (iteration) in which it was computed; 0 = nothing
// received yet.  As in the algorithm: min_clock_accepted = clock - slack; a received
// contribution whose clock is below it is too stale - the paper's process would wait
// for an update there; this sampled form leaves it out and counts it in wait_count.
// The others are reduced in rank order starting from the identity.  The clock of a
// reduction is the minimum of the clocks of what went into it (0 if nothing did).
// ---------------------------------------------------------------------------
int oracle_allreduce_ssp(int P, size_t n, int dtype, int op, size_t seg, const void* const* bufs,
                         const uint32_t* notif_clock, uint32_t clock, uint32_t slack, void* result,
                         uint32_t* contrib_count, uint32_t* seg_clock, uint32_t* wait_count) {
    if (P < 1 || n == 0 || seg == 0 || !bufs || !notif_clock || !result || clock == 0) return -1;
    const size_t S = (n + seg - 1) / seg;
    const long long min_clock_accepted = (long long)clock - (long long)slack;
    for (size_t s = 0; s < S; ++s) {
        const size_t lo = s * seg;
        const size_t hi = (lo + seg < n) ? lo + seg : n;
        uint32_t used = 0, waits = 0, oldest = 0;
        std::vector<int> order((size_t)P, -1);
        for (int r = 0; r < P; ++r) {
            const uint32_t rcv_clock = notif_clock[s * (size_t)P + (size_t)r];
            if (rcv_clock == 0 || (long long)rcv_clock < min_clock_accepted) { ++waits; continue; }   // too stale: would wait
            order[used++] = r;
            if (oldest == 0 || rcv_clock < oldest) oldest = rcv_clock;
        }
        for (size_t i = lo; i < hi; ++i) {
            switch (dtype) {
                case DT_F32: { float acc = identity_of<float>(op);
                    for (uint32_t j = 0; j < used; ++j) acc = combine(op, acc, ((const float*)bufs[order[j]])[i]);
                    ((float*)result)[i] = acc; break; }
                case DT_BF16: { float acc = identity_of<float>(op);
                    for (uint32_t j = 0; j < used; ++j) acc = combine(op, acc, widen_bf16(((const uint16_t*)bufs[order[j]])[i]));
                    ((float*)result)[i] = acc; break; }
                case DT_I64: { int64_t acc = identity_of<int64_t>(op);
                    for (uint32_t j = 0; j < used; ++j) acc = combine(op, acc, ((const int64_t*)bufs[order[j]])[i]);
                    ((int64_t*)result)[i] = acc; break; }
                case DT_F64: { double acc = identity_of<double>(op);
                    for (uint32_t j = 0; j < used; ++j) acc = combine(op, acc, ((const double*)bufs[order[j]])[i]);
                    ((double*)result)[i] = acc; break; }
                default: return -1;
            }
        }
        if (contrib_count) contrib_count[s] = used;
        if (seg_clock) seg_clock[s] = oldest;
        if (wait_count) wait_count[s] = waits;
    }
    return 0;
}

// ---------------------------------------------------------------------------
// allgatherv: fixed slots from the counts of all ranks; notified ranks are copied,
// the slots of the others are left as they were.
// Returns 0, or 1 if the total exceeds out_capacity (then nothing is copied;
// displs are still written).
// ---------------------------------------------------------------------------
int oracle_allgatherv(const void* const* bufs, const int64_t* counts, int P, size_t elem_bytes,
                      const uint64_t* arrival_mask, int64_t* displs, void* out, size_t out_capacity) {
    int64_t running = 0;
    for (int r = 0; r < P; ++r) {
        displs[r] = running;
        running += counts[r];
    }
    displs[P] = running;
    if ((uint64_t)running > (uint64_t)out_capacity) return 1;
    unsigned char* o = (unsigned char*)out;
    for (int r = 0; r < P; ++r) {
        if (!notified(arrival_mask, 1, 0, r)) continue;  // one word row: bit r of the [W] words
        const unsigned char* src = (const unsigned char*)bufs[r];
        for (int64_t e = 0; e < counts[r]; ++e)
            for (size_t b = 0; b < elem_bytes; ++b)
                o[((size_t)displs[r] + (size_t)e) * elem_bytes + b] = src[(size_t)e * elem_bytes + b];
    }
    return 0;
}

// The compact reading of "packed": only notified ranks get a slot; the gathered contributions are
// contiguous from out[0] on.  displs[r+1] - displs[r] = counts[r] if rank r is notified, else 0.
int oracle_allgatherv_compact(const void* const* bufs, const int64_t* counts, int P, size_t elem_bytes,
                              const uint64_t* arrival_mask, int64_t* displs, void* out, size_t out_capacity) {
    int64_t running = 0;
    for (int r = 0; r < P; ++r) {
        displs[r] = running;
        if (notified(arrival_mask, 1, 0, r)) running += counts[r];
    }
    displs[P] = running;
    if ((uint64_t)running > (uint64_t)out_capacity) return 1;
    unsigned char* o = (unsigned char*)out;
    for (int r = 0; r < P; ++r) {
        if (!notified(arrival_mask, 1, 0, r)) continue;
        const unsigned char* src = (const unsigned char*)bufs[r];
        for (size_t b = 0; b < (size_t)counts[r] * elem_bytes; ++b) o[(size_t)displs[r] * elem_bytes + b] = src[b];
    }
    return 0;
}

// ---------------------------------------------------------------------------
// AlltoAll (Sec. IV-B): every rank writes its d-th block into rank d's memory, each write with its
// own notification; the receiver uses what has been notified.  arrival_mask: uint64 [P][W], row d
// = destination, bit s = the block from source s has arrived (NULL = all).  Blocks that have not
// arrived are left as they were.  recv_count[d] = notified blocks of destination d.
// ---------------------------------------------------------------------------
int oracle_alltoall(const void* const* send_bufs, void* const* recv_bufs, int P, size_t block_bytes,
                    const uint64_t* arrival_mask, uint32_t* recv_count) {
    if (!send_bufs || !recv_bufs || P < 1 || block_bytes == 0) return -1;
    const size_t W = (size_t)(P + 63) / 64;
    for (int d = 0; d < P; ++d) {
        uint32_t got = 0;
        for (int s = 0; s < P; ++s) {
            if (!notified(arrival_mask, W, (size_t)d, s)) continue;
            ++got;
            const unsigned char* src = (const unsigned char*)send_bufs[s] + (size_t)d * block_bytes;
            unsigned char* dst = (unsigned char*)recv_bufs[d] + (size_t)s * block_bytes;
            for (size_t b = 0; b < block_bytes; ++b) dst[b] = src[b];
        }
        if (recv_count) recv_count[d] = got;
    }
    return 0;
}

// ---------------------------------------------------------------------------
// K-means (textbook Lloyd iteration; the data-parallel ML workload that stands
// in for the paper's iterative-convergent solver).  Distances in double.
// ---------------------------------------------------------------------------

// label[j] = argmin_k sum_d (x_jd - c_kd)^2, lowest k on equality.  Also the best
// and second-best squared distances (second = +inf when K == 1).
void oracle_kmeans_assign(const float* points, size_t N, int D, const float* centroids, int K,
                          int32_t* labels, double* best, double* second, int32_t* second_label,
                          int threads) {
    (void)threads;
#pragma omp parallel for schedule(static) num_threads(threads)
    for (long long jj = 0; jj < (long long)N; ++jj) {
        const size_t j = (size_t)jj;
        double d1 = std::numeric_limits<double>::infinity(), d2 = d1;
        int32_t k1 = -1, k2 = -1;
        for (int k = 0; k < K; ++k) {
            double dist = 0.0;
            for (int d = 0; d < D; ++d) {
                const double diff = (double)points[j * (size_t)D + (size_t)d] - (double)centroids[(size_t)k * D + d];
                dist += diff * diff;
            }
            if (dist < d1) { d2 = d1; k2 = k1; d1 = dist; k1 = k; }
            else if (dist < d2) { d2 = dist; k2 = k; }
        }
        labels[j] = k1;
        if (best) best[j] = d1;
        if (second) second[j] = d2;
        if (second_label) second_label[j] = k2;
    }
}

// Rank r owns points [r*N/P, (r+1)*N/P).  partials is fp32 [P][K][D+4]:
// columns 0..D-1 the sums of the rank's points with that label, column D the
// number of such points, columns D+1..D+3 zero.  Sums are accumulated in double
// in point order and rounded once.
void oracle_kmeans_partials(const float* points, size_t N, int D, int K, int P, const int32_t* labels,
                            float* partials, int threads) {
    const size_t stride = (size_t)D + 4;
    (void)threads;
#pragma omp parallel for schedule(static) num_threads(threads)
    for (int r = 0; r < P; ++r) {
        std::vector<double> sums((size_t)K * D, 0.0);
        std::vector<long long> cnt((size_t)K, 0);
        const size_t j0 = (size_t)r * N / (size_t)P, j1 = (size_t)(r + 1) * N / (size_t)P;
        for (size_t j = j0; j < j1; ++j) {
            const int32_t k = labels[j];
            for (int d = 0; d < D; ++d) sums[(size_t)k * D + d] += (double)points[j * (size_t)D + d];
            cnt[(size_t)k] += 1;
        }
        for (int k = 0; k < K; ++k) {
            float* row = partials + ((size_t)r * K + (size_t)k) * stride;
            for (int d = 0; d < D; ++d) row[d] = (float)sums[(size_t)k * D + d];
            row[D] = (float)cnt[(size_t)k];
            row[D + 1] = row[D + 2] = row[D + 3] = 0.0f;
        }
    }
}

// reduced is fp32 [K][D+4] (the allreduce result).  A centroid with at least one
// point becomes sums / points; one without keeps its old position.
void oracle_kmeans_update(const float* reduced, int D, int K, const float* old_centroids, float* new_centroids) {
    const size_t stride = (size_t)D + 4;
    for (int k = 0; k < K; ++k) {
        const float pts = reduced[(size_t)k * stride + (size_t)D];
        for (int d = 0; d < D; ++d) {
            if (pts > 0.0f) new_centroids[(size_t)k * D + d] = reduced[(size_t)k * stride + d] / pts;
            else new_centroids[(size_t)k * D + d] = old_centroids[(size_t)k * D + d];
        }
    }
}

int oracle_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

}  // extern "C"
