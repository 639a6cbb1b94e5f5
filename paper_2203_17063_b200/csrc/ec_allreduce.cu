// Eventually consistent allreduce: the segment-wise combine of P rank buffers.
//
// One launch per apply.  A thread block owns one tile of one segment.  Its first
// warp reads the segment's notification words and the "already folded in" words,
// takes the difference (what is new), and - by ballot - decides whether the
// segment has news at all and whether it ever had a contributor.  The block then
// brings in the tile of every new rank - by bulk asynchronous copies through a
// small ring of shared-memory stages (apply_bulk_kernel: up to 64 ranks, 128-bit
// aligned calls), by direct 128-bit loads (apply_kernel: wide rank tables, the
// pairwise tree, unaligned calls), or all at once for short segments
// (apply_short_kernel) - folds in ascending rank order (or as a pairwise tree)
// and writes the result tile.  The block of tile 0
// also writes the segment's updated words and its contributor count.  The folded
// words are double buffered (read one copy, write the other) so that no block can
// see another block's update: there is no inter-block dependency and no wait.
//
// Follows Sec. IV-A (each chunk of the vector is reduced independently, global
// sum), Sec. II (a contribution is used only once its notification is visible)
// and Sec. III (status output: how many took part).

#include <new>

#include "ec_common.cuh"

namespace ec {

thread_local int g_last_cuda_error = 0;

namespace {

// ---------------------------------------------------------------------------------------------
// element types
// ---------------------------------------------------------------------------------------------
template <int DT> struct Elem;
template <> struct Elem<EC_F32> {
    typedef float In; typedef float Acc;
    static constexpr int VEC = 4;  // elements per 16 input bytes
    __device__ static __forceinline__ void unpack(const uint4& r, Acc (&x)[VEC]) {
        x[0] = __uint_as_float(r.x); x[1] = __uint_as_float(r.y); x[2] = __uint_as_float(r.z); x[3] = __uint_as_float(r.w);
    }
    __device__ static __forceinline__ Acc widen(In v) { return v; }
};
template <> struct Elem<EC_BF16> {
    typedef uint16_t In; typedef float Acc;
    static constexpr int VEC = 8;
    __device__ static __forceinline__ void unpack(const uint4& r, Acc (&x)[VEC]) {
        // element 2k is the low half of word k, 2k+1 the high half; widening = bits << 16, exact
        x[0] = __uint_as_float(r.x << 16); x[1] = __uint_as_float(r.x & 0xFFFF0000u);
        x[2] = __uint_as_float(r.y << 16); x[3] = __uint_as_float(r.y & 0xFFFF0000u);
        x[4] = __uint_as_float(r.z << 16); x[5] = __uint_as_float(r.z & 0xFFFF0000u);
        x[6] = __uint_as_float(r.w << 16); x[7] = __uint_as_float(r.w & 0xFFFF0000u);
    }
    __device__ static __forceinline__ Acc widen(In v) { return __uint_as_float((uint32_t)v << 16); }
};
template <> struct Elem<EC_I64> {
    typedef long long In; typedef long long Acc;
    static constexpr int VEC = 2;
    __device__ static __forceinline__ void unpack(const uint4& r, Acc (&x)[VEC]) {
        x[0] = (long long)((unsigned long long)r.x | ((unsigned long long)r.y << 32));
        x[1] = (long long)((unsigned long long)r.z | ((unsigned long long)r.w << 32));
    }
    __device__ static __forceinline__ Acc widen(In v) { return v; }
};
template <> struct Elem<EC_F64> {
    typedef double In; typedef double Acc;
    static constexpr int VEC = 2;
    __device__ static __forceinline__ void unpack(const uint4& r, Acc (&x)[VEC]) {
        x[0] = __longlong_as_double((long long)((unsigned long long)r.x | ((unsigned long long)r.y << 32)));
        x[1] = __longlong_as_double((long long)((unsigned long long)r.z | ((unsigned long long)r.w << 32)));
    }
    __device__ static __forceinline__ Acc widen(In v) { return v; }
};

// ---------------------------------------------------------------------------------------------
// operators.  Sums use the explicit round-to-nearest intrinsics: never contracted, never reordered.
// ---------------------------------------------------------------------------------------------
template <int OP> __device__ __forceinline__ float comb(float a, float x) {
    if (OP == EC_SUM) return __fadd_rn(a, x);
    if (OP == EC_MAX) return (x > a) ? x : a;
    return (x < a) ? x : a;
}
template <int OP> __device__ __forceinline__ double comb(double a, double x) {
    if (OP == EC_SUM) return __dadd_rn(a, x);
    if (OP == EC_MAX) return (x > a) ? x : a;
    return (x < a) ? x : a;
}
template <int OP> __device__ __forceinline__ long long comb(long long a, long long x) {
    if (OP == EC_SUM) return (long long)((unsigned long long)a + (unsigned long long)x);
    if (OP == EC_MAX) return (x > a) ? x : a;
    return (x < a) ? x : a;
}
template <int OP> __device__ __forceinline__ float ident(float) {
    return OP == EC_SUM ? 0.0f : OP == EC_MAX ? -__int_as_float(0x7f800000) : __int_as_float(0x7f800000);
}
template <int OP> __device__ __forceinline__ double ident(double) {
    return OP == EC_SUM ? 0.0 : OP == EC_MAX ? -__longlong_as_double(0x7ff0000000000000LL)
                                             : __longlong_as_double(0x7ff0000000000000LL);
}
template <int OP> __device__ __forceinline__ long long ident(long long) {
    return OP == EC_SUM ? 0LL : OP == EC_MAX ? (long long)0x8000000000000000ULL : 0x7fffffffffffffffLL;
}

// accumulator vector <-> result memory (VEC accumulators = VEC*sizeof(Acc)/16 stores of 16 bytes)
template <class Acc, int VEC>
__device__ __forceinline__ void load_acc(const Acc* p, Acc (&acc)[VEC], uint64_t rpol) {
    constexpr int PER = 16 / sizeof(Acc);
#pragma unroll
    for (int q = 0; q < VEC / PER; ++q) {
        const uint4 r = ld_hint16(p + q * PER, rpol);
        if (sizeof(Acc) == 4) {
            acc[q * PER + 0] = (Acc)__uint_as_float(r.x); acc[q * PER + 1] = (Acc)__uint_as_float(r.y);
            acc[q * PER + 2] = (Acc)__uint_as_float(r.z); acc[q * PER + 3] = (Acc)__uint_as_float(r.w);
        } else {
            const unsigned long long a = (unsigned long long)r.x | ((unsigned long long)r.y << 32);
            const unsigned long long b = (unsigned long long)r.z | ((unsigned long long)r.w << 32);
            memcpy(&acc[q * PER + 0], &a, 8);
            memcpy(&acc[q * PER + 1], &b, 8);
        }
    }
}
template <class Acc, int VEC>
__device__ __forceinline__ void store_acc(Acc* p, const Acc (&acc)[VEC], uint64_t rpol) {
    constexpr int PER = 16 / sizeof(Acc);
#pragma unroll
    for (int q = 0; q < VEC / PER; ++q) {
        uint4 r;
        if (sizeof(Acc) == 4) {
            uint32_t w[4];
            memcpy(w, &acc[q * PER], 16);
            r = make_uint4(w[0], w[1], w[2], w[3]);
        } else {
            unsigned long long w[2];
            memcpy(w, &acc[q * PER], 16);
            r = make_uint4((uint32_t)w[0], (uint32_t)(w[0] >> 32), (uint32_t)w[1], (uint32_t)(w[1] >> 32));
        }
        st_hint16(p + q * PER, r, rpol);
    }
}

struct ApplyArgs {
    size_t n, seg, tile;
    const uint64_t* arrival;     // [S][W] or nullptr
    const uint64_t* applied_in;  // [S][W]
    uint64_t* applied_out;       // [S][W]
    void* result;
    uint32_t* contrib_count;     // [S] or nullptr
    unsigned tiles_per_seg;
    int P, W, first_apply;
    int res_hint;                // 1: the result fits in L2 (stores keep it there), 2: it does not (stores stream out)
    // stale-synchronous mode: acceptance by clock instead of by notification bit (all nullptr / 0 otherwise)
    const uint32_t* notif_clock; // [S][P] clock of the contribution each rank buffer holds; 0 = none
    uint32_t min_clock;          // contributions with clock >= min_clock are accepted
    uint32_t* seg_clock;         // [S] or nullptr: smallest clock among the accepted, 0 if none
    uint32_t* wait_count;        // [S] or nullptr: ranks whose contribution is too stale
    size_t ring_chunk;           // ring order: elements per 1/P chunk of the vector (0 = plain rank order)
    int dependent;               // host side only: launch as a programmatic dependent of the stream's previous kernel
};

// Shape of the streaming loop, chosen by measurement on B200 (config 2 and 3 epochs): what counts
// is resident threads, not loads per thread - 40 registers (6 blocks of 256 threads per SM) beat
// 64 and 96 registers by 2 % and 20 %; spilling to reach 32 loses 10 %.
#ifndef EC_MAXT
#define EC_MAXT 256      // largest block size
#endif
#ifndef EC_MINB
#define EC_MINB 6        // resident blocks of EC_MAXT threads the register allocation must allow
#endif
#ifndef EC_MAIN_RU
#define EC_MAIN_RU 4     // first rounds: rank loads in flight per result vector
#endif
#ifndef EC_LATE_VPT
#define EC_LATE_VPT 2    // late rounds with <= EC_LATE_RU new ranks: result vectors per thread
#endif
#ifndef EC_LATE_RU
#define EC_LATE_RU 2
#endif
#ifndef EC_MID_VPT
#define EC_MID_VPT 1
#endif
#ifndef EC_MID_RU
#define EC_MID_RU 4
#endif
constexpr int RU = 8;        // rank buffers whose loads are issued together (independent loads, ordered adds)
constexpr int MAX_W = EC_MAX_RANKS / 64;
constexpr int TREE_LEVELS = 7;  // 1024 ranks / 8 per leaf block = 128 blocks = 2^7

// Fold the m new ranks into VPT result vectors per thread, RU rank loads per vector in flight.
// Loads are independent and issued together; the adds of one vector stay in ascending rank order.
template <int DT, int OP, int VPT, int RUN>
__device__ __forceinline__ void fold_vectors(const char* const* s_ptr, int m, typename Elem<DT>::Acc* res, size_t nvec,
                                             bool fresh, int tid, int nthr, uint64_t pol, uint64_t rpol_ld, uint64_t rpol_st) {
    typedef Elem<DT> E;
    typedef typename E::Acc Acc;
    constexpr int VEC = E::VEC;
    for (size_t v0 = tid; v0 < nvec; v0 += (size_t)nthr * VPT) {
        Acc acc[VPT][VEC];
#pragma unroll
        for (int p = 0; p < VPT; ++p) {
            const size_t v = v0 + (size_t)p * nthr;
            if (fresh || v >= nvec) {
#pragma unroll
                for (int e = 0; e < VEC; ++e) acc[p][e] = ident<OP>(Acc());
            } else {
                load_acc<Acc, VEC>(res + v * VEC, acc[p], rpol_ld);
            }
        }
        for (int j = 0; j < m; j += RUN) {
            uint4 raw[VPT][RUN];
#pragma unroll
            for (int p = 0; p < VPT; ++p) {
                const size_t v = v0 + (size_t)p * nthr;
#pragma unroll
                for (int u = 0; u < RUN; ++u)
                    if (j + u < m && v < nvec) raw[p][u] = ld_stream16(s_ptr[j + u] + v * 16, pol);
            }
#pragma unroll
            for (int p = 0; p < VPT; ++p) {
                const size_t v = v0 + (size_t)p * nthr;
#pragma unroll
                for (int u = 0; u < RUN; ++u) {
                    if (j + u < m && v < nvec) {
                        Acc x[VEC];
                        E::unpack(raw[p][u], x);
#pragma unroll
                        for (int e = 0; e < VEC; ++e) acc[p][e] = comb<OP>(acc[p][e], x[e]);
                    }
                }
            }
        }
#pragma unroll
        for (int p = 0; p < VPT; ++p) {
            const size_t v = v0 + (size_t)p * nthr;
            if (v < nvec) store_acc<Acc, VEC>(res + v * VEC, acc[p], rpol_st);
        }
    }
}

// Prologue of a block, run by its first warp: which ranks are new for segment s (notification words or
// clocks), the bookkeeping outputs (block t == 0 of the segment writes them), and the ascending (or ring-
// rotated) list of the new ranks in shared memory.
// If s_ptr is given, the address of every listed rank's data (table entry + byte_off) is written beside its rank.
// Returns the number of new ranks (in every lane).
__device__ __forceinline__ int block_prologue(const ApplyArgs& a, unsigned s, unsigned t, uint16_t* s_rank,
                                              uint64_t* s_new, int* s_m, int* s_fresh,
                                              const void* const* table = nullptr, size_t byte_off = 0,
                                              const char** s_ptr = nullptr) {
            const int lane = threadIdx.x;
            uint64_t nw = 0, old = 0;
            if (a.notif_clock != nullptr) {
                // Stale-synchronous acceptance (Algorithm 1): a contribution takes part if its clock is not older
                // than clock - slack.  32 ranks per step; the ballots of two steps make one 64-rank word.
                uint32_t mn = 0xffffffffu;
                int stale = 0;
                for (int c = 0; c * 32 < a.P; ++c) {
                    const int r = c * 32 + lane;
                    const uint32_t ck = r < a.P ? a.notif_clock[(size_t)s * a.P + r] : 0u;
                    const bool ok = r < a.P && ck >= a.min_clock;
                    const unsigned bal = __ballot_sync(0xffffffffu, ok);
                    if (ok) mn = ck < mn ? ck : mn;
                    stale += (r < a.P && !ok) ? 1 : 0;
                    if (lane == (c >> 1)) nw |= (uint64_t)bal << ((c & 1) * 32);
                }
    #pragma unroll
                for (int d = 16; d > 0; d >>= 1) {
                    const uint32_t o = __shfl_xor_sync(0xffffffffu, mn, d);
                    mn = o < mn ? o : mn;
                    stale += __shfl_xor_sync(0xffffffffu, stale, d);
                }
                if (t == 0 && lane == 0) {
                    if (a.seg_clock) a.seg_clock[s] = mn == 0xffffffffu ? 0u : mn;   // the result is as old as its oldest input
                    if (a.wait_count) a.wait_count[s] = (uint32_t)stale;
                }
            } else if (lane < a.W) {
                uint64_t arr = a.arrival ? a.arrival[(size_t)s * a.W + lane] : ~0ull;
                if (lane == a.W - 1 && (a.P & 63)) arr &= (1ull << (a.P & 63)) - 1;   // bits >= P mean nothing
                // the first apply of an epoch starts from "nothing folded in": no need to clear the words
                old = a.first_apply ? 0ull : a.applied_in[(size_t)s * a.W + lane];
                nw = arr & ~old;
            }
            const unsigned any_new = __ballot_sync(0xffffffffu, nw != 0);
            const unsigned any_old = __ballot_sync(0xffffffffu, old != 0);
            const int cnt_new = __popcll(nw);
            int incl = cnt_new, total = __popcll(nw | old);
    #pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int y = __shfl_up_sync(0xffffffffu, incl, d);
                if (lane >= d) incl += y;
                total += __shfl_xor_sync(0xffffffffu, total, d);
            }
            if (t == 0) {
                if (lane < a.W && a.notif_clock == nullptr) a.applied_out[(size_t)s * a.W + lane] = old | nw;
                if (lane == 0 && a.contrib_count) a.contrib_count[s] = (uint32_t)total;
            }
            if (lane < MAX_W) s_new[lane] = nw;
            // Ring order (Scatter-Reduce of the segmented ring, Sec. IV-A): chunk c of the vector is first sent by
            // node c and reduced by nodes c+1, c+2, ... in turn, so its fold starts at rank c and wraps around.
            // The ascending list is rotated: the j0 ranks below c go to the end.
            const int m_all = __shfl_sync(0xffffffffu, incl, 31);
            int j0 = 0;
            if (a.ring_chunk != 0) {
                size_t c = ((size_t)s * a.seg) / a.ring_chunk;
                if (c > (size_t)(a.P - 1)) c = (size_t)(a.P - 1);
                const int rel = (int)c - lane * 64;                       // ranks of this word below c
                const uint64_t below = rel <= 0 ? 0ull : rel >= 64 ? ~0ull : (1ull << rel) - 1;
                j0 = __popcll(nw & below);
    #pragma unroll
                for (int d = 16; d > 0; d >>= 1) j0 += __shfl_xor_sync(0xffffffffu, j0, d);
            }
            // The list of new ranks, ascending (rotated for the ring order): word by word, every lane places
            // the two ranks it owns in the word at the position the popcount of the lower bits gives.
            const int excl = incl - cnt_new;                              // new ranks in the words before this lane's
            for (int wd = 0; wd < a.W; ++wd) {
                const uint32_t lo32 = __shfl_sync(0xffffffffu, (uint32_t)nw, wd);
                const uint32_t hi32 = __shfl_sync(0xffffffffu, (uint32_t)(nw >> 32), wd);
                const int base = __shfl_sync(0xffffffffu, excl, wd);
                const uint64_t word = ((uint64_t)hi32 << 32) | lo32;
                if (word == 0) continue;
    #pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int b = half * 32 + lane;
                    if ((word >> b) & 1ull) {
                        const int j = base + __popcll(word & ((1ull << b) - 1ull));
                        const int pos = j >= j0 ? j - j0 : j + (m_all - j0);
                        s_rank[pos] = (uint16_t)(wd * 64 + b);
                        if (s_ptr != nullptr) s_ptr[pos] = reinterpret_cast<const char*>(table[wd * 64 + b]) + byte_off;
                    }
                }
            }
            if (lane == 31) *s_m = incl;
            if (lane == 0) *s_fresh = (any_old == 0) ? 1 : 0;
            (void)any_new;
            return m_all;
}

// ---------------------------------------------------------------------------------------------
// the apply kernel
// ---------------------------------------------------------------------------------------------
#ifndef EC_PW_MINB
#define EC_PW_MINB 2
#endif
template <int DT, int OP, bool VECTOR, int CAP, int ORDER>
__global__ void __launch_bounds__(EC_MAXT, (ORDER != EC_ORDER_FIXED ? (CAP > 64 ? 2 : EC_PW_MINB) : CAP > 64 ? 4 : EC_MINB))   // tree and wide-table variants need more registers
apply_kernel(const ApplyArgs a, const __grid_constant__ PtrTable<CAP> tbl) {
    grid_dependency_wait();            // (a no-op unless launched as a programmatic dependent)
    typedef Elem<DT> E;
    typedef typename E::In In;
    typedef typename E::Acc Acc;
    constexpr int VEC = E::VEC;

    __shared__ const char* s_ptr[CAP];   // tile base of every new rank, ascending
    __shared__ uint16_t s_rank[CAP];
    __shared__ uint64_t s_new[MAX_W];
    __shared__ int s_m, s_fresh;

    const unsigned s = blockIdx.x / a.tiles_per_seg;
    const unsigned t = blockIdx.x - s * a.tiles_per_seg;
    const size_t lo = (size_t)s * a.seg + (size_t)t * a.tile;
    size_t seg_hi = (size_t)(s + 1) * a.seg;
    if (seg_hi > a.n) seg_hi = a.n;

    if (threadIdx.x < 32) block_prologue(a, s, t, s_rank, s_new, &s_m, &s_fresh);
    __syncthreads();
    const int m = s_m;
    const bool fresh = s_fresh != 0;
    if (m == 0 && !(fresh && a.first_apply)) return;   // nothing new: the segment is neither read nor written
    if (lo >= seg_hi) return;                          // tile beyond a short last segment
    size_t hi = lo + a.tile;
    if (hi > seg_hi) hi = seg_hi;
    const size_t cnt = hi - lo;
    Acc* res = reinterpret_cast<Acc*>(a.result) + lo;
    const int tid = threadIdx.x, nthr = blockDim.x;
    const uint64_t pol = evict_first_policy();
    // Result accesses (measured on config 2 and 3 epochs): loads always keep the line in L2 (evict-last: the
    // next round reads it again); stores keep it too when the whole result fits in L2, and let it go at once
    // (evict-first) when it cannot fit anyway.
    const uint64_t rpol_ld = result_policy(1), rpol_st = result_policy(a.res_hint == 2 ? 2 : 1);

    if (ORDER == EC_ORDER_FIXED) {
        for (int j = tid; j < m; j += nthr)
            s_ptr[j] = reinterpret_cast<const char*>(tbl.p[s_rank[j]]) + lo * sizeof(In);
        __syncthreads();
        const size_t nvec = VECTOR ? cnt / VEC : 0;
        // Few new ranks (a late round): each thread keeps several result vectors in flight;
        // many new ranks (a first round): one vector per thread, eight rank loads in flight.
        // With hundreds of ranks a round rarely brings that few: the wide-table variant keeps the
        // single shape.
        constexpr int LATE = EC_LATE_VPT, MID = EC_MID_VPT;
        if (CAP <= 64 && m <= EC_LATE_RU) fold_vectors<DT, OP, LATE, EC_LATE_RU>(s_ptr, m, res, nvec, fresh, tid, nthr, pol, rpol_ld, rpol_st);
        else if (CAP <= 64 && m <= EC_MID_RU) fold_vectors<DT, OP, MID, EC_MID_RU>(s_ptr, m, res, nvec, fresh, tid, nthr, pol, rpol_ld, rpol_st);
        else fold_vectors<DT, OP, 1, (CAP > 64 ? 8 : EC_MAIN_RU)>(s_ptr, m, res, nvec, fresh, tid, nthr, pol, rpol_ld, rpol_st);   // hundreds of ranks: 8 loads in flight measured best
        // element-wise path: everything when the 128-bit path does not apply, else the ragged tail
        for (size_t i = nvec * VEC + tid; i < cnt; i += nthr) {
            Acc acc = fresh ? ident<OP>(Acc()) : res[i];
            for (int j = 0; j < m; j += RU) {
                In raw[RU];
#pragma unroll
                for (int u = 0; u < RU; ++u)
                    if (j + u < m) raw[u] = reinterpret_cast<const In*>(s_ptr[j + u])[i];
#pragma unroll
                for (int u = 0; u < RU; ++u)
                    if (j + u < m) acc = comb<OP>(acc, E::widen(raw[u]));
            }
            res[i] = acc;
        }
    } else {
        // Pairwise: balanced binary tree over the rank index, P padded to a power of two, ranks that
        // are not new contribute the identity.  Leaves are taken eight ranks at a time (a complete
        // three-level subtree); the subtrees are merged with a binary counter, which reproduces the
        // recursive halving tree exactly.
        int P2 = 1;
        while (P2 < a.P) P2 <<= 1;
        const int leaf = P2 < 8 ? P2 : 8;
        const int nblk = P2 / leaf;
        int nlev = 0;
        while ((1 << nlev) < nblk) ++nlev;
        // Units of PV elements (at most four accumulators per tree node keeps the tree in registers).
        constexpr int PV = VEC > 4 ? 4 : VEC;
        const size_t nvec = VECTOR ? cnt / PV : 0;
        const size_t nunits = nvec + (cnt - nvec * PV);   // vectors first, then single elements
        for (size_t w = tid; w < nunits; w += nthr) {
            const bool isvec = w < nvec;
            const size_t e0 = isvec ? w * PV : nvec * PV + (w - nvec);   // first element of this unit
            constexpr int LEVELS = CAP <= 64 ? 3 : TREE_LEVELS;     // 64 ranks / 8 per leaf block = 2^3 blocks
            Acc stack[LEVELS][PV];
            Acc node[PV];
            // bf16 moves only 8 bytes per rank and thread: the loads of the next leaf block are issued before
            // the current one is reduced, so that twice as many bytes are in flight
            uint2 pre[8];
            auto fetch8 = [&](int blk_i) {
                const int q0 = blk_i * leaf;
                const unsigned bt = (unsigned)(s_new[q0 >> 6] >> (q0 & 63)) & ((1u << leaf) - 1u);
#pragma unroll
                for (int u = 0; u < 8; ++u)
                    if ((bt >> u) & 1u)
                        pre[u] = ld_stream8(reinterpret_cast<const char*>(tbl.p[q0 + u]) + (lo + e0) * sizeof(In), pol);
            };
            if constexpr (DT == EC_BF16) {
                if (isvec) fetch8(0);
            }
            for (int blk = 0; blk < nblk; ++blk) {
                const int r0 = blk * leaf;
                const unsigned byte = (unsigned)(s_new[r0 >> 6] >> (r0 & 63)) & ((1u << leaf) - 1u);
                Acc lv[8][PV];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
#pragma unroll
                    for (int e = 0; e < PV; ++e) lv[u][e] = ident<OP>(Acc());
                }
                uint2 raw[8];                                  // bf16: four values = 8 bytes per rank
                if constexpr (DT == EC_BF16) {
                    if (isvec) {
#pragma unroll
                        for (int u = 0; u < 8; ++u) raw[u] = pre[u];
                        if (blk + 1 < nblk) fetch8(blk + 1);
                    }
                }
                if (byte != 0) {
                    if (isvec) {
                        if constexpr (DT == EC_BF16) {
#pragma unroll
                            for (int u = 0; u < 8; ++u)
                                if ((byte >> u) & 1u) {
                                    lv[u][0] = __uint_as_float(raw[u].x << 16); lv[u][1] = __uint_as_float(raw[u].x & 0xFFFF0000u);
                                    lv[u][2] = __uint_as_float(raw[u].y << 16); lv[u][3] = __uint_as_float(raw[u].y & 0xFFFF0000u);
                                }
                        } else {
                            uint4 raw[8];
#pragma unroll
                            for (int u = 0; u < 8; ++u)
                                if ((byte >> u) & 1u)
                                    raw[u] = ld_stream16(reinterpret_cast<const char*>(tbl.p[r0 + u]) + (lo + e0) * sizeof(In), pol);
#pragma unroll
                            for (int u = 0; u < 8; ++u)
                                if ((byte >> u) & 1u) E::unpack(raw[u], lv[u]);
                        }
                    } else {
#pragma unroll
                        for (int u = 0; u < 8; ++u)
                            if ((byte >> u) & 1u) lv[u][0] = E::widen(reinterpret_cast<const In*>(tbl.p[r0 + u])[lo + e0]);
                    }
                }
#pragma unroll
                for (int e = 0; e < PV; ++e) {
                    if (leaf == 8)
                        node[e] = comb<OP>(comb<OP>(comb<OP>(lv[0][e], lv[1][e]), comb<OP>(lv[2][e], lv[3][e])),
                                           comb<OP>(comb<OP>(lv[4][e], lv[5][e]), comb<OP>(lv[6][e], lv[7][e])));
                    else if (leaf == 4)
                        node[e] = comb<OP>(comb<OP>(lv[0][e], lv[1][e]), comb<OP>(lv[2][e], lv[3][e]));
                    else if (leaf == 2)
                        node[e] = comb<OP>(lv[0][e], lv[1][e]);
                    else
                        node[e] = lv[0][e];
                }
                bool carry = true;
#pragma unroll
                for (int l = 0; l < LEVELS; ++l) {
                    if (l < nlev && carry) {
                        if ((blk >> l) & 1) {
#pragma unroll
                            for (int e = 0; e < PV; ++e) node[e] = comb<OP>(stack[l][e], node[e]);
                        } else {
#pragma unroll
                            for (int e = 0; e < PV; ++e) stack[l][e] = node[e];
                            carry = false;
                        }
                    }
                }
            }
            // node is the root now
            if (isvec) {
                if (!fresh) {
                    Acc acc[PV];
                    load_acc<Acc, PV>(res + e0, acc, rpol_ld);
#pragma unroll
                    for (int e = 0; e < PV; ++e) node[e] = comb<OP>(acc[e], node[e]);
                }
                store_acc<Acc, PV>(res + e0, node, rpol_st);
            } else {
                res[e0] = fresh ? node[0] : comb<OP>(res[e0], node[0]);
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// the apply kernel for short segments
// ---------------------------------------------------------------------------------------------
// A short segment and many ranks (the rows of a small model, e.g. one centroid row per segment): only a few
// threads own a result vector, and the streaming fold, which fetches four ranks at a time, would be a chain of
// m / 4 memory round trips.  Here one block takes a whole segment; all its threads fetch the (rank, vector)
// items of up to STAGE / nv ranks into shared memory at once, then the owners fold them from there in ascending
// rank order.  Same prologue, same order of additions, same bits as apply_kernel.
constexpr int STAGE = 512;           // 16-byte items staged per pass
template <int DT, int OP, int CAP>
__global__ void __launch_bounds__(EC_MAXT)
apply_short_kernel(const ApplyArgs a, const __grid_constant__ PtrTable<CAP> tbl) {
    grid_dependency_wait();            // (a no-op unless launched as a programmatic dependent)
    typedef Elem<DT> E;
    typedef typename E::In In;
    typedef typename E::Acc Acc;
    constexpr int VEC = E::VEC;

    __shared__ const char* s_ptr[CAP];
    __shared__ uint16_t s_rank[CAP];
    __shared__ uint64_t s_new[MAX_W];
    __shared__ int s_m, s_fresh;
    __shared__ uint4 s_stage[STAGE];

    const unsigned s = blockIdx.x;
    const size_t lo = (size_t)s * a.seg;
    size_t hi = lo + a.seg;
    if (hi > a.n) hi = a.n;
    if (threadIdx.x < 32) block_prologue(a, s, 0u, s_rank, s_new, &s_m, &s_fresh);
    __syncthreads();
    const int m = s_m;
    const bool fresh = s_fresh != 0;
    if (m == 0 && !(fresh && a.first_apply)) return;   // nothing new: the segment is neither read nor written
    const size_t cnt = hi - lo;
    Acc* res = reinterpret_cast<Acc*>(a.result) + lo;
    const int tid = threadIdx.x, nthr = blockDim.x;
    const uint64_t pol = evict_first_policy();
    const uint64_t rpol = result_policy(1);            // a result this small stays in L2
    for (int j = tid; j < m; j += nthr)
        s_ptr[j] = reinterpret_cast<const char*>(tbl.p[s_rank[j]]) + lo * sizeof(In);
    __syncthreads();
    const int nv = (int)(cnt / VEC);                   // at most nthr / 4 (the host chose this kernel for that)
    if (nv > 0) {
        const int per_pass = STAGE / nv;
        Acc acc[VEC];
        if (tid < nv) {
            if (fresh) {
#pragma unroll
                for (int e = 0; e < VEC; ++e) acc[e] = ident<OP>(Acc());
            } else {
                load_acc<Acc, VEC>(res + (size_t)tid * VEC, acc, rpol);
            }
        }
        for (int j0 = 0; j0 < m; j0 += per_pass) {
            const int rr = m - j0 < per_pass ? m - j0 : per_pass;
#pragma unroll 4
            for (int i = tid; i < rr * nv; i += nthr) {
                const int j = i / nv, v = i - j * nv;
                s_stage[i] = ld_stream16(s_ptr[j0 + j] + (size_t)v * 16, pol);
            }
            __syncthreads();
            if (tid < nv) {
                for (int j = 0; j < rr; ++j) {
                    Acc x[VEC];
                    E::unpack(s_stage[j * nv + tid], x);
#pragma unroll
                    for (int e = 0; e < VEC; ++e) acc[e] = comb<OP>(acc[e], x[e]);
                }
            }
            __syncthreads();
        }
        if (tid < nv) store_acc<Acc, VEC>(res + (size_t)tid * VEC, acc, rpol);
    }
    // ragged tail of a short last segment, element by element
    for (size_t i = (size_t)nv * VEC + tid; i < cnt; i += nthr) {
        Acc acc = fresh ? ident<OP>(Acc()) : res[i];
        for (int j = 0; j < m; ++j) acc = comb<OP>(acc, E::widen(reinterpret_cast<const In*>(s_ptr[j])[i]));
        res[i] = acc;
    }
}

// ---------------------------------------------------------------------------------------------
// the apply kernel with bulk-copy staging: the default for up to 64 ranks on the 128-bit path
// ---------------------------------------------------------------------------------------------
// The same fold, but the tile of every new rank travels from global to shared memory as one bulk asynchronous
// copy (cp.async.bulk, completion counted in bytes on an mbarrier) through a ring of BK_STAGES buffers, issued by
// one thread; all threads then take their vectors from shared memory in ascending rank order.  No registers are
// tied up by loads in flight, so blocks are small and many: 64 threads, two stages of 4 KB (measured against
// 128/256 threads, 1-8 stages, 4-16 KB: this shape is best or within 0.5 % of the best on the config 2 and 3
// epochs, and beats the direct 128-bit loads of apply_kernel by 2.5 % on both; with one stage or with eight the
// direct loads win).  Every wait is bounded; a wait that gives up falls back to reading that rank's tile directly
// from global memory.
#ifndef EC_BK_THREADS
#define EC_BK_THREADS 64
#endif
#ifndef EC_BK_STAGES
#define EC_BK_STAGES 2
#endif
#ifndef EC_BK_STAGE_BYTES
#define EC_BK_STAGE_BYTES 4096
#endif
constexpr int BK_THREADS = EC_BK_THREADS;
constexpr int BK_STAGES = EC_BK_STAGES;
constexpr int BK_STAGE_BYTES = EC_BK_STAGE_BYTES;
constexpr int BK_VPT = BK_STAGE_BYTES / 16 / BK_THREADS;     // 16-byte input vectors per thread and tile
constexpr uint32_t BK_WAIT_LIMIT = 1u << 22;

__device__ __forceinline__ uint32_t bk_smem(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool bk_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t it = 0; it < BK_WAIT_LIMIT; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n"
            : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
    }
    return false;
}
__device__ __forceinline__ void bk_copy(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t pol) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(pol) : "memory");
}

template <int DT, int OP, bool LATE>
__global__ void __launch_bounds__(BK_THREADS)
apply_bulk_kernel(const ApplyArgs a, const __grid_constant__ PtrTable<64> tbl) {
    grid_dependency_wait();            // (a no-op unless launched as a programmatic dependent)
    typedef Elem<DT> E;
    typedef typename E::In In;
    typedef typename E::Acc Acc;
    constexpr int VEC = E::VEC;

    extern __shared__ __align__(128) unsigned char bk_stage[];          // BK_STAGES x BK_STAGE_BYTES
    __shared__ const char* s_ptr[64];
    __shared__ uint16_t s_rank[64];
    __shared__ uint64_t s_new[MAX_W];
    __shared__ int s_m, s_fresh, s_gave_up;
    __shared__ __align__(8) uint64_t s_bar[BK_STAGES];

    const unsigned s = blockIdx.x / a.tiles_per_seg;
    const unsigned t = blockIdx.x - s * a.tiles_per_seg;
    const size_t lo = (size_t)s * a.seg + (size_t)t * a.tile;
    size_t seg_hi = (size_t)(s + 1) * a.seg;
    if (seg_hi > a.n) seg_hi = a.n;
    const int tid = threadIdx.x;
    if (tid == 0) {
        s_gave_up = 0;
#pragma unroll
        for (int q = 0; q < BK_STAGES; ++q)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bk_smem(&s_bar[q])) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // Later applies of an epoch bring few ranks per segment and their blocks are short-lived: there the first warp
    // also notes the address of every new rank's tile while it builds the list, which saves a pass and a barrier
    // (config 3's late rounds: 5980 / 6050 -> 6630 / 6780 GB/s).  First applies, with many ranks per segment, run
    // 1.5 % faster when all threads fill in the addresses after the barrier (measured both ways on configs 2 and 3),
    // so the host picks the instantiation: LATE = not the first apply of the epoch.
    if (tid < 32) {
        if constexpr (LATE) block_prologue(a, s, t, s_rank, s_new, &s_m, &s_fresh, tbl.p, lo * sizeof(In), s_ptr);
        else block_prologue(a, s, t, s_rank, s_new, &s_m, &s_fresh);
    }
    __syncthreads();
    const int m = s_m;
    const bool fresh = s_fresh != 0;
    if (m == 0 && !(fresh && a.first_apply)) return;
    if (lo >= seg_hi) return;
    size_t hi = lo + a.tile;
    if (hi > seg_hi) hi = seg_hi;
    const size_t cnt = hi - lo;
    const int nvec = (int)(cnt / VEC);                                   // at most BK_STAGE_BYTES / 16
    const uint32_t bytes = (uint32_t)nvec * 16u;
    Acc* res = reinterpret_cast<Acc*>(a.result) + lo;
    const uint64_t pol = evict_first_policy();
    const uint64_t rpol_ld = result_policy(1), rpol_st = result_policy(a.res_hint == 2 ? 2 : 1);
    if constexpr (!LATE) {
        for (int j = tid; j < m; j += BK_THREADS)
            s_ptr[j] = reinterpret_cast<const char*>(tbl.p[s_rank[j]]) + lo * sizeof(In);
        __syncthreads();
    }
    if (tid == 0 && bytes != 0) {
        for (int j = 0; j < m && j < BK_STAGES; ++j)
            bk_copy(bk_smem(bk_stage + (size_t)j * BK_STAGE_BYTES), s_ptr[j], bytes, bk_smem(&s_bar[j]), pol);
    }
    Acc acc[BK_VPT][VEC];
#pragma unroll
    for (int p = 0; p < BK_VPT; ++p) {
        const int v = p * BK_THREADS + tid;
        if (fresh || v >= nvec) {
#pragma unroll
            for (int e = 0; e < VEC; ++e) acc[p][e] = ident<OP>(Acc());
        } else {
            load_acc<Acc, VEC>(res + (size_t)v * VEC, acc[p], rpol_ld);
        }
    }
    // A wait that runs out (never expected) ends the staging for the whole block: the thread that saw it reads its
    // vectors of that rank directly and raises s_gave_up; after the barrier that closes the rank every thread sees
    // the flag, no further copy is issued and the remaining ranks are read directly.  So no barrier is ever armed a
    // second time inside a phase that did not complete, and a late copy can only land in a stage nobody reads again.
    bool direct = false;
    int issued = m < BK_STAGES ? m : BK_STAGES;                           // copies issued so far (thread 0's count)
    if (bytes != 0) {
        for (int j = 0; j < m; ++j) {
            const int st = j % BK_STAGES;
            bool arrived = false;
            if (!direct) {
                arrived = bk_wait(bk_smem(&s_bar[st]), (uint32_t)(j / BK_STAGES) & 1u);
                if (!arrived) *reinterpret_cast<volatile int*>(&s_gave_up) = 1;
            }
            const unsigned char* src = bk_stage + (size_t)st * BK_STAGE_BYTES;
#pragma unroll
            for (int p = 0; p < BK_VPT; ++p) {
                const int v = p * BK_THREADS + tid;
                if (v < nvec) {
                    const uint4 raw = arrived ? *reinterpret_cast<const uint4*>(src + (size_t)v * 16)
                                              : ld_stream16(s_ptr[j] + (size_t)v * 16, pol);     // no copy to read from: read directly
                    Acc x[VEC];
                    E::unpack(raw, x);
#pragma unroll
                    for (int e = 0; e < VEC; ++e) acc[p][e] = comb<OP>(acc[p][e], x[e]);
                }
            }
            __syncthreads();                                             // everybody is done with this stage
            if (!direct && *reinterpret_cast<volatile int*>(&s_gave_up) != 0) direct = true;
            if (tid == 0 && !direct && j + BK_STAGES < m) {
                bk_copy(bk_smem(bk_stage + (size_t)st * BK_STAGE_BYTES), s_ptr[j + BK_STAGES], bytes, bk_smem(&s_bar[st]), pol);
                ++issued;
            }
        }
#pragma unroll
        for (int p = 0; p < BK_VPT; ++p) {
            const int v = p * BK_THREADS + tid;
            if (v < nvec) store_acc<Acc, VEC>(res + (size_t)v * VEC, acc[p], rpol_st);
        }
    }
    // elements after the last whole vector of a ragged tile
    for (size_t i = (size_t)nvec * VEC + tid; i < cnt; i += BK_THREADS) {
        Acc x = fresh ? ident<OP>(Acc()) : res[i];
        for (int j = 0; j < m; ++j) x = comb<OP>(x, E::widen(reinterpret_cast<const In*>(s_ptr[j])[i]));
        res[i] = x;
    }
    // Copies that were given up on, or issued ahead and never read, may still be on their way into this block's
    // shared memory: thread 0 gives the last copy of every stage one more bounded wait before the block retires.
    if (direct && tid == 0 && bytes != 0) {
        for (int st = 0; st < BK_STAGES && st < issued; ++st) {
            const int last_j = st + ((issued - 1 - st) / BK_STAGES) * BK_STAGES;
            bk_wait(bk_smem(&s_bar[st]), (uint32_t)(last_j / BK_STAGES) & 1u);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// the pairwise tree with bulk-copy staging: up to 64 ranks on the 128-bit path
// ---------------------------------------------------------------------------------------------
// The same balanced tree over the rank index as apply_kernel's pairwise branch (leaves eight ranks at a time, the
// subtrees merged by a binary counter: the additions of the recursive halving tree, bit for bit), but no load is held in
// a register.  A stage of shared memory takes the tiles (2 KB each) of the new ranks of one leaf block of eight, fetched
// by bulk asynchronous copies that report to the stage's mbarrier; the next leaf block's stage is under way while the
// threads reduce the one at hand out of shared memory and push it onto their binary counter.  Every wait is bounded;
// once one gives up the block stops staging and reads the remaining leaf blocks directly.  Shape by measurement on
// 32 bf16 ranks x 2^25 and 16 fp32 ranks x 2^24, all at once (threads / tile bytes / stages -> GB/s): 128/2048/2 6033
// and 6642; 64/1024/2 5702, 6733; 128/2048/3 5322, 5253; 256/4096/3 5203, 5115; 256/4096/2 5112, 6530; one stage 4133,
// 4682; all tiles of a block behind one barrier (no pipeline) 3290, 3915; the direct-load tree 4640, 6106.
#ifndef EC_PW_THREADS
#define EC_PW_THREADS 128
#endif
#ifndef EC_PW_TILE_BYTES
#define EC_PW_TILE_BYTES 2048
#endif
#ifndef EC_PW_STAGES
#define EC_PW_STAGES 2
#endif
constexpr int PW_THREADS = EC_PW_THREADS;
constexpr int PW_TILE_BYTES = EC_PW_TILE_BYTES;
constexpr int PW_STAGES = EC_PW_STAGES;
constexpr int PW_SMEM = PW_STAGES * 8 * PW_TILE_BYTES;

// One tree, rank by rank from global memory: fetch(r, out) delivers the PVU values of new rank r.
template <class Acc, int PVU, class Fetch>
__device__ __forceinline__ void pw_tree(uint64_t word, int P, Fetch fetch, Acc (&node)[PVU]) {
    int P2 = 1;
    while (P2 < P) P2 <<= 1;
    const int leaf = P2 < 8 ? P2 : 8;
    const int nblk = P2 / leaf;
    int nlev = 0;
    while ((1 << nlev) < nblk) ++nlev;
    Acc stack[3][PVU];
    for (int blk = 0; blk < nblk; ++blk) {
        const int r0 = blk * leaf;
        const unsigned byte = (unsigned)(word >> r0) & ((1u << leaf) - 1u);
        Acc lv[8][PVU];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
#pragma unroll
            for (int e = 0; e < PVU; ++e) lv[u][e] = ident<EC_SUM>(Acc());
            if ((byte >> u) & 1u) fetch(r0 + u, lv[u]);
        }
#pragma unroll
        for (int e = 0; e < PVU; ++e) {
            if (leaf == 8)
                node[e] = comb<EC_SUM>(comb<EC_SUM>(comb<EC_SUM>(lv[0][e], lv[1][e]), comb<EC_SUM>(lv[2][e], lv[3][e])),
                                       comb<EC_SUM>(comb<EC_SUM>(lv[4][e], lv[5][e]), comb<EC_SUM>(lv[6][e], lv[7][e])));
            else if (leaf == 4)
                node[e] = comb<EC_SUM>(comb<EC_SUM>(lv[0][e], lv[1][e]), comb<EC_SUM>(lv[2][e], lv[3][e]));
            else if (leaf == 2)
                node[e] = comb<EC_SUM>(lv[0][e], lv[1][e]);
            else
                node[e] = lv[0][e];
        }
        bool carry = true;
#pragma unroll
        for (int l = 0; l < 3; ++l) {
            if (l < nlev && carry) {
                if ((blk >> l) & 1) {
#pragma unroll
                    for (int e = 0; e < PVU; ++e) node[e] = comb<EC_SUM>(stack[l][e], node[e]);
                } else {
#pragma unroll
                    for (int e = 0; e < PVU; ++e) stack[l][e] = node[e];
                    carry = false;
                }
            }
        }
    }
}

template <int DT>
__global__ void __launch_bounds__(PW_THREADS)
apply_pw_bulk_kernel(const ApplyArgs a, const __grid_constant__ PtrTable<64> tbl) {
    grid_dependency_wait();            // (a no-op unless launched as a programmatic dependent)
    typedef Elem<DT> E;
    typedef typename E::In In;
    typedef typename E::Acc Acc;
    constexpr int PV = E::VEC > 4 ? 4 : E::VEC;                        // elements per tree walk (at most four accumulators per node)
    constexpr int UNIT_BYTES = PV * (int)sizeof(In);
    constexpr int UPT = PW_TILE_BYTES / UNIT_BYTES / PW_THREADS;       // units per thread: 1 (fp32, fp64) or 2 (bf16)
    static_assert(UPT >= 1 && UPT * UNIT_BYTES * PW_THREADS == PW_TILE_BYTES, "a tile is a whole number of units per thread");

    extern __shared__ __align__(128) unsigned char pw_stage[];         // [PW_STAGES][8 ranks][PW_TILE_BYTES]
    __shared__ uint16_t s_rank[64];
    __shared__ uint64_t s_new[MAX_W];
    __shared__ int s_m, s_fresh, s_gave_up;
    __shared__ __align__(8) uint64_t s_bar[PW_STAGES];

    const unsigned s = blockIdx.x / a.tiles_per_seg;
    const unsigned t = blockIdx.x - s * a.tiles_per_seg;
    const size_t lo = (size_t)s * a.seg + (size_t)t * a.tile;
    size_t seg_hi = (size_t)(s + 1) * a.seg;
    if (seg_hi > a.n) seg_hi = a.n;
    const int tid = threadIdx.x;
    if (tid == 0) {
        s_gave_up = 0;
#pragma unroll
        for (int q = 0; q < PW_STAGES; ++q)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bk_smem(&s_bar[q])) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < 32) block_prologue(a, s, t, s_rank, s_new, &s_m, &s_fresh);
    __syncthreads();
    const int m = s_m;
    const bool fresh = s_fresh != 0;
    if (m == 0 && !(fresh && a.first_apply)) return;
    if (lo >= seg_hi) return;
    size_t hi = lo + a.tile;
    if (hi > seg_hi) hi = seg_hi;
    const size_t cnt = hi - lo;
    const uint32_t bytes = (uint32_t)(cnt * sizeof(In) / 16) * 16u;    // staged part of a rank's tile: whole 16-byte vectors
    const int nunits = (int)(bytes / UNIT_BYTES);
    Acc* res = reinterpret_cast<Acc*>(a.result) + lo;
    const uint64_t pol = evict_first_policy();
    const uint64_t rpol_ld = result_policy(1), rpol_st = result_policy(a.res_hint == 2 ? 2 : 1);
    const uint64_t word = s_new[0];
    int P2 = 1;
    while (P2 < a.P) P2 <<= 1;
    const int leaf = P2 < 8 ? P2 : 8;
    const int nblk = P2 / leaf;
    int nlev = 0;
    while ((1 << nlev) < nblk) ++nlev;

    // thread 0 issues, for leaf block b, one copy per new rank of the block into stage b % PW_STAGES, side by side
    auto issue = [&](int b) {
        const int r0 = b * leaf;
        const unsigned byte = (unsigned)(word >> r0) & ((1u << leaf) - 1u);
        if (byte == 0u || bytes == 0u) return;
        const uint32_t bar = bk_smem(&s_bar[b % PW_STAGES]);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes * (uint32_t)__popc(byte)) : "memory");
        unsigned char* dst = pw_stage + (size_t)(b % PW_STAGES) * 8 * PW_TILE_BYTES;
        for (unsigned rest = byte; rest != 0u; rest &= rest - 1u) {
            const int u = __ffs((int)rest) - 1;
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                         ::"r"(bk_smem(dst)), "l"(reinterpret_cast<const char*>(tbl.p[r0 + u]) + lo * sizeof(In)), "r"(bytes), "r"(bar), "l"(pol)
                         : "memory");
            dst += PW_TILE_BYTES;
        }
    };
    if (tid == 0)
        for (int b = 0; b < nblk && b < PW_STAGES; ++b) issue(b);

    Acc node[UPT][PV], stack[UPT][3][PV];
    bool direct = false;
    uint32_t waits[PW_STAGES];                                          // completed phases of every stage's barrier so far
#pragma unroll
    for (int q = 0; q < PW_STAGES; ++q) waits[q] = 0u;
    for (int blk = 0; blk < nblk; ++blk) {
        const int r0 = blk * leaf, st = blk % PW_STAGES;
        const unsigned byte = (unsigned)(word >> r0) & ((1u << leaf) - 1u);
        bool staged = false;
        if (byte != 0u && bytes != 0u && !direct) {
            uint32_t par = 0u;
#pragma unroll
            for (int q = 0; q < PW_STAGES; ++q)
                if (q == st) { par = waits[q] & 1u; ++waits[q]; }
            staged = bk_wait(bk_smem(&s_bar[st]), par);
            if (!staged) *reinterpret_cast<volatile int*>(&s_gave_up) = 1;
        }
        const unsigned char* sbase = pw_stage + (size_t)st * 8 * PW_TILE_BYTES;
#pragma unroll
        for (int q = 0; q < UPT; ++q) {
            const int w = q * PW_THREADS + tid;
            Acc lv[8][PV];
            if (w < nunits) {
                auto from_stage = [&](int slot, Acc (&out)[PV]) {
                    const unsigned char* src = sbase + (size_t)slot * PW_TILE_BYTES + (size_t)w * UNIT_BYTES;
                    if constexpr (DT == EC_BF16) {
                        const uint2 r = *reinterpret_cast<const uint2*>(src);
                        out[0] = __uint_as_float(r.x << 16); out[1] = __uint_as_float(r.x & 0xFFFF0000u);
                        out[2] = __uint_as_float(r.y << 16); out[3] = __uint_as_float(r.y & 0xFFFF0000u);
                    } else {
                        E::unpack(*reinterpret_cast<const uint4*>(src), out);
                    }
                };
                auto from_global = [&](int r, Acc (&out)[PV]) {
                    const char* src = reinterpret_cast<const char*>(tbl.p[r]) + lo * sizeof(In) + (size_t)w * UNIT_BYTES;
                    if constexpr (DT == EC_BF16) {
                        const uint2 v = ld_stream8(src, pol);
                        out[0] = __uint_as_float(v.x << 16); out[1] = __uint_as_float(v.x & 0xFFFF0000u);
                        out[2] = __uint_as_float(v.y << 16); out[3] = __uint_as_float(v.y & 0xFFFF0000u);
                    } else {
                        E::unpack(ld_stream16(src, pol), out);
                    }
                };
                if (staged && leaf == 8 && byte == 0xFFu) {             // all eight ranks new: the usual case in a first apply
#pragma unroll
                    for (int u = 0; u < 8; ++u) from_stage(u, lv[u]);
                } else {
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
#pragma unroll
                        for (int e = 0; e < PV; ++e) lv[u][e] = ident<EC_SUM>(Acc());
                        if ((byte >> u) & 1u) {
                            if (staged) from_stage(__popc(byte & ((1u << u) - 1u)), lv[u]);
                            else from_global(r0 + u, lv[u]);
                        }
                    }
                }
#pragma unroll
                for (int e = 0; e < PV; ++e) {
                    if (leaf == 8)
                        node[q][e] = comb<EC_SUM>(comb<EC_SUM>(comb<EC_SUM>(lv[0][e], lv[1][e]), comb<EC_SUM>(lv[2][e], lv[3][e])),
                                                  comb<EC_SUM>(comb<EC_SUM>(lv[4][e], lv[5][e]), comb<EC_SUM>(lv[6][e], lv[7][e])));
                    else if (leaf == 4)
                        node[q][e] = comb<EC_SUM>(comb<EC_SUM>(lv[0][e], lv[1][e]), comb<EC_SUM>(lv[2][e], lv[3][e]));
                    else if (leaf == 2)
                        node[q][e] = comb<EC_SUM>(lv[0][e], lv[1][e]);
                    else
                        node[q][e] = lv[0][e];
                }
                bool carry = true;
#pragma unroll
                for (int l = 0; l < 3; ++l) {
                    if (l < nlev && carry) {
                        if ((blk >> l) & 1) {
#pragma unroll
                            for (int e = 0; e < PV; ++e) node[q][e] = comb<EC_SUM>(stack[q][l][e], node[q][e]);
                        } else {
#pragma unroll
                            for (int e = 0; e < PV; ++e) stack[q][l][e] = node[q][e];
                            carry = false;
                        }
                    }
                }
            }
        }
        if (blk + 1 < nblk) {
            __syncthreads();                                            // everybody is done with this stage
            if (!direct && *reinterpret_cast<volatile int*>(&s_gave_up) != 0) direct = true;
            if (tid == 0 && !direct && blk + PW_STAGES < nblk) issue(blk + PW_STAGES);
        }
    }
    // node is the root now
#pragma unroll
    for (int q = 0; q < UPT; ++q) {
        const int w = q * PW_THREADS + tid;
        if (w < nunits) {
            if (!fresh) {
                Acc acc[PV];
                load_acc<Acc, PV>(res + (size_t)w * PV, acc, rpol_ld);
#pragma unroll
                for (int e = 0; e < PV; ++e) node[q][e] = comb<EC_SUM>(acc[e], node[q][e]);
            }
            store_acc<Acc, PV>(res + (size_t)w * PV, node[q], rpol_st);
        }
    }
    // elements after the last whole vector of a ragged tile: the same tree, element by element, from the rank buffers
    for (size_t i = (size_t)nunits * PV + tid; i < cnt; i += PW_THREADS) {
        Acc root[1];
        pw_tree<Acc, 1>(word, a.P, [&](int r, Acc (&out)[1]) { out[0] = E::widen(reinterpret_cast<const In*>(tbl.p[r])[lo + i]); }, root);
        res[i] = fresh ? root[0] : comb<EC_SUM>(res[i], root[0]);
    }
    // copies that were given up on, or issued ahead and never read, may still be on their way into this block's
    // shared memory: thread 0 gives every stage's barrier one more bounded wait before the block retires
    if (tid == 0 && *reinterpret_cast<volatile int*>(&s_gave_up) != 0) {
#pragma unroll
        for (int q = 0; q < PW_STAGES; ++q) bk_wait(bk_smem(&s_bar[q]), waits[q] & 1u);
    }
}

template <int DT>
int launch_pw_bulk(const ApplyArgs& a, const void* const* bufs, unsigned grid, cudaStream_t st) {
    PtrTable<64> tbl;
    for (int r = 0; r < 64; ++r) tbl.p[r] = r < a.P ? bufs[r] : nullptr;
    if (a.dependent) EC_CUDA(launch_dependent(apply_pw_bulk_kernel<DT>, grid, PW_THREADS, PW_SMEM, st, a, tbl));
    else apply_pw_bulk_kernel<DT><<<grid, PW_THREADS, PW_SMEM, st>>>(a, tbl);
    EC_CUDA(cudaGetLastError());
    return EC_OK;
}

template <int DT, int OP, bool VECTOR, int ORDER>
int launch_cap(const ApplyArgs& a, const void* const* bufs, unsigned grid, int threads, bool short_seg, cudaStream_t st) {
    if (a.P <= 64) {
        PtrTable<64> tbl;
        for (int r = 0; r < 64; ++r) tbl.p[r] = r < a.P ? bufs[r] : nullptr;
        if constexpr (VECTOR && ORDER == EC_ORDER_FIXED) {
            if (short_seg) {
                if (a.dependent) EC_CUDA(launch_dependent(apply_short_kernel<DT, OP, 64>, grid, (unsigned)threads, 0, st, a, tbl));
                else apply_short_kernel<DT, OP, 64><<<grid, threads, 0, st>>>(a, tbl);
                EC_CUDA(cudaGetLastError());
                return EC_OK;
            }
        }
        if (a.dependent) EC_CUDA(launch_dependent(apply_kernel<DT, OP, VECTOR, 64, ORDER>, grid, (unsigned)threads, 0, st, a, tbl));
        else apply_kernel<DT, OP, VECTOR, 64, ORDER><<<grid, threads, 0, st>>>(a, tbl);
    } else {
        PtrTable<EC_MAX_RANKS> tbl;
        for (int r = 0; r < EC_MAX_RANKS; ++r) tbl.p[r] = r < a.P ? bufs[r] : nullptr;
        if (a.dependent) EC_CUDA(launch_dependent(apply_kernel<DT, OP, VECTOR, EC_MAX_RANKS, ORDER>, grid, (unsigned)threads, 0, st, a, tbl));
        else apply_kernel<DT, OP, VECTOR, EC_MAX_RANKS, ORDER><<<grid, threads, 0, st>>>(a, tbl);
    }
    EC_CUDA(cudaGetLastError());
    return EC_OK;
}

template <int DT, int OP>
int launch_op(const ApplyArgs& a, const void* const* bufs, bool vector, int order, unsigned grid, int threads,
              bool short_seg, cudaStream_t st) {
    if (order == EC_ORDER_FIXED || order == EC_ORDER_RING)     // ring order = rank order rotated per chunk (a.ring_chunk)
        return vector ? launch_cap<DT, OP, true, EC_ORDER_FIXED>(a, bufs, grid, threads, short_seg, st)
                      : launch_cap<DT, OP, false, EC_ORDER_FIXED>(a, bufs, grid, threads, false, st);
    if constexpr (OP == EC_SUM && DT != EC_I64)
        return vector ? launch_cap<DT, EC_SUM, true, EC_ORDER_PAIRWISE>(a, bufs, grid, threads, false, st)
                      : launch_cap<DT, EC_SUM, false, EC_ORDER_PAIRWISE>(a, bufs, grid, threads, false, st);
    return EC_ERR_UNSUPPORTED;
}

template <int DT>
int launch_dt(const ApplyArgs& a, const void* const* bufs, int op, bool vector, int order, unsigned grid,
              int threads, bool short_seg, cudaStream_t st) {
    switch (op) {
        case EC_SUM: return launch_op<DT, EC_SUM>(a, bufs, vector, order, grid, threads, short_seg, st);
        case EC_MAX: return launch_op<DT, EC_MAX>(a, bufs, vector, order, grid, threads, short_seg, st);
        case EC_MIN: return launch_op<DT, EC_MIN>(a, bufs, vector, order, grid, threads, short_seg, st);
    }
    return EC_ERR_INVALID;
}

template <int DT, int OP>
int launch_bulk_op(const ApplyArgs& a, const void* const* bufs, unsigned grid, cudaStream_t st) {
    PtrTable<64> tbl;
    for (int r = 0; r < 64; ++r) tbl.p[r] = r < a.P ? bufs[r] : nullptr;
    if (a.dependent) {
        if (a.first_apply) EC_CUDA(launch_dependent(apply_bulk_kernel<DT, OP, false>, grid, BK_THREADS, BK_STAGES * BK_STAGE_BYTES, st, a, tbl));
        else EC_CUDA(launch_dependent(apply_bulk_kernel<DT, OP, true>, grid, BK_THREADS, BK_STAGES * BK_STAGE_BYTES, st, a, tbl));
    } else if (a.first_apply) apply_bulk_kernel<DT, OP, false><<<grid, BK_THREADS, BK_STAGES * BK_STAGE_BYTES, st>>>(a, tbl);
    else apply_bulk_kernel<DT, OP, true><<<grid, BK_THREADS, BK_STAGES * BK_STAGE_BYTES, st>>>(a, tbl);
    EC_CUDA(cudaGetLastError());
    return EC_OK;
}
template <int DT>
int launch_bulk_dt(const ApplyArgs& a, const void* const* bufs, int op, unsigned grid, cudaStream_t st) {
    switch (op) {
        case EC_SUM: return launch_bulk_op<DT, EC_SUM>(a, bufs, grid, st);
        case EC_MAX: return launch_bulk_op<DT, EC_MAX>(a, bufs, grid, st);
        case EC_MIN: return launch_bulk_op<DT, EC_MIN>(a, bufs, grid, st);
    }
    return EC_ERR_INVALID;
}
int launch_bulk(const ApplyArgs& a, const void* const* bufs, int dtype, int op, unsigned grid, cudaStream_t st) {
    switch (dtype) {
        case EC_F32: return launch_bulk_dt<EC_F32>(a, bufs, op, grid, st);
        case EC_BF16: return launch_bulk_dt<EC_BF16>(a, bufs, op, grid, st);
        case EC_I64: return launch_bulk_dt<EC_I64>(a, bufs, op, grid, st);
        case EC_F64: return launch_bulk_dt<EC_F64>(a, bufs, op, grid, st);
    }
    return EC_ERR_INVALID;
}

size_t words_bytes(int P, size_t n, size_t seg) {
    const size_t S = (n + seg - 1) / seg;
    const size_t W = (size_t)(P + 63) / 64;
    return align_up(S * W * sizeof(uint64_t), 256);
}

bool bad_shape(int P, size_t n, size_t seg) {
    return P < 1 || P > EC_MAX_RANKS || n == 0 || seg == 0 || (n + seg - 1) / seg > 0x7fffffffull;
}

}  // namespace
}  // namespace ec

struct ec_ctx {
    int P, W, dtype, op, order;
    size_t n, seg, S;
    void* ws;
    bool own_ws;
    uint64_t* applied[2];
    int cur;           // which copy holds the current words
    bool first_apply;  // no apply yet in this epoch
    int threads;
    size_t tile;       // elements per block
    int res_hint;      // L2 policy of the result accesses
    int path;          // 1: bulk-copy staging where it applies (the default when the context allows it), 0: direct loads
    bool dependent;    // apply kernels are launched as programmatic dependents (set by the drivers, see ec_common.cuh)
};

void ec::allreduce_set_dependent_launch(ec_ctx* ctx, bool on) {
    if (ctx) ctx->dependent = on;
}

using namespace ec;

extern "C" {

size_t ec_allreduce_workspace_bytes(int P, size_t n, size_t segment_size) {
    if (bad_shape(P, n, segment_size)) return 0;
    return 2 * words_bytes(P, n, segment_size);
}

int ec_allreduce_init(ec_ctx_t** out, int P, size_t n, ec_dtype_t dtype, ec_op_t op, size_t segment_size,
                      ec_order_t order, void* workspace, size_t workspace_bytes) {
    if (!out) return EC_ERR_INVALID;
    *out = nullptr;
    if (bad_shape(P, n, segment_size)) return EC_ERR_INVALID;
    if ((int)dtype < 0 || (int)dtype > EC_F64 || (int)op < 0 || (int)op > EC_MIN) return EC_ERR_INVALID;
    if ((int)order != EC_ORDER_FIXED && (int)order != EC_ORDER_PAIRWISE && (int)order != EC_ORDER_RING) return EC_ERR_INVALID;
    // ring order: the vector is cut into P chunks of ceil(n/P) elements; a segment must lie inside one chunk
    if (order == EC_ORDER_RING && ((n + (size_t)P - 1) / (size_t)P) % segment_size != 0) return EC_ERR_INVALID;
    if (order == EC_ORDER_PAIRWISE && (op != EC_SUM || dtype == EC_I64)) return EC_ERR_UNSUPPORTED;
    const size_t need = ec_allreduce_workspace_bytes(P, n, segment_size);
    if (workspace && (workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255u))) return EC_ERR_CAPACITY;
    ec_ctx* c = new (std::nothrow) ec_ctx();
    if (!c) return EC_ERR_INVALID;
    c->P = P; c->W = (P + 63) / 64; c->dtype = dtype; c->op = op; c->order = order;
    c->n = n; c->seg = segment_size; c->S = (n + segment_size - 1) / segment_size;
    c->own_ws = workspace == nullptr;
    c->ws = workspace;
    if (c->own_ws) {
        cudaError_t e = cudaMalloc(&c->ws, need);
        if (e != cudaSuccess) { delete c; return cuda_fail(e); }
    }
    cudaError_t e = cudaMemsetAsync(c->ws, 0, need, 0);
    if (e == cudaSuccess) e = cudaStreamSynchronize(0);
    if (e != cudaSuccess) {
        if (c->own_ws) cudaFree(c->ws);
        delete c;
        return cuda_fail(e);
    }
    c->applied[0] = reinterpret_cast<uint64_t*>(c->ws);
    c->applied[1] = reinterpret_cast<uint64_t*>(reinterpret_cast<char*>(c->ws) + need / 2);
    c->cur = 0;
    c->first_apply = true;
    c->dependent = true;    // (see ec_common.cuh: the apply kernels wait on the device for whatever precedes them in the stream)
    {
        int dev = 0, l2 = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, dev) != cudaSuccess)
            l2 = 0;
        c->res_hint = (double)n * (double)out_bytes(dtype) <= 0.75 * (double)l2 ? 1 : 2;   // does the result fit in L2?
    }
    // Few ranks: many small blocks overlap their start-up latency best.  Hundreds of ranks: a block
    // lives long anyway and wider blocks read longer contiguous runs of each buffer (both measured).
    c->path = P <= 64 ? 1 : 0;
    if (order == EC_ORDER_PAIRWISE && P <= 64 && PW_SMEM > 48 * 1024) {   // the limit of dynamic shared memory has to be raised
        cudaError_t e2 = cudaFuncSetAttribute(apply_pw_bulk_kernel<EC_F32>, cudaFuncAttributeMaxDynamicSharedMemorySize, PW_SMEM);
        if (e2 == cudaSuccess) e2 = cudaFuncSetAttribute(apply_pw_bulk_kernel<EC_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, PW_SMEM);
        if (e2 == cudaSuccess) e2 = cudaFuncSetAttribute(apply_pw_bulk_kernel<EC_F64>, cudaFuncAttributeMaxDynamicSharedMemorySize, PW_SMEM);
        if (e2 != cudaSuccess) { cudaGetLastError(); c->path = 0; }
    }
    c->threads = P > 64 ? 256 : 128;
    c->tile = dtype == EC_BF16 ? 2048 : 8192 / in_bytes(dtype);   // 8 KB of every rank buffer per block (4 KB for bf16), measured
    *out = c;
    return EC_OK;
}

int ec_allreduce_set_path(ec_ctx_t* c, int path) {
    if (!c || (path != 0 && path != 1)) return EC_ERR_INVALID;
    if (path == 1 && c->P > 64) return EC_ERR_UNSUPPORTED;
    c->path = path;
    return EC_OK;
}

int ec_allreduce_set_tile(ec_ctx_t* c, int threads, size_t tile_elems) {
    if (!c) return EC_ERR_INVALID;
    if (threads != 0) {
        if (threads < 64 || threads > EC_MAXT || threads % 32) return EC_ERR_INVALID;
        c->threads = threads;
    }
    if (tile_elems != 0) {
        const size_t vec = 16 / in_bytes(c->dtype);
        c->tile = align_up(tile_elems, vec);
    }
    return EC_OK;
}

namespace {
// Validation, tiling and launch shared by the notification-bit apply and the stale-synchronous apply.
int apply_common(ec_ctx_t* c, const void* const* rank_bufs, int P, size_t n, ec_dtype_t dtype, ec_op_t op,
                 size_t segment_size, void* result, ApplyArgs& a, ec_stream_t stream) {
    if (!c || !rank_bufs || !result) return EC_ERR_INVALID;
    if (P != c->P || n != c->n || (int)dtype != c->dtype || (int)op != c->op || segment_size != c->seg)
        return EC_ERR_INVALID;
    bool vector = aligned16(result) && (c->seg * in_bytes(c->dtype)) % 16 == 0;
    for (int r = 0; r < P; ++r) {
        if (!rank_bufs[r] || rank_bufs[r] == result) return EC_ERR_INVALID;
        vector = vector && aligned16(rank_bufs[r]);
    }
    const size_t seg_len = c->seg < c->n ? c->seg : c->n;
    const size_t tiles = (seg_len + c->tile - 1) / c->tile;
    if (tiles * c->S > 0x7fffffffull) return EC_ERR_CAPACITY;
    a.n = c->n; a.seg = c->seg; a.tile = c->tile;
    a.result = result;
    a.tiles_per_seg = (unsigned)tiles;
    a.P = c->P; a.W = c->W;
    a.res_hint = c->res_hint;
    a.dependent = c->dependent ? 1 : 0;
    a.ring_chunk = c->order == EC_ORDER_RING ? (c->n + (size_t)c->P - 1) / (size_t)c->P : 0;
    unsigned grid = (unsigned)(tiles * c->S);
    // short segments and more ranks than the streaming fold keeps in flight: one block per segment, staged fold
    // (measured: 12.4 -> 10.3 us for 64 ranks x 64 rows of 36 floats, 36.8 -> 30.7 us for 4096 such rows; with
    // hundreds of ranks the staging passes cost more than they save, so those stay on the streaming kernel)
    const bool short_seg = vector && c->order != EC_ORDER_PAIRWISE && c->P > EC_MAIN_RU && c->P <= 64 &&
                           (seg_len * in_bytes(c->dtype) / 16) * 4 <= (size_t)c->threads;
    if (short_seg) {
        a.tiles_per_seg = 1;
        grid = (unsigned)c->S;
    }
    if (c->path == 1 && vector && !short_seg && c->order != EC_ORDER_PAIRWISE && c->P <= 64) {
        // bulk-copy staging: tiles of one stage buffer (8 KB of every rank)
        a.tile = BK_STAGE_BYTES / in_bytes(c->dtype);
        const size_t btiles = (seg_len + a.tile - 1) / a.tile;
        if (btiles * c->S > 0x7fffffffull) return EC_ERR_CAPACITY;
        a.tiles_per_seg = (unsigned)btiles;
        return launch_bulk(a, rank_bufs, c->dtype, c->op, (unsigned)(btiles * c->S), stream);
    }
    if (c->path == 1 && vector && c->order == EC_ORDER_PAIRWISE && c->P <= 64 && a.notif_clock == nullptr) {
        // the pairwise tree out of bulk-staged tiles: 2 KB of every rank per block
        a.tile = PW_TILE_BYTES / in_bytes(c->dtype);
        const size_t ptiles = (seg_len + a.tile - 1) / a.tile;
        if (ptiles * c->S > 0x7fffffffull) return EC_ERR_CAPACITY;
        a.tiles_per_seg = (unsigned)ptiles;
        const unsigned pgrid = (unsigned)(ptiles * c->S);
        switch (c->dtype) {
            case EC_F32: return launch_pw_bulk<EC_F32>(a, rank_bufs, pgrid, stream);
            case EC_BF16: return launch_pw_bulk<EC_BF16>(a, rank_bufs, pgrid, stream);
            case EC_F64: return launch_pw_bulk<EC_F64>(a, rank_bufs, pgrid, stream);
        }
    }
    switch (c->dtype) {
        case EC_F32: return launch_dt<EC_F32>(a, rank_bufs, c->op, vector, c->order, grid, c->threads, short_seg, stream);
        case EC_BF16: return launch_dt<EC_BF16>(a, rank_bufs, c->op, vector, c->order, grid, c->threads, short_seg, stream);
        case EC_I64: return launch_dt<EC_I64>(a, rank_bufs, c->op, vector, c->order, grid, c->threads, short_seg, stream);
        case EC_F64: return launch_dt<EC_F64>(a, rank_bufs, c->op, vector, c->order, grid, c->threads, short_seg, stream);
    }
    return EC_ERR_INVALID;
}
}  // namespace

int ec_allreduce_apply(ec_ctx_t* c, const void* const* rank_bufs, int P, size_t n, ec_dtype_t dtype, ec_op_t op,
                       size_t segment_size, const uint64_t* arrival_mask, void* result, uint32_t* contrib_count,
                       ec_stream_t stream) {
    if (!c) return EC_ERR_INVALID;
    ApplyArgs a = {};
    a.arrival = arrival_mask;
    a.applied_in = c->applied[c->cur];
    a.applied_out = c->applied[c->cur ^ 1];
    a.contrib_count = contrib_count;
    a.first_apply = c->first_apply ? 1 : 0;
    const int rc = apply_common(c, rank_bufs, P, n, dtype, op, segment_size, result, a, stream);
    if (rc != EC_OK) return rc;
    c->cur ^= 1;
    c->first_apply = false;
    return EC_OK;
}

int ec_allreduce_ssp_apply(ec_ctx_t* c, const void* const* rank_bufs, int P, size_t n, ec_dtype_t dtype, ec_op_t op,
                           size_t segment_size, const uint32_t* notif_clock, uint32_t clock, uint32_t slack,
                           void* result, uint32_t* contrib_count, uint32_t* seg_clock, uint32_t* wait_count,
                           ec_stream_t stream) {
    if (!c || !notif_clock || clock == 0) return EC_ERR_INVALID;
    ApplyArgs a = {};
    a.applied_in = c->applied[c->cur];        // not used: this call keeps no state
    a.applied_out = c->applied[c->cur ^ 1];
    a.contrib_count = contrib_count;
    a.first_apply = 1;                        // every segment is rebuilt from the identity
    a.notif_clock = notif_clock;
    a.min_clock = clock > slack ? clock - slack : 1u;   // clocks start at 1; 0 means "nothing received yet"
    a.seg_clock = seg_clock;
    a.wait_count = wait_count;
    return apply_common(c, rank_bufs, P, n, dtype, op, segment_size, result, a, stream);
}

int ec_allreduce_reset(ec_ctx_t* c, ec_stream_t stream) {
    if (!c) return EC_ERR_INVALID;
    (void)stream;               // nothing to enqueue: the next apply ignores the stored words
    c->first_apply = true;
    return EC_OK;
}

size_t ec_allreduce_host_staging_bytes(const ec_ctx_t* c, int rounds) {
    if (!c || rounds < 1) return 0;
    const size_t buf = align_up(c->n * in_bytes(c->dtype), 256);
    const size_t words = align_up(c->S * (size_t)c->W * sizeof(uint64_t), 256);
    return (size_t)c->P * buf + (size_t)rounds * words + align_up(c->n * out_bytes(c->dtype), 256) +
           align_up(c->S * sizeof(uint32_t), 256);
}

int ec_allreduce_epoch_host(ec_ctx_t* c, const void* const* host_rank_bufs, const uint64_t* const* host_masks,
                            int rounds, void* host_result, uint32_t* host_contrib_count, void* staging,
                            size_t staging_bytes, ec_stream_t stream) {
    if (!c || !host_rank_bufs || !host_masks || !host_result || !staging || rounds < 1) return EC_ERR_INVALID;
    if (staging_bytes < ec_allreduce_host_staging_bytes(c, rounds) || (reinterpret_cast<uintptr_t>(staging) & 255u))
        return EC_ERR_CAPACITY;
    for (int r = 0; r < c->P; ++r)
        if (!host_rank_bufs[r]) return EC_ERR_INVALID;
    for (int k = 0; k < rounds; ++k)
        if (!host_masks[k]) return EC_ERR_INVALID;
    const size_t in_b = c->n * in_bytes(c->dtype), out_b = c->n * out_bytes(c->dtype);
    const size_t buf = align_up(in_b, 256);
    const size_t words_b = c->S * (size_t)c->W * sizeof(uint64_t), words = align_up(words_b, 256);
    char* p = static_cast<char*>(staging);
    const void* dev_bufs[EC_MAX_RANKS];
    for (int r = 0; r < c->P; ++r) {       // one plain copy per rank buffer; they queue behind one another on the stream
        dev_bufs[r] = p;
        EC_CUDA(cudaMemcpyAsync(p, host_rank_bufs[r], in_b, cudaMemcpyHostToDevice, stream));
        p += buf;
    }
    const uint64_t* dev_masks = reinterpret_cast<const uint64_t*>(p);
    for (int k = 0; k < rounds; ++k) {
        EC_CUDA(cudaMemcpyAsync(p, host_masks[k], words_b, cudaMemcpyHostToDevice, stream));
        p += words;
    }
    void* dev_result = p;
    p += align_up(out_b, 256);
    uint32_t* dev_count = reinterpret_cast<uint32_t*>(p);
    int rc = ec_allreduce_reset(c, stream);
    for (int k = 0; k < rounds && rc == EC_OK; ++k)
        rc = ec_allreduce_apply(c, dev_bufs, c->P, c->n, (ec_dtype_t)c->dtype, (ec_op_t)c->op, c->seg,
                                dev_masks + (size_t)k * (words / sizeof(uint64_t)), dev_result, dev_count, stream);
    if (rc != EC_OK) return rc;
    EC_CUDA(cudaMemcpyAsync(host_result, dev_result, out_b, cudaMemcpyDeviceToHost, stream));
    if (host_contrib_count)
        EC_CUDA(cudaMemcpyAsync(host_contrib_count, dev_count, c->S * sizeof(uint32_t), cudaMemcpyDeviceToHost, stream));
    return EC_OK;
}

int ec_allreduce_destroy(ec_ctx_t* c) {
    if (!c) return EC_ERR_INVALID;
    int rc = EC_OK;
    if (c->own_ws && c->ws) {
        cudaError_t e = cudaFree(c->ws);
        if (e != cudaSuccess) rc = cuda_fail(e);
    }
    delete c;
    return rc;
}

const char* ec_strerror(int code) {
    switch (code) {
        case EC_OK: return "ok";
        case EC_ERR_INVALID: return "invalid argument";
        case EC_ERR_UNSUPPORTED: return "unsupported combination of dtype, op and order";
        case EC_ERR_CUDA: return "CUDA runtime error (see ec_last_cuda_error)";
        case EC_ERR_STATE: return "call not allowed in this state";
        case EC_ERR_CAPACITY: return "size beyond a limit, or workspace too small";
    }
    return "unknown error code";
}

int ec_last_cuda_error(void) { return g_last_cuda_error; }
int ec_version(void) { return 1000; }

}  // extern "C"
