// K-means assignment + partial sums on the 5th-generation tensor cores (tcgen05, tensor memory).
//
// Candidate search.  The squared distance to centroid k is |x|^2 + v_k with v_k = |c_k|^2 - 2 x.c_k.
// The inner products of a tile of 128 points with all centroids are one small GEMM: points and
// centroids are rounded to bf16, staged in shared memory in the tensor core's canonical layout,
// multiplied by tcgen05.mma into an fp32 accumulator in tensor memory and read back with tcgen05.ld,
// one point per thread.  bf16 makes v_k approximate, so it only proposes: the smallest and second
// smallest v are tracked and whenever they are closer than a bound on the error of v (tau) the point
// is decided again in fp32 by the exact form sum_d (x-c)^2 over all centroids.  Labels are therefore
// those of the exact form; only speed depends on how well separated the data is.
//
// Partial sums.  sums[d][k] = sum_j x[j][d] onehot[j][k] is a GEMM too: the points, split into bf16
// high and low parts (16 significand bits, relative error 2^-17 per coordinate, far inside the 1e-4
// tolerance of the sums) and extended by a constant column of ones that yields the exact counts,
// times the one-hot label matrix of the tile (exact in bf16).  The accumulator (row = coordinate,
// column = centroid) stays in tensor memory over all tiles of the block and is written out once.
// The shared-memory tile of the high parts serves both GEMMs: as the K-major A operand of the
// search (row = point) and as the MN-major A operand here (row = coordinate) - both see the same
// 8-point x 8-coordinate core matrices.  The sums MMA always works on 128 rows; rows beyond the
// D + 16 real ones read whatever follows the tile in shared memory and are never looked at.
//
// Delta mode (iterations after the first): the labels of the previous iteration are read back, a point that
// keeps its label contributes nothing, one that moves puts +1 in the one-hot column of its new cluster and
// -1 in that of its old one, so the accumulator collects the change of the sums; a tile without a move
// issues no sums MMA at all (and the low parts, needed only by that MMA, are staged on demand from L2), a
// block without one leaves its row block unwritten and says so in a flag.  Once the clustering has settled
// an iteration is the search alone.
//
// Distance bounds (delta mode): every point also carries an upper bound on the distance to its own centroid and
// a lower bound on the distance to any other, every centroid the sum of its moves; bounds_check_kernel marks the
// tiles in which a label can still change and only those are searched (details at the tile loop).
//
// Run (r, c) is the c-th of C parts of rank r's points and yields one [K][D+4] row block of scratch; the rows of
// a rank are folded in order afterwards.  The grid is one wave of resident blocks; block b takes the runs b,
// b + gridDim.x, ..., so the set-up (centroid operand, tensor memory) is paid once per block.  Every wait on
// the tensor core is bounded; if one gives up, the block finishes in plain fp32 (exact form, atomic adds into
// its row block) and a status word records it.
#pragma once

#include <cuda_bf16.h>

namespace ec {
namespace tc {

#ifndef EC_TC_MINB
#define EC_TC_MINB 4                   // resident blocks the register allocation must allow
#endif
constexpr int THREADS = 128;           // four warps: one tensor-memory lane (= one point, one centroid row) per thread
constexpr int TILE = THREADS;          // points per tile
constexpr int MROWS = 128;             // rows of both accumulators
constexpr uint32_t WAIT_LIMIT = 1u << 20;
constexpr uint32_t OCHUNK = TILE * 16;        // one-hot tile: bytes between chunks of 8 centroids (128 points x 16 bytes)
// Point tiles: bytes between chunks of 8 coordinates.  Eight consecutive threads store one quarter-warp's 16-byte
// items: D/8 chunks of 8/(D/8) consecutive points.  The padding of 1024/D bytes puts them on all 32 banks
// (D = 32: chunks 32 bytes apart modulo 128, points 16 bytes apart; D = 16: chunks 64 bytes apart).
__host__ __device__ constexpr uint32_t xchunk_of(int D) { return TILE * 16 + 1024u / (uint32_t)D; }

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
    for (uint32_t it = 0; it < WAIT_LIMIT; ++it)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem], bf16 inputs, fp32 accumulate, issued by one thread.
__device__ __forceinline__ void mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 consecutive fp32 columns of this thread's tensor-memory lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
// Shared-memory matrix descriptor without swizzle: the operand is an array of core matrices of
// 8 x 16 bytes (eight 16-byte lines, 16 bytes apart).  lbo = bytes between core matrices adjacent
// along the GEMM's K dimension, sbo = bytes between core matrices adjacent along the M/N dimension
// (for K-major and for MN-major operands alike).
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo >> 4) & 0x3FFFu) << 32;
    d |= 1ull << 46;                       // descriptor version of this architecture
    return d;                              // bits 61-63 = 0: no swizzle
}
// Instruction descriptor: fp32 accumulator, bf16 A and B, M x N tile; mn_major = both operands MN-major.
__host__ __device__ inline uint32_t instr_desc(int M, int N, bool mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (mn_major ? (3u << 15) : 0u) | ((uint32_t)(N >> 3) << 17) |
           ((uint32_t)(M >> 4) << 24);
}

__host__ __device__ inline int npad_of(int K) { return (K + 31) & ~31; }   // columns of the search accumulator
__host__ __device__ inline int dpad_of(int D) { return (D + 15) & ~15; }   // K extent of the search GEMM
__host__ __device__ inline uint32_t tmem_cols_of(int D, int K, bool partials) {
    (void)D;
    uint32_t need = (uint32_t)npad_of(K) * (partials ? 2u : 1u), c = 32;       // search accumulator + sums accumulator
    while (c < need) c <<= 1;
    return c;
}

// Shared memory of a block (byte offsets).  The point tile is one array of 16 chunk columns
// (XCHUNK bytes each, chunk = 8 coordinates x 128 points): columns 0..KCH-1 hold the bf16 high parts,
// column KCH the constants [1,1,0,..,0], column KCH+1 zeros; columns 8..8+KCH-1 the low parts,
// 8+KCH and 8+KCH+1 zeros.  Read as a 128-row MN-major operand this puts the high parts (and the
// ones) in rows 0..63 and the low parts in rows 64..127 of one MMA.  The columns in between are never
// looked at as results, so they carry other data: |c|^2 and |x|^2 in columns 6-7, the centroid operand
// from column 14 on.
struct Layout {
    size_t x, cn, xn, b, oh, bar, total;
};
__host__ __device__ inline Layout layout_of(int D, int K, bool partials) {
    const size_t npad = npad_of(K), kch = dpad_of(D) / 8;
    const size_t XCHUNK = xchunk_of(D);
    Layout L;
    L.x = 0;
    L.cn = 6 * (size_t)XCHUNK;                       // npad floats (at most 256) ...
    L.xn = L.cn + 1024;                               // ... then 128 floats, then npad floats of centroid drift; all inside columns 6-7 (at least 4160 bytes)
    L.b = 14 * (size_t)XCHUNK;                        // centroid operand: npad rows x (kch + 2) chunks of 16 bytes
    size_t off = L.b + npad * (kch + 2) * 16;
    if (off < 16 * (size_t)XCHUNK) off = 16 * (size_t)XCHUNK;   // all 16 columns lie inside the allocation
    off = (off + 127) & ~(size_t)127;
    L.oh = off; off += partials ? npad / 8 * (size_t)OCHUNK : 0;   // one-hot labels; reused to combine high and low sums at the end
    L.bar = off; off += 32;                           // two mbarriers + tensor-memory address
    L.total = off;
    return L;
}

template <int D>
__device__ __forceinline__ int exact_argmin_global(const float (&x)[D], const float* __restrict__ centroids, int K) {
    float best = __int_as_float(0x7f800000);
    int bi = 0;
    for (int k = 0; k < K; ++k) {
        const float4* c = reinterpret_cast<const float4*>(centroids + (size_t)k * D);
        float d0 = 0.0f;
#pragma unroll
        for (int q = 0; q < D / 4; ++q) {
            const float4 a = __ldg(c + q);
            float t;
            t = x[4 * q] - a.x; d0 = fmaf(t, t, d0);
            t = x[4 * q + 1] - a.y; d0 = fmaf(t, t, d0);
            t = x[4 * q + 2] - a.z; d0 = fmaf(t, t, d0);
            t = x[4 * q + 3] - a.w; d0 = fmaf(t, t, d0);
        }
        if (d0 < best) { best = d0; bi = k; }     // strict <: the lowest index wins a tie
    }
    return bi;
}

template <int D>
__device__ __forceinline__ void load_point(const float* __restrict__ points, size_t j, float (&x)[D]) {
    const float4* rowp = reinterpret_cast<const float4*>(points + j * D);
#pragma unroll
    for (int q = 0; q < D / 4; ++q) {
        const float4 v = __ldg(rowp + q);
        x[4 * q] = v.x; x[4 * q + 1] = v.y; x[4 * q + 2] = v.z; x[4 * q + 3] = v.w;
    }
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);   // .x = lo (low half), .y = hi
    uint32_t u;
    memcpy(&u, &v, 4);
    return u;
}

// One 16-byte chunk of a one-hot row: the bf16 number `one` (0x3F80 = 1.0, 0xBF80 = -1.0) at position pos (0..7) of eight,
// zeros elsewhere.  (Selects, not an array indexed by pos: that would live in local memory.)
__device__ __forceinline__ uint4 onehot_chunk(int pos, uint32_t one) {
    const uint32_t v = one << (16 * (pos & 1));
    const int q = (pos & 7) >> 1;
    return make_uint4(q == 0 ? v : 0u, q == 1 ? v : 0u, q == 2 ? v : 0u, q == 3 ? v : 0u);
}
__device__ __forceinline__ uint4 or4(uint4 a, uint4 b) { return make_uint4(a.x | b.x, a.y | b.y, a.z | b.z, a.w | b.w); }

__device__ __forceinline__ float min3(float a, float b, float c) {
    float d;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// Best two of 16 scores whose low 7 mantissa bits are replaced by their column index (here: 0..15 in the low four; the
// caller adds the number of the group of 16): sorted pairs, then the same again on the smaller halves; the second best
// is the smallest of all the larger halves (the partner of the winner is among them, and every other larger half is at
// least the second best of the smaller ones).  16 at a time, so that the next 16 can be on their way from tensor memory.
// (raw & mask) | tag is ONE logic instruction when the mask comes in a register (two immediates would take two).
__device__ __forceinline__ void best_two_of_16(const uint32_t (&raw)[16], uint32_t mask, float& c1, float& c2) {
    float lo[8], hi[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        uint32_t ra, rb;
        asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(ra) : "r"(raw[2 * i]), "r"(mask), "r"((uint32_t)(2 * i)));
        asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(rb) : "r"(raw[2 * i + 1]), "r"(mask), "r"((uint32_t)(2 * i + 1)));
        const float a = __uint_as_float(ra), b = __uint_as_float(rb);
        lo[i] = fminf(a, b);
        hi[i] = fmaxf(a, b);
    }
    float hi_min = min3(min3(hi[0], hi[1], hi[2]), min3(hi[3], hi[4], hi[5]), fminf(hi[6], hi[7]));
    float l4[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) l4[i] = fminf(lo[2 * i], lo[2 * i + 1]);
    hi_min = min3(hi_min, fmaxf(lo[0], lo[1]), fmaxf(lo[2], lo[3]));
    hi_min = min3(hi_min, fmaxf(lo[4], lo[5]), fmaxf(lo[6], lo[7]));
    const float a = fminf(l4[0], l4[1]), b = fminf(l4[2], l4[3]);
    hi_min = min3(hi_min, fmaxf(l4[0], l4[1]), fmaxf(l4[2], l4[3]));
    c1 = fminf(a, b);
    c2 = fminf(hi_min, fmaxf(a, b));
}

// Which tiles of a delta-mode pass have to be searched (see the bounds in tc_fused_kernel).  Same runs as the
// fused kernel (block = run c of rank r), but nothing else to carry, so the SMs are full of warps: a warp takes
// 32 consecutive points at a time and leaves one byte, nonzero if the bounds of one of them no longer hold.
// need: [blocks][need_words] words; byte p of a block's words = points [32p, 32p + 32) of its run, so a word is a
// tile of the fused kernel.
#ifndef EC_BC_THREADS
#define EC_BC_THREADS 128
#endif
constexpr int BC_THREADS = EC_BC_THREADS;
constexpr int NEED_WORDS_MAX = 256;
__global__ void __launch_bounds__(BC_THREADS)
bounds_check_kernel(size_t N, int P, int C, int K, const int32_t* __restrict__ labels, const float2* __restrict__ bounds,
                    const float* __restrict__ drift, uint32_t* __restrict__ need, int need_words,
                    uint32_t* __restrict__ dirty, uint32_t* __restrict__ any_work) {
    __shared__ float s_d[1024 + 1];
    grid_dependency_wait();                              // (launched as a programmatic dependent of the centroid update)
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    for (int k = tid; k <= K; k += BC_THREADS) s_d[k] = drift[k];
    __syncthreads();
    const float dmax = s_d[K];
    const int r = blockIdx.x / C, c = blockIdx.x - r * C;
    const size_t j0 = (size_t)r * N / P, j1 = (size_t)(r + 1) * N / P;
    const size_t len = j1 - j0;
    const size_t b0 = j0 + len * c / C, b1 = j0 + len * (c + 1) / C;
    unsigned char* out = reinterpret_cast<unsigned char*>(need + (size_t)blockIdx.x * need_words);
    const int pieces = (int)((b1 - b0 + 31) / 32), slots = need_words * 4;
    bool mine = false;                                                 // one of this thread's points may change its label
#ifndef EC_BC_U
#define EC_BC_U 4
#endif
    constexpr int BC_U = EC_BC_U;                                            // pieces a warp has in flight
    for (int p0 = w; p0 < slots; p0 += BC_U * (BC_THREADS / 32)) {
        bool fail[BC_U];
        float2 bd[BC_U];
        int lb[BC_U];
#pragma unroll
        for (int q = 0; q < BC_U; ++q) {
            const int p = p0 + q * (BC_THREADS / 32);
            const size_t j = b0 + (size_t)p * 32 + lane;
            lb[q] = -2;
            if (p < pieces && j < b1) {
                lb[q] = labels[j];
                bd[q] = bounds[j];
            }
        }
#pragma unroll
        for (int q = 0; q < BC_U; ++q) {
            const int p = p0 + q * (BC_THREADS / 32);
            fail[q] = lb[q] == -1;                               // a point without a label
            if (lb[q] >= 0) fail[q] = !(__fmul_ru(__fadd_ru(bd[q].x, s_d[lb[q]]), 1.001f) < __fsub_rd(bd[q].y, dmax));
            const bool any = __any_sync(0xffffffffu, fail[q]);
            if (lane == 0 && p < slots) out[p] = any ? 1 : 0;    // bytes beyond the run are cleared, too
            mine = mine || fail[q];
        }
    }
    // A run without a marked tile is settled here (its row block is left alone); if there is none at all,
    // *any_work (cleared by the update kernel of the iteration before) stays 0 and the fused kernel's blocks leave at once.
    const bool any_run = __syncthreads_or(mine ? 1 : 0) != 0;
    if (tid == 0) {
        if (any_run) atomicOr(any_work, 1u);
        else dirty[blockIdx.x] = 0u;
    }
}

// Some point of this warp has its two best scores closer than the search's error bound (redo: this thread's point
// has).  The true nearest centroid's score is within tau of the best score, so the exact form decides among the columns
// with v <= lim = best + tau alone.  The scores are read once more from tensor memory (all lanes: the read is warp-wide),
// every thread notes its candidates - up to four column numbers packed in a word - and then works through its own list
// in ascending order with strict <, so the lowest index wins an exact tie as it does over all centroids; a point with
// more than four candidates is decided over all centroids.
template <int D>
__device__ __noinline__ int redecide_candidates(bool redo, int kb, float lim, const float* __restrict__ points, size_t j,
                                                uint32_t col0, int npad, const float* __restrict__ centroids, int K) {
    uint32_t cand = 0;
    int cnt = 0;
    for (int ch = 0; ch < npad / 32; ++ch) {
        uint32_t vv[32];
        tmem_ld32(col0 + (uint32_t)(ch * 32), vv);
#pragma unroll
        for (int e = 0; e < 32; ++e) {
            const bool in = __uint_as_float(vv[e]) <= lim && ch * 32 + e < K;
            cand = in ? (cand << 8) | (uint32_t)(ch * 32 + e) : cand;
            cnt += in ? 1 : 0;
        }
    }
    if (!redo) return kb;
    float x[D];
    load_point<D>(points, j, x);
    if (cnt > 4 || cnt == 0) return exact_argmin_global<D>(x, centroids, K);
    float best = __int_as_float(0x7f800000);
    for (int s = cnt - 1; s >= 0; --s) {                 // the first candidate noted sits highest in the word
        const int k = (int)((cand >> (8 * s)) & 0xFFu);
        const float4* c = reinterpret_cast<const float4*>(centroids + (size_t)k * D);
        float d0 = 0.0f;
#pragma unroll
        for (int q = 0; q < D / 4; ++q) {
            const float4 a = __ldg(c + q);
            float u;
            u = x[4 * q] - a.x; d0 = fmaf(u, u, d0);
            u = x[4 * q + 1] - a.y; d0 = fmaf(u, u, d0);
            u = x[4 * q + 2] - a.z; d0 = fmaf(u, u, d0);
            u = x[4 * q + 3] - a.w; d0 = fmaf(u, u, d0);
        }
        if (d0 < best) { best = d0; kb = k; }
    }
    return kb;
}

template <int D, bool PARTIALS, bool DELTA, bool BOUNDS>
__global__ void __launch_bounds__(THREADS, EC_TC_MINB)
tc_fused_kernel(const float* __restrict__ points, size_t N, int P, int C, const float* __restrict__ centroids, int K,
                int32_t* __restrict__ labels, float* __restrict__ scratch, float tau_scale, uint32_t* __restrict__ status,
                uint32_t* __restrict__ dirty, float2* __restrict__ bounds, const float* __restrict__ drift,
                const uint32_t* __restrict__ need, int need_words) {
    grid_dependency_wait();                              // (a no-op unless launched as a programmatic dependent)
    constexpr bool delta = DELTA;                        // sum only what changed since the labels were written last
    constexpr int KCH = D / 8;                           // 16-byte chunks of coordinates per point
    static_assert(D % 16 == 0 && KCH + 2 <= 8 && (KCH & (KCH - 1)) == 0, "D is 16 or 32");
    constexpr int LO = 8;                                // first chunk column of the low parts
    constexpr uint32_t XCHUNK = xchunk_of(D);
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int npad = npad_of(K);
    const Layout L = layout_of(D, K, PARTIALS);
    unsigned char* s_x = smem_raw + L.x;
    float* s_cn = reinterpret_cast<float*>(smem_raw + L.cn);
    float* s_xn = reinterpret_cast<float*>(smem_raw + L.xn);
    float* s_drift = s_xn + TILE;                        // [npad]: how far every centroid has moved in all (bounds only)
    unsigned char* s_b = smem_raw + L.b;
    unsigned char* s_oh = smem_raw + L.oh;
    uint64_t* s_bar = reinterpret_cast<uint64_t*>(smem_raw + L.bar);
    uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem_raw + L.bar + 16);

    const int tid = threadIdx.x, w = tid >> 5;
    const uint32_t ncols = tmem_cols_of(D, K, PARTIALS);
    const uint32_t bar1 = smem_u32(s_bar), bar2 = smem_u32(s_bar + 1);

    // A block works through the runs blockIdx.x, blockIdx.x + gridDim.x, ... (run = (rank r, part c) of the points;
    // the grid is one wave of resident blocks), so the set-up below is paid once per block.
    const int runs = P * C;
    // Delta mode with distance bounds: bounds_check_kernel has looked at every point and left one byte per 32
    // points, nonzero if one of them may change its label; a word is a tile.  A run without such a tile is
    // done at once, and a block none of whose runs has one before anything is set up: once the centroids have
    // settled that is every block.
    const bool skipping = DELTA && PARTIALS && BOUNDS && need != nullptr;
    uint32_t* s_need = reinterpret_cast<uint32_t*>(s_xn + TILE + 256);   // [need_words] (at most 256), after the drift table
    if (skipping) {
        if (reinterpret_cast<const uint32_t*>(drift)[K + 1] == 0u) return;   // no tile anywhere: the check has settled every run
        bool any = false;
        for (int run = blockIdx.x; run < runs; run += gridDim.x)
            for (int q = tid; q < need_words; q += THREADS) any = any || need[(size_t)run * need_words + q] != 0u;
        if (!__syncthreads_or(any ? 1 : 0)) {
            for (int run = blockIdx.x + tid * gridDim.x; run < runs; run += THREADS * gridDim.x) dirty[run] = 0u;   // the row blocks are left alone
            return;
        }
    }
    if (w == 0) tmem_alloc(smem_u32(s_tmem), ncols);
    if (tid == 0) {
        mbar_init(bar1, 1);
        mbar_init(bar2, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // Centroid operand (K-major, chunk kc of centroid n at kc*(npad*16) + n*16): -2 c in bf16 (the doubling is
    // exact), then one chunk [hi(|c|^2), lo(|c|^2), 0, ...] that meets the points' [1, 1, 0, ...] chunk, so
    // that the GEMM delivers v = |c|^2 - 2 x.c itself; padding centroids get a |c|^2 that can never win.
    for (int k = tid; k < npad; k += THREADS) {
        float s = 3.0e38f;
        if (k < K) {
            s = 0.0f;
            for (int d = 0; d < D; ++d) s = fmaf(centroids[(size_t)k * D + d], centroids[(size_t)k * D + d], s);
        }
        s_cn[k] = s;
        const uint32_t hl = pack_bf16(s, 0.0f) & 0xFFFFu;
        const float hi = __uint_as_float(hl << 16);
        const uint32_t both = hl | (pack_bf16(s - hi, 0.0f) << 16);
        *reinterpret_cast<uint4*>(s_b + (size_t)KCH * npad * 16 + (size_t)k * 16) = make_uint4(both, 0u, 0u, 0u);
        *reinterpret_cast<uint4*>(s_b + (size_t)(KCH + 1) * npad * 16 + (size_t)k * 16) = make_uint4(0u, 0u, 0u, 0u);
    }
    for (int i = tid; i < npad * KCH; i += THREADS) {
        const int kc = i / npad, n = i - kc * npad;
        float v[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) v[e] = n < K ? -2.0f * centroids[(size_t)n * D + kc * 8 + e] : 0.0f;
        *reinterpret_cast<uint4*>(s_b + (size_t)kc * npad * 16 + (size_t)n * 16) =
            make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
    }
    if (PARTIALS && BOUNDS)
        for (int k = tid; k < npad; k += THREADS) s_drift[k] = k < K ? drift[k] : 0.0f;
    // constant chunk columns of the point tile
    *reinterpret_cast<uint4*>(s_x + (size_t)KCH * XCHUNK + (size_t)tid * 16) = make_uint4(0x3F803F80u, 0u, 0u, 0u);   // [1, 1, 0, ...]
    *reinterpret_cast<uint4*>(s_x + (size_t)(KCH + 1) * XCHUNK + (size_t)tid * 16) = make_uint4(0u, 0u, 0u, 0u);
    if (PARTIALS) {
        *reinterpret_cast<uint4*>(s_x + (size_t)(LO + KCH) * XCHUNK + (size_t)tid * 16) = make_uint4(0u, 0u, 0u, 0u);
        *reinterpret_cast<uint4*>(s_x + (size_t)(LO + KCH + 1) * XCHUNK + (size_t)tid * 16) = make_uint4(0u, 0u, 0u, 0u);
        for (int ch = 0; ch < npad / 8; ++ch)
            *reinterpret_cast<uint4*>(s_oh + (size_t)ch * OCHUNK + (size_t)tid * 16) = make_uint4(0u, 0u, 0u, 0u);
    }
    fence_async_smem();
    fence_before_sync();
    __syncthreads();
    fence_after_sync();
    const uint32_t tmem_base = *s_tmem;
    const uint32_t tmem_lane = tmem_base + ((uint32_t)(w * 32) << 16);   // this warp's 32 lanes
    float cmax = 0.0f;
    for (int k = 0; k < K; ++k) cmax = fmaxf(cmax, s_cn[k]);
    uint32_t tag_mask;                                   // 0xFFFFFF00 in a register (see best_two_of_16; up to 256 columns here)
    asm volatile("mov.u32 %0, 0xFFFFFF00;" : "=r"(tag_mask));
    const uint32_t idesc_search = instr_desc(MROWS, npad, false);
    const uint32_t idesc_sum = instr_desc(MROWS, npad, true);
    const uint32_t b_base = smem_u32(s_b), x_base = smem_u32(s_x), oh_base = smem_u32(s_oh);

    const int stride = D + 4;
    uint32_t phase1 = 0, phase2 = 0;
    bool healthy = true;             // false once a wait on the tensor core gave up: plain fp32 from then on
    bool oh_clean = true;            // the one-hot tile is all zeros
    constexpr bool keep_bounds = PARTIALS && BOUNDS;     // (the host passes the arrays whenever it picks this instantiation)
    const float drift_max = keep_bounds ? drift[K] : 0.0f;

    for (int run = blockIdx.x; run < runs; run += gridDim.x) {
    const int r = run / C, c = run - r * C;
    const size_t j0 = (size_t)r * N / P, j1 = (size_t)(r + 1) * N / P;
    const size_t len = j1 - j0;
    const size_t b0 = j0 + len * c / C, b1 = j0 + len * (c + 1) / C;
    if (skipping) {
        bool any = false;
        for (int q = tid; q < need_words; q += THREADS) {
            const uint32_t wd = need[(size_t)run * need_words + q];
            s_need[q] = wd;
            any = any || wd != 0u;
        }
        if (!__syncthreads_or(any ? 1 : 0)) {
            if (tid == 0) dirty[run] = 0u;               // the row block is left alone
            continue;
        }
    }
    float* row_block = PARTIALS ? scratch + (size_t)run * (size_t)K * stride : nullptr;
    if (PARTIALS && !oh_clean) {     // the run before used the one-hot tile as scratch for its sums
        for (int ch = 0; ch < npad / 8; ++ch)
            *reinterpret_cast<uint4*>(s_oh + (size_t)ch * OCHUNK + (size_t)tid * 16) = make_uint4(0u, 0u, 0u, 0u);
        oh_clean = true;
    }
    bool sums_started = false;       // a sums MMA has been issued (the accumulator holds data)
    bool sums_pending = false;       // ... and its completion has not been waited for yet
    int prev_chunk = -1;             // one-hot chunk this thread set in the previous tile
    int prev_chunk2 = -1;            // ... and a second one (delta mode: the chunk of the label the point left)
    bool by_hand = false;            // some points were added to the row block with atomic adds

    // A thread stages KCH items (point row, chunk kc of 8 coordinates) of a tile: consecutive threads take
    // consecutive 32-byte pieces of the points, so every load instruction of a warp covers 1 KB of contiguous
    // memory.  The loads of the next tile are issued as soon as the current one is staged and stay in flight
    // while the current tile is searched.
    float4 va[KCH], vb[KCH];
    auto issue_loads = [&](size_t tile_base) {
#pragma unroll
        for (int q = 0; q < KCH; ++q) {
            const int idx = q * THREADS + tid, row = idx / KCH, kc = idx % KCH;
            const size_t jr = tile_base + row;
            if (jr < b1) {
                const float4* src = reinterpret_cast<const float4*>(points + jr * D + kc * 8);
                va[q] = __ldg(src);
                vb[q] = __ldg(src + 1);
            } else {
                va[q] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                vb[q] = va[q];
            }
        }
    };
    // Bounds (delta mode): for every point an upper bound u on the distance to its own centroid and a lower
    // bound l on the distance to any other, both taken when the point was last searched and stored relative to
    // the drift sums of then (u - drift[label], l + drift_max).  Centroid k has since moved by at most
    // drift[k] - (its value then), any centroid by at most drift_max - (its value then), so u + drift[label] still
    // bounds the one distance from above and l - drift_max the others from below (triangle inequality; all
    // roundings directed).  A tile in which every point has u < l by a margin far above the rounding of the
    // exact form keeps its labels: it is not read at all.
    bool pts_ready = false;                              // the registers hold the loads of the tile at hand
    if (!skipping) {
        issue_loads(b0);
        pts_ready = true;
    }

    for (size_t base = b0; base < b1; base += TILE) {
        if (skipping && s_need[(base - b0) / TILE] == 0u) {  // nothing in this tile can change
            pts_ready = false;
            continue;
        }
        const size_t j = base + tid;
        const bool live = j < b1;
        if (!pts_ready) issue_loads(base);               // the tile before was skipped: its points are fetched now
        pts_ready = false;
        const int old = (delta && live) ? labels[j] : -1;   // delta mode: the label this point had (asked for early: used after the search)
        if (PARTIALS && sums_pending) {
            // the previous tile's sums MMA still reads the tile: wait for it (its latency hid behind the search)
            const bool ok = mbar_wait_bounded(bar2, phase2);
            phase2 ^= 1u;
            sums_pending = false;
            if (!ok) healthy = false;
        }
        if (PARTIALS && prev_chunk >= 0) {
            *reinterpret_cast<uint4*>(s_oh + (size_t)prev_chunk * OCHUNK + (size_t)tid * 16) = make_uint4(0u, 0u, 0u, 0u);
            prev_chunk = -1;
        }
        if (PARTIALS && prev_chunk2 >= 0) {
            *reinterpret_cast<uint4*>(s_oh + (size_t)prev_chunk2 * OCHUNK + (size_t)tid * 16) = make_uint4(0u, 0u, 0u, 0u);
            prev_chunk2 = -1;
        }
        // bf16 high parts and low parts (low = bf16(x - high)) at chunk column kc resp. LO + kc, row*16
#pragma unroll
        for (int q = 0; q < KCH; ++q) {
            const int idx = q * THREADS + tid, row = idx / KCH, kc = idx % KCH;
            const float v[8] = {va[q].x, va[q].y, va[q].z, va[q].w, vb[q].x, vb[q].y, vb[q].z, vb[q].w};
            uint32_t hw[4], lw[4];
            float sq = 0.0f;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float a = v[2 * e], b = v[2 * e + 1];
                sq = fmaf(a, a, sq);
                sq = fmaf(b, b, sq);
                hw[e] = pack_bf16(a, b);
            }
            *reinterpret_cast<uint4*>(s_x + (size_t)kc * XCHUNK + (size_t)row * 16) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
            if (PARTIALS && !delta) {    // delta mode: the low parts are made only for a tile that turns out to hold a change
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float ah = __uint_as_float(hw[e] << 16), bh = __uint_as_float(hw[e] & 0xFFFF0000u);
                    lw[e] = pack_bf16(v[2 * e] - ah, v[2 * e + 1] - bh);
                }
                *reinterpret_cast<uint4*>(s_x + (size_t)(LO + kc) * XCHUNK + (size_t)row * 16) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
            }
            // |x|^2 of the row: its KCH chunks sit in KCH consecutive lanes
#pragma unroll
            for (int o = 1; o < KCH; o <<= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
            if (kc == 0) s_xn[row] = sq;
        }
        if (base + TILE < b1) {      // this tile had to be searched: the next one probably has to be, too
            issue_loads(base + TILE);
            pts_ready = true;
        }
        fence_async_smem();          // the tensor core reads shared memory through the async proxy
        healthy = __syncthreads_and(healthy) != 0;
        const float xn = s_xn[tid];  // taken now: a warp that runs ahead stages the next tile's norms over this array
        if (tid == 0 && healthy) {
            fence_after_sync();
#pragma unroll
            for (int ks = 0; ks < D / 16 + 1; ++ks) {    // search: rows = points (K-major), columns = centroids; last step adds |c|^2
                const uint64_t ad = smem_desc(x_base + ks * 2 * XCHUNK, XCHUNK, 128);
                const uint64_t bd = smem_desc(b_base + ks * 2 * npad * 16, npad * 16, 128);
                mma_bf16(tmem_base, ad, bd, idesc_search, ks > 0 ? 1u : 0u);
            }
            mma_commit(bar1);
        }
        bool done = healthy && mbar_wait_bounded(bar1, phase1);
        phase1 ^= 1u;
        done = __syncthreads_and(done) != 0;     // all threads take the same path
        if (PARTIALS && !done && !by_hand) {     // first tile without the tensor core: clear the base of the by-hand adds
            for (int i = tid; i < K * stride; i += THREADS) row_block[i] = 0.0f;
            by_hand = true;
            __syncthreads();
        }
        healthy = done;
        fence_after_sync();
        float m1 = __int_as_float(0x7f800000), m2 = m1;
        int kb = 0;
        if (done) {
            // the best two scores by a tournament of min/max pairs; the low 7 mantissa bits of a score are replaced by its
            // column (a change of less than 2^-16 of the score: far inside the margin of tau)
            for (int ch = 0; ch < npad / 32; ++ch) {
                uint32_t vv[32];
                tmem_ld32(tmem_lane + (uint32_t)(ch * 32), vv);
                uint32_t lo_half[16], hi_half[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) { lo_half[e] = vv[e]; hi_half[e] = vv[16 + e]; }
                float c1, c2;
                best_two_of_16(lo_half, tag_mask, c1, c2);
                c1 = __uint_as_float(__float_as_uint(c1) | (uint32_t)(ch << 5));
                m2 = min3(m2, c2, fmaxf(m1, c1));
                m1 = fminf(m1, c1);
                best_two_of_16(hi_half, tag_mask, c1, c2);
                c1 = __uint_as_float(__float_as_uint(c1) | (uint32_t)((ch << 5) | 16));
                m2 = min3(m2, c2, fmaxf(m1, c1));
                m1 = fminf(m1, c1);
            }
            kb = (int)(__float_as_uint(m1) & 255u);
        } else if (tid == 0 && status != nullptr) {
            atomicOr(status, 1u);    // the tensor core did not answer in time
        }
        fence_before_sync();         // accumulator reads are done before the next tile's MMA may overwrite it
        // Error of the search.  bf16 keeps 8 significant bits: rounding to nearest changes a number by a factor
        // (1 + e) with |e| <= u/(1+u), u = 2^-8, so a product of two rounded numbers is off by less than 2u of
        // itself and the term -2 x.c_k by less than 4u sum_d |x_d c_kd| <= 4u |x||c_k| <= 2u (|x|^2 + |c_k|^2):
        // one candidate's v is wrong by less than 2^-7 (|x|^2 + |c_k|^2), the difference of two candidates' v by less
        // than 2^-6 (|x|^2 + |c|max^2).  The rest is far smaller: |c_k|^2 enters as hi + lo with 16 significant bits
        // (2^-16 |c_k|^2) and the D + 2 products, exact in fp32, are added up in fp32 (at most (D+2) 2^-23 of the
        // largest partial sum).  tau = (2^-6 + 2^-10)(|x|^2 + |c|max^2) covers the first part exactly and leaves
        // 2^-10 (|x|^2 + |c|max^2), 64 times the rest for D = 32, for the second.
        const float tau = tau_scale * (xn + cmax);
        const bool redo = live && (!done || !(m2 - m1 > tau));
        // Delta mode: the row block receives only what changed since the labels were written last: +x for the
        // cluster a point joins, -x for the one it leaves (old label < 0: it was in none).  A tile in which no
        // label changed needs no sums MMA at all.  Otherwise every live point joins its cluster.
        if (done && __any_sync(0xffffffffu, redo))        // (the accumulator is still this tile's: the next MMA comes after the next barrier)
        {
            kb = redecide_candidates<D>(redo, kb, m1 + tau, points, j, tmem_lane, npad, centroids, K);
            fence_before_sync();                         // these reads, too, come before the barrier that lets the next MMA start
        }
        if (live && !done) {
            float x[D];
            load_point<D>(points, j, x);                 // the tensor core is out of service: plain fp32 for this point
            kb = exact_argmin_global<D>(x, centroids, K);
            if (PARTIALS && !done && !(delta && old == kb)) {   // tensor core out of service: add this point by hand
#pragma unroll
                for (int d = 0; d < D; ++d) atomicAdd(row_block + (size_t)kb * stride + d, x[d]);
                atomicAdd(row_block + (size_t)kb * stride + D, 1.0f);
                if (old >= 0) {
#pragma unroll
                    for (int d = 0; d < D; ++d) atomicAdd(row_block + (size_t)old * stride + d, -x[d]);
                    atomicAdd(row_block + (size_t)old * stride + D, -1.0f);
                }
            }
        }
        const bool changed = live && !(delta && old == kb);
        if (changed) labels[j] = kb;
        if (keep_bounds && live) {
            float2 w = make_float2(__int_as_float(0x7f800000), 0.0f);      // decided by the exact form: searched again next time
            if (done && !redo) {
                // |x - c|^2 = |x|^2 + v; the search knows v to within tau
                const float u = __fsqrt_ru(fmaxf(__fadd_ru(__fadd_ru(xn, m1), tau), 0.0f));
                const float l = __fsqrt_rd(fmaxf(__fsub_rd(__fadd_rd(xn, m2), tau), 0.0f));
                w = make_float2(__fsub_ru(u, s_drift[kb]), __fadd_rd(l, drift_max));
            }
            bounds[j] = w;
        }
        if (PARTIALS && done) {
            if (changed) {
                // one-hot row of this point: 16-byte chunk kb/8, bf16 1.0 at position kb%8 (and -1.0 for the old label)
                uint4 wv = onehot_chunk(kb, 0x3F80u);
                prev_chunk = kb >> 3;
                if (old >= 0 && (old >> 3) == prev_chunk) wv = or4(wv, onehot_chunk(old, 0xBF80u));
                *reinterpret_cast<uint4*>(s_oh + (size_t)prev_chunk * OCHUNK + (size_t)tid * 16) = wv;
                if (old >= 0 && (old >> 3) != prev_chunk) {
                    prev_chunk2 = old >> 3;
                    *reinterpret_cast<uint4*>(s_oh + (size_t)prev_chunk2 * OCHUNK + (size_t)tid * 16) = onehot_chunk(old, 0xBF80u);
                }
            }
            fence_async_smem();
            const bool any_changed = __syncthreads_or(changed ? 1 : 0) != 0;
            if (any_changed && delta) {
                // rare once the labels have settled: read the tile again (it is still in L2) and stage the low parts
#pragma unroll
                for (int q = 0; q < KCH; ++q) {
                    const int idx = q * THREADS + tid, row = idx / KCH, kc = idx % KCH;
                    const size_t jr = base + row;
                    float4 ta = make_float4(0.0f, 0.0f, 0.0f, 0.0f), tb = ta;
                    if (jr < b1) {
                        const float4* src = reinterpret_cast<const float4*>(points + jr * D + kc * 8);
                        ta = __ldg(src);
                        tb = __ldg(src + 1);
                    }
                    const float v[8] = {ta.x, ta.y, ta.z, ta.w, tb.x, tb.y, tb.z, tb.w};
                    uint32_t lw[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float a = v[2 * e], b = v[2 * e + 1];
                        const uint32_t h = pack_bf16(a, b);
                        lw[e] = pack_bf16(a - __uint_as_float(h << 16), b - __uint_as_float(h & 0xFFFF0000u));
                    }
                    *reinterpret_cast<uint4*>(s_x + (size_t)(LO + kc) * XCHUNK + (size_t)row * 16) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
                }
                fence_async_smem();
                __syncthreads();
            }
            if (any_changed && tid == 0) {
                fence_after_sync();
                // sums[row][k] += sum_j X[j][row] * onehot[j][k], 16 points per step, both operands MN-major:
                // consecutive points are 16 bytes apart (K direction: 8 points = 128 bytes), consecutive chunks
                // of 8 rows / 8 centroids are XCHUNK / OCHUNK bytes apart (M/N direction).  One MMA covers the
                // high parts with the ones (rows 0..63) and the low parts (rows 64..127).
#pragma unroll
#pragma unroll
                for (int ks = 0; ks < TILE / 16; ++ks) {
                    const uint64_t ad = smem_desc(x_base + ks * 256, 128, XCHUNK);
                    const uint64_t bd = smem_desc(oh_base + ks * 256, 128, OCHUNK);
                    mma_bf16(tmem_base + (uint32_t)npad, ad, bd, idesc_sum, (sums_started || ks > 0) ? 1u : 0u);
                }
                mma_commit(bar2);
            }
            if (any_changed) {
                sums_started = true;
                sums_pending = true;
            }
        }
    }
    if (PARTIALS) {
        bool ok = true;
        if (sums_pending) {
            ok = mbar_wait_bounded(bar2, phase2);
            phase2 ^= 1u;                        // the block goes on with its next run
            sums_pending = false;
            if (!ok) healthy = false;
        }
        ok = __syncthreads_and(ok) != 0;
        fence_after_sync();
        if (!ok && tid == 0 && status != nullptr) atomicOr(status, 1u);
        // This thread's tensor-memory lane is row tid of the accumulator; columns are the centroids.
        // Rows 0..D-1: high-part sums of coordinate tid; row D: the counts; rows 64..64+D-1: low-part sums.
        // The low rows go through shared memory (the one-hot tile is free now) to the thread of their coordinate.
        if (ok && sums_started) {
            float* s_lo = reinterpret_cast<float*>(s_oh);          // [npad][D] floats <= npad/8 * 2048 bytes for D <= 32... (D*4 <= 256)
            oh_clean = false;
            const bool is_hi = tid < D, is_cnt = tid == D, is_pad = tid > D && tid < D + 4, is_lo = tid >= 64 && tid < 64 + D;
            for (int ch = 0; ch < npad / 32; ++ch) {
                uint32_t v[32];
                tmem_ld32(tmem_lane + (uint32_t)(npad + ch * 32), v);
                if (is_lo) {
#pragma unroll
                    for (int e = 0; e < 32; ++e) s_lo[(size_t)(ch * 32 + e) * D + (tid - 64)] = __uint_as_float(v[e]);
                }
                __syncthreads();
                if (is_hi || is_cnt || is_pad) {
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        const int k = ch * 32 + e;
                        if (k < K) {
                            float val = is_pad ? 0.0f : __uint_as_float(v[e]);
                            if (is_hi) val = __fadd_rn(val, s_lo[(size_t)k * D + tid]);
                            float* dst = row_block + (size_t)k * stride + tid;   // column tid: coordinate, D = the count, then zeros
                            if (!by_hand) *dst = val;
                            else if (!is_pad) atomicAdd(dst, val);                // some tiles were added by hand
                        }
                    }
                }
            }
        }
    }
    if (PARTIALS && delta) {                     // delta mode: a run without changes leaves its row block alone and says so
        if (tid == 0) dirty[run] = (sums_started || by_hand) ? 1u : 0u;
    } else if (PARTIALS && !sums_started && !by_hand) {   // an empty run: its row block is all zeros
        for (int i = tid; i < K * stride; i += THREADS) row_block[i] = 0.0f;
    }
    // A run that issued a sums MMA leaves entries in the one-hot tile (the last tile's, and the sums scratch above):
    // the next run clears the whole tile before it uses it.  (Not here: other warps may still be reading the scratch.)
    if (sums_started) oh_clean = false;
    fence_before_sync();
    __syncthreads();                             // the run's shared memory (sums scratch, tile flags) is free for the next one
    fence_after_sync();
    }   // runs
    fence_before_sync();
    __syncthreads();
    if (w == 0) tmem_dealloc(tmem_base, ncols);
}

}  // namespace tc
}  // namespace ec
