// K-means assignment + partial sums, warp-specialised: the form ec_kmeans_iterate takes for D in {16, 32}, K <= 128.
//
// One persistent block per SM.  The fp32 points never pass through registers on their way to the tensor core:
//
//   producer (one thread)    walks the block's runs and, for every tile of 128 points that has to be searched,
//                            issues one bulk tensor copy (cp.async.bulk.tensor.2d, 128-byte swizzle, this block only,
//                            this GPU's memory only) into a ring of shared-memory stages, each with its mbarrier;
//   search issuers (two threads: even tiles, odd tiles) multiply a landed tile, as it lies, with the centroid
//                            operand: tcgen05.mma kind::tf32,
//                            A = the stage (128 points x D floats, K-major), B = -2 c rounded to tf32 (K-major, same
//                            swizzle), plus one step of a constant [1,1,1,0..] chunk against [hi, mid, lo](|c|^2), so
//                            the accumulator in tensor memory holds v_k = |c_k|^2 - 2 x.c_k for 128 points x all
//                            centroids.  Tile i goes to accumulator i mod A, A = as many as tensor memory holds beside
//                            the sums (six for K = 64), so the search runs ahead of the groups;
//   epilogue groups (4 warps each, tile i goes to group i mod G): read the scores with tcgen05.ld (one point per
//                            thread, 16 columns at a time with the next 16 on their way), find the best two by a
//                            tournament of min/max pairs whose low mantissa bits carry the column index, decide (exact
//                            fp32 form from the staged row whenever the two are closer than the search's error bound tau),
//                            write label and distance bounds, and - only a thread whose label changed - convert the
//                            staged row to bf16 high + low parts and set the one-hot row for the sums GEMM.  The warps
//                            of a group never meet: each waits and arrives for itself (one lane per warp);
//   sums issuer (one thread)  sums[d][k] += sum_j x[j][d] onehot[j][k] as tcgen05.mma kind::f16 over such tiles, in
//                            tile order (so the sums repeat bit for bit), accumulator in tensor memory per run, double
//                            buffered so that a run is written out while the next one accumulates.
//
// Every wait (mbarrier) is bounded; a wait that gives up raises an abort flag that every role polls, the block sets a
// status word, waits (bounded) for its copies in flight, frees its tensor memory and returns.  The results of a launch
// whose status word is nonzero are not valid.
//
// Error of the search (kind::tf32).  The tensor core keeps 11 significant bits of an fp32 operand; whether it rounds
// or truncates, a point's coordinate is changed by a factor (1 + e), |e| <= 2^-10.  The centroids are rounded to
// nearest here, |e| <= 2^-11.  A product is off by less than 1.5001 * 2^-10 of itself, the term -2 x.c_k by less
// than 3.0002 * 2^-10 |x||c_k| <= 1.5001 * 2^-10 (|x|^2 + |c_k|^2); |c_k|^2 enters exactly (three tf32 terms), the
// products are exact in fp32 and the few additions cost at most (D/8 + 2) 2^-23 of the largest partial sum.  Tagging a
// score with its column (7 low mantissa bits) moves it by less than 2^-16 |v| <= 2^-15 (|x|^2 + |c|^2).  The
// difference of two candidates' scores is therefore known to within 3.0002 * 2^-10 + 2^-14 + ... < 3.1 * 2^-10 of
// (|x|^2 + |c|max^2); tau = 2^-8 = 4 * 2^-10 of it.  One score alone is within tau / 2.
#pragma once

#include <cuda.h>

#ifndef EC_WS_HINT
#define EC_WS_HINT 20000
#endif

namespace ec {
namespace ws {

using tc::fence_after_sync;
using tc::fence_async_smem;
using tc::fence_before_sync;
using tc::best_two_of_16;
using tc::mbar_init;
using tc::min3;
using tc::mma_commit;
using tc::npad_of;
using tc::pack_bf16;
using tc::smem_desc;
using tc::smem_u32;
using tc::tmem_alloc;
using tc::tmem_dealloc;

constexpr int TILE = 128;                       // points per tile = rows of an accumulator
constexpr int MAX_GROUPS = 4;                   // epilogue groups of four warps (3: the same speed; 5, 6: slower, registers spill)
constexpr int MAX_STAGES = 8;
constexpr int MAX_ACCS = 8;
constexpr int MAX_SLOTS = 4;                    // operand buffers of the sums GEMM: 2 when only changes are summed, else 4
constexpr int MAX_THREADS = (4 * MAX_GROUPS + 4) * 32;
constexpr uint32_t WAIT_LIMIT = 1u << 24;
constexpr uint32_t OCHUNK = TILE * 16;          // one-hot tile: bytes between chunks of 8 centroids
constexpr float TAU_SCALE = 0.00390625f;        // 2^-8, see above
// bf16 operand of the sums GEMM: bytes between chunk columns (8 coordinates x 128 points x 2 bytes, padded so that
// consecutive columns start in different banks)
__host__ __device__ constexpr uint32_t xchunk_of(int D) { return TILE * 16 + 1024u / (uint32_t)D; }

// Shared memory of a block (byte offsets from a 1024-byte aligned base) and its tensor-memory columns.
struct Plan {
    int groups, stages, slots, accs;                // accs: search accumulators in tensor memory (tile i uses i mod accs)
    uint32_t tmem_cols;
    uint32_t stage_bytes, slot_bytes, oh_off;       // oh_off: one-hot tile inside a slot
    uint32_t stage, b, ones, cnb, slot, prev, cn, drift, need, desc, ctrl, bar, total;
};
__host__ __device__ inline Plan plan_of(int D, int K, bool partials, bool delta) {
    Plan p;
    const uint32_t npad = (uint32_t)npad_of(K), XC = xchunk_of(D);
    const uint32_t acc = partials ? 2u : 0u;
    int g = (int)(512u / npad) - (int)acc;
    p.groups = g > MAX_GROUPS ? MAX_GROUPS : g < 1 ? 1 : g;
    // All points summed: four slots for three groups, so that the slot a group converts into was last used by another
    // group's tile, decided a whole tile earlier - its sums GEMM is over (measured on N = 2^22, D = 32, K = 64: 269 us per
    // iteration; four groups on four slots 314, four groups on three slots with the rows converted after the decision 375;
    // a group converting the next group's tile instead of its own: 310 with four groups, 325 with three).
    if (partials && !delta && p.groups > 3) p.groups = 3;
    // Search accumulators: as many as tensor memory holds beside the two of the sums (at most MAX_ACCS), so that the search
    // of a group's next tile is over before the group asks for it, whatever else the tensor core had queued.
#ifndef EC_WS_ACCS
#define EC_WS_ACCS MAX_ACCS
#endif
    int a = (int)(512u / npad) - (int)acc;
    p.accs = a > EC_WS_ACCS ? EC_WS_ACCS : a < p.groups ? p.groups : a;
    if (p.accs > p.groups && (p.accs & 1)) --p.accs;   // even, if that costs no group its accumulator: both search issuers can work
    uint32_t need = ((uint32_t)p.accs + acc) * npad, cols = 32;
    while (cols < need) cols <<= 1;
    p.tmem_cols = cols;
    p.stage_bytes = (uint32_t)TILE * (uint32_t)D * 4u;
    const uint32_t kch = (uint32_t)D / 8u;
    p.oh_off = ((2u * kch + 1u) * XC + 127u) & ~127u;   // high/low columns interleaved, then the ones column
    uint32_t slot = p.oh_off + npad / 8u * OCHUNK;
    if (slot < 16u * XC) slot = 16u * XC;            // the sums MMA reads 128 rows = 16 chunk columns from the slot's start
    p.slot_bytes = (slot + 127u) & ~127u;
    // Slots.  Only changes summed: one per group if that leaves four stages - a group then has its slot to itself and asks
    // nobody about its state (7220 instead of 6720 iterations/s on N = 2^22, D = 32, K = 64 with every tile searched: with
    // two slots a group's hand-over waited until the group two tiles behind had handed over) - else two.  All points
    // summed: four if that leaves three stages, else three.
    p.slots = partials ? (delta ? p.groups : MAX_SLOTS) : 0;
    uint32_t off = 0;
    for (;;) {
        const uint32_t SLOTS = (uint32_t)p.slots;
        const uint32_t fixed_after_stages = npad * (uint32_t)D * 4u + 1024u   // b (1024-aligned)
            + 4096u + npad * 32u                                              // ones, cnb
            + SLOTS * p.slot_bytes + SLOTS * TILE * 2u                        // slots, previous one-hot chunks
            + npad * 8u + 1024u + 4096u;                                       // cn, drift, need words, descriptors, control, barriers
        const int st = fixed_after_stages < 226u * 1024u ? (int)((226u * 1024u - fixed_after_stages) / p.stage_bytes) : 0;
        p.stages = st > MAX_STAGES ? MAX_STAGES : st;
        if (partials && !delta && p.slots > 3 && p.stages < 3) { p.slots = 3; continue; }
        if (partials && delta && p.slots > 2 && p.stages < 4) { p.slots = 2; continue; }
        break;
    }
    const uint32_t SLOTS = (uint32_t)p.slots;
    p.stage = off; off += (uint32_t)p.stages * p.stage_bytes;
    off = (off + 1023u) & ~1023u;
    p.b = off; off += npad * (uint32_t)D * 4u;       // -2 c, tf32, K-major, swizzled like the stages
    p.ones = off; off += 4096u;                      // [2 chunks][128 rows][16 bytes]: (1,1,1,0 | 0,0,0,0), no swizzle
    p.cnb = off; off += npad * 32u;                  // [2 chunks][npad rows][16 bytes]: (hi, mid, lo, 0 | 0...) of |c|^2
    off = (off + 127u) & ~127u;
    p.slot = off; off += SLOTS * p.slot_bytes;
    p.prev = off; off += SLOTS * TILE * 2u;
    p.cn = off; off += npad * 4u;
    p.drift = off; off += npad * 4u;
    p.need = off; off += 1024u;
    p.desc = off; off += MAX_STAGES * 32u;
    p.ctrl = off; off += 256u;
    p.bar = off; off += 512u;
    p.total = off + 1024u;                           // slack to align the base
    return p;
}
inline int threads_of(const Plan& p) { return (4 * p.groups + 4) * 32; }

// What the producer says about the tile in a stage.
struct TileDesc {
    unsigned long long base;     // index of the tile's first point
    unsigned long long end;      // one past the run's last point
    int run;                     // run index (row block), -1: no more tiles
    int run_seq;                 // how many runs with tiles this block has started before this tile's run
    int last;                    // the run's last tile
    int pad;                     // the tile's number in the block's sequence (what a reader expects to find)
};

// One try; the thread may sleep in hardware until the phase completes or the hinted time (nanoseconds) has passed, so
// a waiting warp costs few issue slots.
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"((uint32_t)EC_WS_HINT)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void tma_tile_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
// Bounded wait (in tries and in time: about two seconds); gives up early when another role has raised the abort flag.
__device__ __forceinline__ bool wait_or_abort(uint32_t bar, uint32_t parity, volatile int* abort_flag, int where) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 63u) {
            if (*abort_flag != 0) return false;
            if (clock64() - t0 > 4000000000LL) break;
        }
    }
    if (*abort_flag == 0) *abort_flag = where;               // which wait gave up first (reported in the status word)
    return false;
}
__device__ __forceinline__ void mma_tf32(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// K-major operand whose rows are one swizzle span wide (128 bytes for D = 32, 64 bytes for D = 16): groups of 8 rows
// are 8 spans apart.
template <int D>
__device__ __forceinline__ uint64_t swz_desc(uint32_t saddr) {
    constexpr uint32_t span = D * 4;
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;                                   // leading byte offset: not used by swizzled K-major operands
    d |= (uint64_t)((8u * span) >> 4) << 32;                  // stride between groups of 8 rows
    d |= 1ull << 46;
    d |= (uint64_t)(span == 128 ? 2 : 4) << 61;               // 128-byte / 64-byte swizzle
    return d;
}
__host__ __device__ inline uint32_t idesc_tf32(int M, int N) {
    return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
// byte offset of logical 16-byte chunk q of row r inside a swizzled tile
template <int D>
__device__ __forceinline__ uint32_t swz_off(int r, int q) {
    if (D == 32) return (uint32_t)r * 128u + (uint32_t)((q ^ (r & 7)) << 4);
    return (uint32_t)r * 64u + (uint32_t)((q ^ ((r >> 1) & 3)) << 4);
}
__device__ __forceinline__ void tmem_ld32_nowait(uint32_t taddr, uint32_t (&r)[32]) {
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
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld16_nowait(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
// The search cannot separate the best candidates of some point of this warp (redo: of this thread's point).  The true
// nearest centroid's score is within tau of the best score (each score is within tau / 2 of its exact value), so the
// exact form sum_d (x - c)^2 decides among the columns with v <= lim = best + tau alone.  The scores are read once more
// (all lanes: the read is warp-wide) and every thread notes its candidates, up to four column numbers packed in a word;
// then each thread works through its own list - no thread waits for another's columns.  Candidates are taken in
// ascending order with strict <, so the lowest index wins an exact tie as it does over all centroids; a point with
// more than four candidates is decided over all centroids.
template <int D>
__device__ __noinline__ int redecide(bool redo, int kb, float lim, const float* __restrict__ xrow, uint32_t col0, int npad,
                                     const float* __restrict__ centroids, int K) {
    constexpr int Q = D / 4;
    uint32_t cand = 0;
    int cnt = 0;
    for (int ch = 0; ch < npad / 16; ++ch) {
        uint32_t vv[16];
        tmem_ld16_nowait(col0 + (uint32_t)(ch * 16), vv);
        tmem_ld_wait();
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            const bool in = __uint_as_float(vv[e]) <= lim && ch * 16 + e < K;
            cand = in ? (cand << 8) | (uint32_t)(ch * 16 + e) : cand;     // (column numbers are below 128)
            cnt += in ? 1 : 0;
        }
    }
    if (!redo) return kb;
    float x[D];                                          // the point, from global memory (its stage went back after the search)
#pragma unroll
    for (int q = 0; q < Q; ++q) {
        const float4 v = __ldg(reinterpret_cast<const float4*>(xrow) + q);
        x[4 * q] = v.x; x[4 * q + 1] = v.y; x[4 * q + 2] = v.z; x[4 * q + 3] = v.w;
    }
    if (cnt > 4 || cnt == 0) return tc::exact_argmin_global<D>(x, centroids, K);
    float best = __int_as_float(0x7f800000);
    for (int s = cnt - 1; s >= 0; --s) {                 // the first candidate noted sits highest in the word
        const int k = (int)((cand >> (8 * s)) & 0xFFu);
        const float4* c = reinterpret_cast<const float4*>(centroids + (size_t)k * D);
        float d0 = 0.0f;
#pragma unroll
        for (int q = 0; q < Q; ++q) {
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
__global__ void __launch_bounds__(MAX_THREADS, 1)
ws_fused_kernel(const __grid_constant__ CUtensorMap pmap, const float* __restrict__ points, const float* __restrict__ xnorm,
                size_t N, int P, int C,
                const float* __restrict__ centroids, int K, int32_t* __restrict__ labels, float* __restrict__ scratch,
                uint32_t* __restrict__ status, uint32_t* __restrict__ dirty, float2* __restrict__ bounds,
                const float* __restrict__ drift, const uint32_t* __restrict__ need, int need_words) {
    grid_dependency_wait();                                 // (a no-op unless launched as a programmatic dependent)
    constexpr int KCH = D / 8;                              // 16-byte bf16 chunks (8 coordinates) per point
    constexpr int Q = D / 4;                                // 16-byte fp32 chunks per point
    constexpr uint32_t XC = xchunk_of(D);
    static_assert(D == 16 || D == 32, "a row is one 64- or 128-byte swizzle span");
    extern __shared__ unsigned char ws_smem_raw[];
    const Plan pl = plan_of(D, K, PARTIALS, DELTA);
    const int SLOTS = pl.slots;
    const int npad = npad_of(K);
    const int G = pl.groups, NST = pl.stages, A = pl.accs;
    unsigned char* sm = ws_smem_raw + ((1024u - (smem_u32(ws_smem_raw) & 1023u)) & 1023u);
    const uint32_t sm_u = smem_u32(sm);
    float* s_cn = reinterpret_cast<float*>(sm + pl.cn);
    float* s_drift = reinterpret_cast<float*>(sm + pl.drift);
    uint32_t* s_need = reinterpret_cast<uint32_t*>(sm + pl.need);
    TileDesc* s_desc = reinterpret_cast<TileDesc*>(sm + pl.desc);
    // control words: [0..3] what a group says about its tile (CTRL_*), [4..5] run had sums, [6] tensor-memory address,
    // [7] abort, [25] runs whose end the sums issuer has
    // signalled, [26] tiles it is through with, [28..31] sums GEMMs issued from each slot, [32 + 4 slot + w] rows of warp w
    // of the slot's last user have one-hot entries set
    volatile int* s_ctrl = reinterpret_cast<volatile int*>(sm + pl.ctrl);
    volatile int* s_abort = s_ctrl + 7;
    constexpr int CTRL_SUMS = 1, CTRL_LAST = 2, CTRL_END = 8;
    // barriers (8 bytes each)
    const uint32_t bar0 = sm_u + pl.bar;
    auto B_full = [&](int s) { return bar0 + 8u * (uint32_t)s; };
    auto B_empty = [&](int s) { return bar0 + 8u * (uint32_t)(MAX_STAGES + s); };
    auto B_accfull = [&](int a) { return bar0 + 8u * (uint32_t)(2 * MAX_STAGES + a); };
    auto B_accempty = [&](int a) { return bar0 + 8u * (uint32_t)(2 * MAX_STAGES + MAX_ACCS + a); };
    constexpr int BAR_GROUPS = 2 * MAX_STAGES + 2 * MAX_ACCS;     // index of the first per-group barrier
    auto B_decided = [&](int g) { return bar0 + 8u * (uint32_t)(BAR_GROUPS + g); };
    auto B_tiledone = [&](int g) { return bar0 + 8u * (uint32_t)(BAR_GROUPS + MAX_GROUPS + g); };
    auto B_rundone = [&](int p) { return bar0 + 8u * (uint32_t)(BAR_GROUPS + 2 * MAX_GROUPS + p); };
    auto B_drained = [&](int p) { return bar0 + 8u * (uint32_t)(BAR_GROUPS + 2 * MAX_GROUPS + 2 + p); };
    auto B_slotfree = [&](int sl) { return bar0 + 8u * (uint32_t)(BAR_GROUPS + 2 * MAX_GROUPS + 4 + sl); };   // (MAX_SLOTS of them: 48 barriers in all)

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nthreads = (4 * G + 4) * 32;
    if (tid >= nthreads) return;                             // (the launch uses exactly nthreads; kept for safety)
    const int runs = P * C;
    const bool skipping = DELTA && PARTIALS && BOUNDS && need != nullptr;
    if (skipping) {
        if (reinterpret_cast<const uint32_t*>(drift)[K + 1] == 0u) return;   // no tile anywhere: the check has settled every run
        bool any = false;
        for (int run = blockIdx.x; run < runs; run += gridDim.x)
            for (int q = tid; q < need_words; q += nthreads) any = any || need[(size_t)run * need_words + q] != 0u;
        if (!__syncthreads_or(any ? 1 : 0)) {
            for (int run = blockIdx.x + tid * gridDim.x; run < runs; run += nthreads * gridDim.x) dirty[run] = 0u;
            return;
        }
    }
    // ---- set-up, all threads ------------------------------------------------------------------------------------
    if (warp == 4 * G + 1) tmem_alloc(smem_u32(const_cast<int*>(s_ctrl + 6)), pl.tmem_cols);
    if (tid == 0) {
        for (int s = 0; s < NST; ++s) { mbar_init(B_full(s), 1); mbar_init(B_empty(s), 5); }   // empty: the search's commit + the four warps that read the descriptor
        for (int a = 0; a < A; ++a) { mbar_init(B_accfull(a), 1); mbar_init(B_accempty(a), 4); }
        for (int g = 0; g < G; ++g) mbar_init(B_decided(g), 4);
        for (int g = 0; g < G; ++g) mbar_init(B_tiledone(g), 1);
        for (int sl = 0; sl < MAX_SLOTS; ++sl) mbar_init(B_slotfree(sl), 1);
        s_ctrl[0] = 0; s_ctrl[1] = 0; s_ctrl[2] = 0; s_ctrl[3] = 0;
        s_ctrl[25] = 0; s_ctrl[26] = 0; s_ctrl[28] = 0; s_ctrl[29] = 0; s_ctrl[30] = 0; s_ctrl[31] = 0;
        for (int q = 32; q < 48; ++q) s_ctrl[q] = 0;
        for (int p = 0; p < 2; ++p) { mbar_init(B_rundone(p), 1); mbar_init(B_drained(p), 4); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        *s_abort = 0;
    }
    for (int k = tid; k < npad; k += nthreads) {
        float s = 3.0e38f;
        if (k < K) {
            s = 0.0f;
            for (int d = 0; d < D; ++d) s = fmaf(centroids[(size_t)k * D + d], centroids[(size_t)k * D + d], s);
        }
        s_cn[k] = s;
        // |c|^2 as three numbers of 11 significant bits each: exact, and exact in tf32 whether it rounds or truncates
        const float hi = __uint_as_float(__float_as_uint(s) & 0xFFFFE000u);
        const float r1 = s - hi;
        const float mid = __uint_as_float(__float_as_uint(r1) & 0xFFFFE000u);
        const float lo = r1 - mid;
        *reinterpret_cast<float4*>(sm + pl.cnb + (size_t)k * 16) = make_float4(hi, mid, lo, 0.0f);
        *reinterpret_cast<float4*>(sm + pl.cnb + (size_t)npad * 16 + (size_t)k * 16) = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        if (PARTIALS && BOUNDS) s_drift[k] = k < K ? drift[k] : 0.0f;
    }
    for (int i = tid; i < npad * Q; i += nthreads) {          // -2 c rounded to 11 significant bits (nearest, ties away)
        const int n = i / Q, q = i - n * Q;
        float v[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float c = n < K ? -2.0f * centroids[(size_t)n * D + q * 4 + e] : 0.0f;
            v[e] = __uint_as_float((__float_as_uint(c) + 0x1000u) & 0xFFFFE000u);
        }
        *reinterpret_cast<float4*>(sm + pl.b + swz_off<D>(n, q)) = make_float4(v[0], v[1], v[2], v[3]);
    }
    for (int r = tid; r < TILE; r += nthreads) {
        *reinterpret_cast<float4*>(sm + pl.ones + (size_t)r * 16) = make_float4(1.0f, 1.0f, 1.0f, 0.0f);
        *reinterpret_cast<float4*>(sm + pl.ones + 2048 + (size_t)r * 16) = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
    }
    if (PARTIALS) {
        for (int i = tid; i < (int)(SLOTS * pl.slot_bytes / 16); i += nthreads)
            *reinterpret_cast<uint4*>(sm + pl.slot + (size_t)i * 16) = make_uint4(0u, 0u, 0u, 0u);
        for (int i = tid; i < SLOTS * TILE; i += nthreads) reinterpret_cast<uint16_t*>(sm + pl.prev)[i] = 0xFFFFu;
        __syncthreads();                                     // (other threads' zeros must not land on top of the ones)
        for (int s = 0; s < SLOTS; ++s)                      // the ones column of a slot: [1, 1, 0, ...] for every point
            for (int r = tid; r < TILE; r += nthreads)
                *reinterpret_cast<uint4*>(sm + pl.slot + (size_t)s * pl.slot_bytes + (size_t)(2 * KCH) * XC + (size_t)r * 16) = make_uint4(0x3F803F80u, 0u, 0u, 0u);
    }
    fence_async_smem();
    fence_before_sync();
    __syncthreads();
    fence_after_sync();
    const uint32_t tmem_base = (uint32_t)s_ctrl[6];
    const uint32_t sums_col0 = (uint32_t)(A * npad);
    bool ok = true;                                           // this thread has seen no wait give up

    if (warp == 4 * G) {
        // ---- producer ---------------------------------------------------------------------------------------------
        // (all lanes walk the runs: they fetch the run's tile marks together; lane 0 does the rest)
        int i = 0, run_seq = 0;
        for (int run = blockIdx.x; run < runs; run += gridDim.x) {
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
            if (skipping) {
                __syncwarp();
                for (int q = lane; q < need_words; q += 32) s_need[q] = need[(size_t)run * need_words + q];
                __syncwarp();
            }
            if (lane != 0) continue;
            const int r = run / C, c = run - r * C;
            const size_t j0 = (size_t)r * N / P, j1 = (size_t)(r + 1) * N / P;
            const size_t len = j1 - j0;
            const size_t b0 = j0 + len * c / C, b1 = j0 + len * (c + 1) / C;
            const size_t ntiles = (b1 - b0 + TILE - 1) / TILE;
            size_t t = 0;                                    // first tile that has to be searched
            if (skipping) while (t < ntiles && s_need[t] == 0u) ++t;
            if (t >= ntiles) {                               // nothing to do in this run
                if (PARTIALS && DELTA) dirty[run] = 0u;
                else if (PARTIALS) for (int q = 0; q < K * (D + 4); ++q) scratch[(size_t)run * K * (D + 4) + q] = 0.0f;   // an empty run
                continue;
            }
            while (t < ntiles) {
                size_t tn = t + 1;
                if (skipping) while (tn < ntiles && s_need[tn] == 0u) ++tn;
                const int s = i % NST, use = i / NST;
                if (use > 0 && !wait_or_abort(B_empty(s), (uint32_t)(use - 1) & 1u, s_abort, 1)) { ok = false; break; }
                TileDesc d;
                d.base = b0 + t * TILE; d.end = b1; d.run = run; d.run_seq = run_seq; d.last = tn >= ntiles ? 1 : 0; d.pad = i;
                s_desc[s] = d;
                mbar_expect_tx(B_full(s), pl.stage_bytes);
                tma_tile_2d(sm_u + pl.stage + (uint32_t)s * pl.stage_bytes, &pmap, 0, (int)(b0 + t * TILE), B_full(s));
                ++i;
                t = tn;
            }
            ++run_seq;
        }
        if (lane == 0) {
            for (int e = 0; e < G && ok; ++e) {               // end markers: one for every epilogue group
                const int s = i % NST, use = i / NST;
                if (use > 0 && !wait_or_abort(B_empty(s), (uint32_t)(use - 1) & 1u, s_abort, 1)) { ok = false; break; }
                TileDesc d;
                d.base = 0; d.end = 0; d.run = -1; d.run_seq = e; d.last = 0; d.pad = i;
                s_desc[s] = d;
                mbar_arrive(B_full(s));
                ++i;
            }
            if (!ok) {                                        // copies still in flight must land before the block may go
                for (int back = 1; back <= NST && back <= i; ++back) {
                    const int ii = i - back;
                    for (uint32_t it = 0; it < WAIT_LIMIT; ++it)
                        if (mbar_try_wait(B_full(ii % NST), (uint32_t)(ii / NST) & 1u)) break;
                }
            }
        }
    } else if (warp == 4 * G + 1 || warp == 4 * G + 3) {
        // ---- search issuers --------------------------------------------------------------------------------------------
        // Two of them, one for the even tiles and one for the odd ones: a thread gets a small MMA issued every 72 cycles
        // at best, the tensor core takes one every 48, and five per tile from one thread alone were what the epilogue
        // groups waited for (assignment of N = 2^22, D = 32, K = 64: 1400 of a group's 3250 cycles per tile).
        if (lane == 0) {
            // Everything that does not change from tile to tile is made once: this one thread's instruction stream is
            // what every tile waits for.  A descriptor's address field counts 16-byte units, so a step of 32 bytes adds 2
            // and the next stage adds stage_bytes / 16.
            const uint32_t idesc = idesc_tf32(TILE, npad);
            uint64_t bdesc[D / 8];
#pragma unroll
            for (int ks = 0; ks < D / 8; ++ks) bdesc[ks] = swz_desc<D>(sm_u + pl.b + ks * 32);
            const uint64_t adesc0 = swz_desc<D>(sm_u + pl.stage);
            const uint64_t ones_desc = smem_desc(sm_u + pl.ones, 2048, 128), cnb_desc = smem_desc(sm_u + pl.cnb, (uint32_t)npad * 16, 128);
            const uint32_t stage_units = pl.stage_bytes >> 4;
            // tile i = first, first + step, ...: stage i mod stages on its laps-th use, accumulator i mod accs on its lapa-th.
            // Both take part only when the numbers of stages and of accumulators are even: a stage and an accumulator then
            // always meet the same issuer, which sees every phase of their barriers - an issuer that skipped a phase (the
            // other one's) could find the barrier two phases back and take its parity for "done".
            const int step = (NST % 2 == 0 && A % 2 == 0) ? 2 : 1;
            const int first = warp == 4 * G + 1 ? 0 : 1;
            int s = first % NST, a = first % A;
            uint32_t laps = (uint32_t)(first / NST), lapa = (uint32_t)(first / A);
            for (; first < step;) {
                if (!wait_or_abort(B_full(s), laps & 1u, s_abort, 3)) { ok = false; break; }
                if (s_desc[s].run < 0) break;
                if (lapa > 0 && !wait_or_abort(B_accempty(a), (lapa - 1u) & 1u, s_abort, 4)) { ok = false; break; }
                fence_after_sync();
                const uint32_t acc = tmem_base + (uint32_t)(a * npad);
                const uint64_t adesc = adesc0 + (uint64_t)((uint32_t)s * stage_units);
#pragma unroll
                for (int ks = 0; ks < D / 8; ++ks)             // 8 coordinates (32 bytes) per step
                    mma_tf32(acc, adesc + (uint64_t)(2 * ks), bdesc[ks], idesc, ks > 0 ? 1u : 0u);
                mma_tf32(acc, ones_desc, cnb_desc, idesc, 1u);
                mma_commit(B_accfull(a));
                mma_commit(B_empty(s));                        // the tile has been read: its stage goes back to the producer
                s += step;
                while (s >= NST) { s -= NST; ++laps; }
                a += step;
                while (a >= A) { a -= A; ++lapa; }
            }
        }
    } else if (warp == 4 * G + 2) {
        // ---- sums issuer -----------------------------------------------------------------------------------------------
        if (PARTIALS && lane == 0) {
            const uint32_t idesc = tc::instr_desc(TILE, npad, true);
            const uint64_t xdesc0 = smem_desc(sm_u + pl.slot, 128, XC), odesc0 = smem_desc(sm_u + pl.slot + pl.oh_off, 128, OCHUNK);
            const uint32_t slot_units = pl.slot_bytes >> 4;
            bool started = false, run_checked = false;
            int nruns[2] = {0, 0};                            // runs finished on each accumulator so far
            int slot = 0;
            int g = 0;
            uint32_t dec_par = 0;
            for (int i = 0;; ++i) {
                if (!wait_or_abort(B_decided(g), dec_par, s_abort, 5 | (i << 8))) { ok = false; break; }
                const int ctrl = atomicExch(const_cast<int*>(s_ctrl + g), 0);   // taken and cleared: the warps or their flags in
                mbar_arrive(B_tiledone(g));                    // the group's control word may be written again
                if (ctrl & CTRL_END) break;
                const int par = (nruns[0] + nruns[1]) & 1, last = ctrl & CTRL_LAST;   // runs alternate between the two accumulators
                if (!run_checked && (ctrl & (CTRL_SUMS | CTRL_LAST))) {
                    // the run before last used this accumulator and this "had sums" word: its last tile's group must be
                    // through with both (it says so after writing the sums out, or after seeing that there were none)
                    if (nruns[par] > 0 && !wait_or_abort(B_drained(par), (uint32_t)(nruns[par] - 1) & 1u, s_abort, 6)) { ok = false; break; }
                    run_checked = true;
                }
                if (ctrl & CTRL_SUMS) {
                    fence_after_sync();
                    const uint32_t acc = tmem_base + sums_col0 + (uint32_t)(par * npad);
                    const uint64_t xd = xdesc0 + (uint64_t)((uint32_t)slot * slot_units), od = odesc0 + (uint64_t)((uint32_t)slot * slot_units);
#pragma unroll
                    for (int ks = 0; ks < TILE / 16; ++ks)     // 16 points (256 bytes) per step, both operands MN-major
                        tc::mma_bf16(acc, xd + (uint64_t)(16 * ks), od + (uint64_t)(16 * ks), idesc, (started || ks > 0) ? 1u : 0u);
                    started = true;
                    mma_commit(B_slotfree(slot));
                    s_ctrl[28 + slot] = s_ctrl[28 + slot] + 1;
                }
                __threadfence_block();
                s_ctrl[26] = i + 1;                            // through with tile i (its sums GEMM, if any, is on its way)
                if (last) {
                    s_ctrl[4 + par] = started ? 1 : 0;
                    __threadfence_block();
                    if (started) mma_commit(B_rundone(par));
                    else mbar_arrive(B_rundone(par));
                    ++nruns[par];
                    s_ctrl[25] = nruns[0] + nruns[1];          // runs whose end has been signalled
                    started = false;
                    run_checked = false;
                }
                if (++g == G) { g = 0; dec_par ^= 1u; }
                if (++slot == SLOTS) slot = 0;
            }
        }
    } else {
        // ---- epilogue groups ------------------------------------------------------------------------------------------
        const int g = warp >> 2, t = tid & 127;              // t: this thread's point of the tile = row of the accumulator
        const uint32_t lane_base = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
        const int stride = D + 4;
        float cmax = 0.0f;
        for (int k = 0; k < K; ++k) cmax = fmaxf(cmax, s_cn[k]);
        const float drift_max = (PARTIALS && BOUNDS) ? drift[K] : 0.0f;
        uint32_t tag_mask;                                    // 0xFFFFFF80, kept in a register (see best_two_of_16)
        asm volatile("mov.u32 %0, 0xFFFFFF80;" : "=r"(tag_mask));
        // One lane per warp arrives for its warp (the barriers of the groups count warps, not threads): 32 times fewer
        // barrier operations; all lanes wait (the same instruction count as one lane waiting, without the divergence).
        auto wwait = [&](uint32_t bar, uint32_t par, int where) -> bool {
            return __all_sync(0xffffffffu, wait_or_abort(bar, par, s_abort, where)) != 0;   // (all lanes: one instruction either way, no divergence)
        };
        auto warrive = [&](uint32_t bar) {
            __syncwarp();
            if (lane == 0) mbar_arrive(bar);
        };
        // tile i = g, g + G, ...: stage s = i mod stages on its lap-th use, this group's n-th tile, slot i mod 2
        int s = g % NST, n = 0;
        uint32_t lap = (uint32_t)(g / NST);
        int slot = PARTIALS ? g % SLOTS : 0;
        const bool own_slot = PARTIALS && DELTA && SLOTS == G;   // slot g belongs to group g alone
        bool my_stale = false;                                // own_slot: this warp's rows of the slot have one-hot entries set
        int a = g % A;                                        // the tile's search accumulator, on its lapa-th use
        uint32_t lapa = (uint32_t)(g / A);
        for (int i = g; ok; i += G, ++n) {
            if (n > 0) {
                s += G;
                while (s >= NST) { s -= NST; ++lap; }
                a += G;
                while (a >= A) { a -= A; ++lapa; }
                if (PARTIALS) {
                    slot += G;
                    while (slot >= SLOTS) slot -= SLOTS;
                }
            }
            if (!wwait(B_full(s), lap & 1u, 3)) { ok = false; break; }
            TileDesc td = s_desc[s];
            // When the stages do not divide evenly among the groups, the stage's previous tile was another group's and this
            // group has not seen that phase of the barrier: had that phase not been over yet, the parity asked for above
            // would have been taken for done two phases early.  The descriptor tells: the producer writes this tile's only
            // after the previous tile has been released, i.e. after that phase.  (Never seen to happen; one compare.)
            if (td.pad != i) {
                const long long t0 = clock64();
                while (reinterpret_cast<volatile TileDesc*>(s_desc)[s].pad != i) {
                    if (*s_abort != 0 || clock64() - t0 > 4000000000LL) { if (*s_abort == 0) *s_abort = 2; ok = false; break; }
                }
                if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
                if (!wwait(B_full(s), lap & 1u, 3)) { ok = false; break; }
                td = s_desc[s];
            }
            if (td.run < 0) {                                // no more tiles: the sums issuer hears it from the first group that does
                if (PARTIALS && td.run_seq == 0) {          // (the first of the G end markers)
                    if (n > 0 && !wwait(B_tiledone(g), (uint32_t)(n - 1) & 1u, 12 | (i << 8))) { ok = false; break; }
                    if (t == 0) atomicOr(const_cast<int*>(s_ctrl + g), CTRL_END);
                    warrive(B_decided(g));
                }
                break;
            }
            const size_t j = (size_t)td.base + (size_t)t;
            const bool live = j < (size_t)td.end;
            // The groups take turns on the slots.  Once the sums issuer is through with tile i - SLOTS (the slot's last possible
            // user before this tile) the slot's book-keeping is final: whether the rows of this warp's position still have
            // one-hot entries set (they must be cleared before the slot's next GEMM), and how many GEMMs were issued from
            // the slot, which says which phase of its barrier to wait for before the operands may be touched - at most one
            // phase back, because every user waits for its predecessor.
            int info = 0;                                        // bit 0: stale rows, bits 1..: GEMMs issued from the slot
            auto slot_info = [&]() -> bool {
                // the sums issuer must have taken what the group said about its previous tile
                if (n > 0 && !wwait(B_tiledone(g), (uint32_t)(n - 1) & 1u, 10 | (i << 8))) return false;
                if (lane == 0 && i >= SLOTS) {
                    const long long t0 = clock64();
                    while (s_ctrl[26] < i - SLOTS + 1) {
                        if (*s_abort != 0 || clock64() - t0 > 4000000000LL) { if (*s_abort == 0) *s_abort = 14; info = -1; break; }
                    }
                    if (info == 0) info = (s_ctrl[32 + 4 * slot + (warp & 3)] != 0 ? 1 : 0) | (s_ctrl[28 + slot] << 1);
                }
                info = __shfl_sync(0xffffffffu, info, 0);
                return info >= 0;
            };
            // A group that has its slot to itself (own_slot) keeps "my rows still have one-hot entries set" in a register and
            // asks for the slot's GEMM count only when it is about to touch the slot: it then waits until the issuer is through
            // the group's previous tile (the count is final) by reading the issuer's counter.
            auto own_info = [&]() -> bool {
                if (lane == 0) {
                    if (i >= G) {
                        const long long t0 = clock64();
                        while (s_ctrl[26] < i - G + 1) {
                            if (*s_abort != 0 || clock64() - t0 > 4000000000LL) { if (*s_abort == 0) *s_abort = 14; info = -1; break; }
                        }
                    }
                    if (info == 0) info = s_ctrl[28 + slot] << 1;
                }
                info = __shfl_sync(0xffffffffu, info, 0);
                return info >= 0;
            };
            if (PARTIALS && !DELTA) {
                // All points are summed: the operand rows do not depend on the labels, so they are made now, out of the staged
                // tile, while the search's MMAs run - bf16 high and low parts of the row (low = bf16(x - high)): chunk column
                // 2 kc resp. 2 kc + 1 of the slot.
                if (!slot_info()) { ok = false; break; }
                const int uses = info >> 1;
                if (uses > 0 && !wwait(B_slotfree(slot), (uint32_t)(uses - 1) & 1u, 7)) { ok = false; break; }
                if (live) {
                    const unsigned char* row = sm + pl.stage + (size_t)s * pl.stage_bytes;
                    unsigned char* xs = sm + pl.slot + (size_t)slot * pl.slot_bytes;
#pragma unroll
                    for (int kc = 0; kc < KCH; ++kc) {
                        const float4 va = *reinterpret_cast<const float4*>(row + swz_off<D>(t, 2 * kc));
                        const float4 vb = *reinterpret_cast<const float4*>(row + swz_off<D>(t, 2 * kc + 1));
                        const float v[8] = {va.x, va.y, va.z, va.w, vb.x, vb.y, vb.z, vb.w};
                        uint32_t hw[4], lw[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            hw[e] = pack_bf16(v[2 * e], v[2 * e + 1]);
                            const float ah = __uint_as_float(hw[e] << 16), bh = __uint_as_float(hw[e] & 0xFFFF0000u);
                            lw[e] = pack_bf16(v[2 * e] - ah, v[2 * e + 1] - bh);
                        }
                        *reinterpret_cast<uint4*>(xs + (size_t)(2 * kc) * XC + (size_t)t * 16) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
                        *reinterpret_cast<uint4*>(xs + (size_t)(2 * kc + 1) * XC + (size_t)t * 16) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
                    }
                }
            }
            // The stage goes back to the producer once the search has read the tile (the issuer's commit) and this group's
            // four warps are through with it (here): the descriptor taken and, when all points are summed, the rows converted.
            warrive(B_empty(s));
            const int old = (DELTA && live) ? labels[j] : -1;
            const float xn = live ? __ldg(xnorm + j) : 0.0f;      // |x|^2, made once per context: the staged tile is the tensor core's alone
            if (!wwait(B_accfull(a), lapa & 1u, 8)) { ok = false; break; }
            fence_after_sync();
            float m1 = __int_as_float(0x7f800000), m2 = m1;
            {
                // 16 columns at a time, the next 16 on their way while these are looked at (npad / 16 is even)
                const uint32_t col0 = lane_base + (uint32_t)(a * npad);
                uint32_t va[16], vb[16];
                tmem_ld16_nowait(col0, va);
                for (int ch = 0; ch < npad / 16; ch += 2) {
                    float c1, c2;
                    tmem_ld_wait();
                    tmem_ld16_nowait(col0 + (uint32_t)(ch * 16 + 16), vb);
                    best_two_of_16(va, tag_mask, c1, c2);    // tags 0..15; bits 4-6 (zero so far) take the chunk number
                    c1 = __uint_as_float(__float_as_uint(c1) | (uint32_t)(ch << 4));
                    m2 = min3(m2, c2, fmaxf(m1, c1));
                    m1 = fminf(m1, c1);
                    tmem_ld_wait();
                    if (ch + 2 < npad / 16) tmem_ld16_nowait(col0 + (uint32_t)(ch * 16 + 32), va);
                    best_two_of_16(vb, tag_mask, c1, c2);
                    c1 = __uint_as_float(__float_as_uint(c1) | (uint32_t)((ch + 1) << 4));
                    m2 = min3(m2, c2, fmaxf(m1, c1));
                    m1 = fminf(m1, c1);
                }
            }
            int kb = (int)(__float_as_uint(m1) & 127u);
            const float tau = TAU_SCALE * (xn + cmax);
            const bool redo = live && !(m2 - m1 > tau);
            if (__any_sync(0xffffffffu, redo))            // rare on separated data: kept out of line, away from this loop's registers
                kb = redecide<D>(redo, kb, m1 + tau, points + j * D, lane_base + (uint32_t)(a * npad), npad, centroids, K);
            fence_before_sync();
            warrive(B_accempty(a));                      // the accumulator may take another tile
            const bool changed = live && !(DELTA && old == kb);
            if (changed) labels[j] = kb;
            if (PARTIALS && BOUNDS && live) {
                float2 w = make_float2(__int_as_float(0x7f800000), 0.0f);      // decided by the exact form: searched again next time
                if (!redo) {
                    // |x - c|^2 = |x|^2 + v; the search knows v to within tau (tags included)
                    const float u = __fsqrt_ru(fmaxf(__fadd_ru(__fadd_ru(xn, m1), tau), 0.0f));
                    const float l = __fsqrt_rd(fmaxf(__fsub_rd(__fadd_rd(xn, m2), tau), 0.0f));
                    w = make_float2(__fsub_ru(u, s_drift[kb]), __fadd_rd(l, drift_max));
                }
                bounds[j] = w;
            }
            if (PARTIALS) {
                // Every warp goes its own way: no meeting of the group's four warps.  A warp tells the sums issuer whether one
                // of its points changed the sums (flags or-ed into the group's control word, which the issuer takes and
                // clears); only a thread whose label changed converts its row and sets its one-hot row - the other rows of
                // the slot keep whatever finite numbers they hold, against one-hot rows that are zero.
                const bool any_w = __any_sync(0xffffffffu, changed);
                bool stale;
                if (own_slot) {
                    stale = my_stale;
                    // The sums issuer must have taken what the group said about its previous tile: the control word is free again,
                    // and the issuer is never more than one phase behind on the barrier the warps arrive on below.
                    if (n > 0 && !wwait(B_tiledone(g), (uint32_t)(n - 1) & 1u, 10 | (i << 8))) { ok = false; break; }
                    if ((any_w || stale) && !own_info()) { ok = false; break; }
                } else {
                    if (DELTA && !slot_info()) { ok = false; break; }
                    stale = (info & 1) != 0;
                }
                if (any_w || stale) {
                    const int uses = info >> 1;
                    if (DELTA && uses > 0 && !wwait(B_slotfree(slot), (uint32_t)(uses - 1) & 1u, 7)) { ok = false; break; }
                    unsigned char* xs = sm + pl.slot + (size_t)slot * pl.slot_bytes;
                    unsigned char* oh = xs + pl.oh_off;
                    uint16_t* prev = reinterpret_cast<uint16_t*>(sm + pl.prev) + slot * TILE + t;
                    const uint16_t pv = *prev;
                    if ((pv & 0xFFu) != 0xFFu) *reinterpret_cast<uint4*>(oh + (size_t)(pv & 0xFFu) * OCHUNK + (size_t)t * 16) = make_uint4(0u, 0u, 0u, 0u);
                    if ((pv >> 8) != 0xFFu) *reinterpret_cast<uint4*>(oh + (size_t)(pv >> 8) * OCHUNK + (size_t)t * 16) = make_uint4(0u, 0u, 0u, 0u);
                    uint16_t nv = 0xFFFFu;
                    if (changed) {
                        // one-hot row of this point: 16-byte chunk kb/8, bf16 1.0 at position kb%8 (and -1.0 for the label it leaves)
                        uint4 wv = tc::onehot_chunk(kb, 0x3F80u);
                        const int ck = kb >> 3;
                        if (old >= 0 && (old >> 3) == ck) wv = tc::or4(wv, tc::onehot_chunk(old, 0xBF80u));
                        *reinterpret_cast<uint4*>(oh + (size_t)ck * OCHUNK + (size_t)t * 16) = wv;
                        nv = (uint16_t)(0xFF00u | (uint32_t)ck);
                        if (old >= 0 && (old >> 3) != ck) {
                            *reinterpret_cast<uint4*>(oh + (size_t)(old >> 3) * OCHUNK + (size_t)t * 16) = tc::onehot_chunk(old, 0xBF80u);
                            nv = (uint16_t)(((uint32_t)(old >> 3) << 8) | (uint32_t)ck);
                        }
                        // bf16 high and low parts of the row (low = bf16(x - high)): chunk column 2 kc resp. 2 kc + 1
#pragma unroll
                        for (int kc = 0; DELTA && kc < KCH; ++kc) {
                            const float4 va = __ldg(reinterpret_cast<const float4*>(points + j * D) + 2 * kc);   // (from L2: the tile was just read)
                            const float4 vb = __ldg(reinterpret_cast<const float4*>(points + j * D) + 2 * kc + 1);
                            const float v[8] = {va.x, va.y, va.z, va.w, vb.x, vb.y, vb.z, vb.w};
                            uint32_t hw[4], lw[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                hw[e] = pack_bf16(v[2 * e], v[2 * e + 1]);
                                const float ah = __uint_as_float(hw[e] << 16), bh = __uint_as_float(hw[e] & 0xFFFF0000u);
                                lw[e] = pack_bf16(v[2 * e] - ah, v[2 * e + 1] - bh);
                            }
                            *reinterpret_cast<uint4*>(xs + (size_t)(2 * kc) * XC + (size_t)t * 16) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
                            *reinterpret_cast<uint4*>(xs + (size_t)(2 * kc + 1) * XC + (size_t)t * 16) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
                        }
                    }
                    *prev = nv;
                    my_stale = any_w;
                    if (lane == 0) s_ctrl[32 + 4 * slot + (warp & 3)] = any_w ? 1 : 0;
                    fence_async_smem();                      // the tensor core reads shared memory through the async proxy
                }
                if (lane == 0) {
                    const int flags = (any_w ? CTRL_SUMS : 0) | (((warp & 3) == 0 && td.last) ? CTRL_LAST : 0);
                    if (flags) atomicOr(const_cast<int*>(s_ctrl + g), flags);
                }
                fence_before_sync();
                warrive(B_decided(g));
            }
            if (PARTIALS && td.last) {
                // the run's last tile: its group writes the run's sums out once the sums issuer is through the run
                // (first until the sums issuer has signalled the end of this run: it has then seen the run before last written
                // out, so the barrier is at most one phase behind this wait - different runs' ends are waited for by
                // different groups, none of which sees every phase)
                const int par = td.run_seq & 1;
                {
                    const long long t0 = clock64();
                    while (s_ctrl[25] <= td.run_seq) {
                        if (*s_abort != 0 || clock64() - t0 > 4000000000LL) { if (*s_abort == 0) *s_abort = 13; ok = false; break; }
                    }
                    if (!ok) break;
                }
                if (!wwait(B_rundone(par), (uint32_t)(td.run_seq >> 1) & 1u, 11)) { ok = false; break; }
                fence_after_sync();
                const bool had_sums = s_ctrl[4 + par] != 0;
                float* row_block = scratch + (size_t)td.run * (size_t)K * stride;
                if (had_sums) {
                    // Accumulator rows: 16 (d / 8) + d % 8 holds the high-part sums of coordinate d, 8 rows further on the
                    // low-part sums (same warp, 8 lanes up), row 2 D the counts.  Columns are the centroids.
                    const int d_of = (t >> 4) * 8 + (t & 7);
                    const bool is_hi = (t & 8) == 0 && t < 2 * D, is_cnt = t == 2 * D;
                    for (int ch = 0; ch < npad / 32; ++ch) {
                        uint32_t v[32];
                        tmem_ld32_nowait(lane_base + sums_col0 + (uint32_t)(par * npad + ch * 32), v);
                        tmem_ld_wait();
#pragma unroll
                        for (int e = 0; e < 32; ++e) {
                            const float lo = __shfl_down_sync(0xffffffffu, __uint_as_float(v[e]), 8);
                            const int k = ch * 32 + e;
                            if (k < K) {
                                if (is_hi) row_block[(size_t)k * stride + d_of] = __fadd_rn(__uint_as_float(v[e]), lo);
                                if (is_cnt) {
                                    row_block[(size_t)k * stride + D] = __uint_as_float(v[e]);
                                    row_block[(size_t)k * stride + D + 1] = 0.0f;
                                    row_block[(size_t)k * stride + D + 2] = 0.0f;
                                    row_block[(size_t)k * stride + D + 3] = 0.0f;
                                }
                            }
                        }
                    }
                    fence_before_sync();
                } else if (!DELTA) {
                    for (int q = t; q < K * stride; q += TILE) row_block[q] = 0.0f;
                }
                warrive(B_drained(par));                 // the accumulator and the "had sums" word may serve another run
                if (DELTA && t == 0) dirty[td.run] = had_sums ? 1u : 0u;
            }
        }
    }
    if (!ok && *s_abort == 0) *s_abort = 15;
    fence_before_sync();
    __syncthreads();
    if (tid == 0 && *s_abort != 0 && status != nullptr) atomicCAS(status, 0u, 2u | (((uint32_t)*s_abort & 0xFFFu) << 4) | ((uint32_t)s_ctrl[24] << 16));   // the first block to report stays
    if (warp == 4 * G + 1) {
        fence_after_sync();
        tmem_dealloc(tmem_base, pl.tmem_cols);
    }
}

}  // namespace ws
}  // namespace ec
