// K-means assignment + partial sums with the candidate search on the 5th-generation tensor cores.
//
// The squared distance to centroid k is |x|^2 + v_k with v_k = |c_k|^2 - 2 x.c_k.  The inner products
// x.c_k of a tile of points with all centroids are one small GEMM (128 points x NPAD centroids x D):
// the points and centroids are rounded to bf16, staged in shared memory in the tensor core's
// canonical K-major layout, multiplied by tcgen05.mma into an fp32 accumulator in tensor memory, and
// read back with tcgen05.ld, one point per thread.  bf16 makes v_k approximate, so it only proposes:
// the smallest and second smallest v are tracked and whenever they are closer than a bound on the
// error of v (tau) the point is decided again in fp32 by the exact form sum_d (x-c)^2 over all
// centroids - the same rule as the fp32 fused kernel, with a wider tau.  Labels are therefore those
// of the exact form; only speed depends on how well separated the data is.
//
// Partial sums as in the fp32 fused kernel: points pass through shared memory transposed, each warp
// adds its 32 points in order into its own [K][D] slab (lane = coordinate), fixed order, no atomics.
//
// Every wait on the tensor core is bounded; if one gives up the tile falls back to the exact form
// (results stay correct) and a status word records it.
#pragma once

#include <cuda_bf16.h>

namespace ec {
namespace tc {

#ifndef EC_TC_GROUPS
#define EC_TC_GROUPS 1                 // groups of four warps per block; each group owns a 128-point accumulator
#endif
#ifndef EC_TC_MINB
#define EC_TC_MINB 4                   // resident blocks the register allocation must allow
#endif
constexpr int GROUPS = EC_TC_GROUPS;
constexpr int THREADS = 128 * GROUPS;
constexpr int TILE = THREADS;          // points per tile, one per thread
constexpr int WARPS = THREADS / 32;
constexpr uint32_t WAIT_LIMIT = 1u << 20;

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

// D[tmem] (+)= A[smem] * B[smem]^T, bf16 inputs, fp32 accumulate, issued by one thread.
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

// Shared-memory matrix descriptor, K-major, no swizzle: the operand is an array of 8-row x 16-byte
// core matrices (rows 16 bytes apart); lbo = bytes between core matrices adjacent along K,
// sbo = bytes between core matrices adjacent along the row dimension.
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo >> 4) & 0x3FFFu) << 32;
    d |= 1ull << 46;                       // descriptor version of this architecture
    return d;                              // bits 61-63 = 0: no swizzle
}
// Instruction descriptor: fp32 accumulator, bf16 A and B, both K-major, M x N tile.
__host__ __device__ inline uint32_t instr_desc(int M, int N) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

__host__ __device__ inline int npad_of(int K) { return (K + 31) & ~31; }             // accumulator columns per group
__host__ __device__ inline int dpad_of(int D) { return (D + 15) & ~15; }             // K extent of the GEMM
__host__ __device__ inline uint32_t tmem_cols_of(int K) {
    uint32_t need = (uint32_t)GROUPS * (uint32_t)npad_of(K), c = 32;
    while (c < need) c <<= 1;
    return c;
}

struct Layout {   // byte offsets into dynamic shared memory
    size_t cn, b, ax, lab, acc, cnt, bar, total;
};
__host__ __device__ inline Layout layout_of(int D, int K, bool partials) {
    const size_t npad = npad_of(K), dpad = dpad_of(D);
    Layout L;
    size_t off = 0;
    L.cn = off; off += npad * 4;
    off = (off + 1023) & ~(size_t)1023;
    L.b = off; off += npad * dpad * 2;                                   // bf16 centroids
    off = (off + 1023) & ~(size_t)1023;
    const size_t a_bytes = (size_t)TILE * dpad * 2;                      // bf16 points of a tile
    const size_t x_bytes = partials ? (size_t)TILE * (D + 1) * 4 : 0;    // transposed fp32 points (same storage, later)
    L.ax = off; off += a_bytes > x_bytes ? a_bytes : x_bytes;
    off = (off + 15) & ~(size_t)15;
    L.lab = off; off += partials ? (size_t)TILE * 4 : 0;
    L.acc = off; off += partials ? (size_t)WARPS * K * D * 4 : 0;
    L.cnt = off; off += partials ? (size_t)WARPS * K * 4 : 0;
    off = (off + 15) & ~(size_t)15;
    L.bar = off; off += 16;                                              // mbarrier (8 bytes) + tensor-memory address
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

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);   // .x = lo (low half), .y = hi
    uint32_t u;
    memcpy(&u, &v, 4);
    return u;
}

template <int D, bool PARTIALS>
__global__ void __launch_bounds__(THREADS, EC_TC_MINB)
tc_fused_kernel(const float* __restrict__ points, size_t N, int P, int C, const float* __restrict__ centroids, int K,
                int32_t* __restrict__ labels, float* __restrict__ scratch, float tau_scale, uint32_t* __restrict__ status) {
    constexpr int DPAD = (D + 15) & ~15;
    constexpr int KCH = DPAD / 8;                        // 16-byte chunks along K per row
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    const int npad = npad_of(K);
    const Layout L = layout_of(D, K, PARTIALS);
    float* s_cn = reinterpret_cast<float*>(smem_raw + L.cn);
    unsigned char* s_b = smem_raw + L.b;
    unsigned char* s_a = smem_raw + L.ax;                // bf16 operand tiles: group g at g * 128 * DPAD * 2
    float* s_x = reinterpret_cast<float*>(smem_raw + L.ax);
    int* s_lab = reinterpret_cast<int*>(smem_raw + L.lab);
    float* s_acc = reinterpret_cast<float*>(smem_raw + L.acc);
    int* s_cnt = reinterpret_cast<int*>(smem_raw + L.cnt);
    uint64_t* s_bar = reinterpret_cast<uint64_t*>(smem_raw + L.bar);
    uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem_raw + L.bar + 8);

    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5, g = tid >> 7, row = tid & 127;
    const size_t KD = (size_t)K * D;
    const uint32_t ncols = tmem_cols_of(K);
    const uint32_t bar = smem_u32(s_bar);

    if (w == 0) tmem_alloc(smem_u32(s_tmem), ncols);
    if (tid == 0) {
        mbar_init(bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // |c|^2 (padding columns get a value that can never win) and the bf16 centroids in operand layout
    for (int k = tid; k < npad; k += THREADS) {
        float s = 3.0e38f;
        if (k < K) {
            s = 0.0f;
            for (int d = 0; d < D; ++d) s = fmaf(centroids[(size_t)k * D + d], centroids[(size_t)k * D + d], s);
        }
        s_cn[k] = s;
    }
    for (int i = tid; i < npad * KCH; i += THREADS) {
        const int kc = i / npad, n = i - kc * npad;      // chunk kc of centroid n lives at kc * (npad*16) + n*16
        float v[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int d = kc * 8 + e;
            v[e] = (n < K && d < D) ? centroids[(size_t)n * D + d] : 0.0f;
        }
        const uint4 q = make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
        *reinterpret_cast<uint4*>(s_b + (size_t)kc * npad * 16 + (size_t)n * 16) = q;
    }
    if (PARTIALS) {
        for (size_t i = tid; i < (size_t)WARPS * KD; i += THREADS) s_acc[i] = 0.0f;
        for (int i = tid; i < WARPS * K; i += THREADS) s_cnt[i] = 0;
    }
    fence_async_smem();
    fence_before_sync();
    __syncthreads();
    fence_after_sync();
    const uint32_t tmem_base = *s_tmem;
    float cmax = 0.0f;
    for (int k = 0; k < K; ++k) cmax = fmaxf(cmax, s_cn[k]);
    const uint32_t idesc = instr_desc(128, npad);
    const uint32_t a_base = smem_u32(s_a), b_base = smem_u32(s_b);

    const int r = blockIdx.x / C, c = blockIdx.x - r * C;
    const size_t j0 = (size_t)r * N / P, j1 = (size_t)(r + 1) * N / P;
    const size_t len = j1 - j0;
    const size_t b0 = j0 + len * c / C, b1 = j0 + len * (c + 1) / C;
    uint32_t phase = 0;
    bool healthy = true;             // false once a wait on the tensor core gave up: exact form from then on

    for (size_t base = b0; base < b1; base += TILE) {
        const size_t j = base + tid;
        const bool live = j < b1;
        float x[D];
        float xn = 0.0f;
        if (live) {
            const float4* rowp = reinterpret_cast<const float4*>(points + j * D);
#pragma unroll
            for (int q = 0; q < D / 4; ++q) {
                const float4 v = __ldg(rowp + q);
                x[4 * q] = v.x; x[4 * q + 1] = v.y; x[4 * q + 2] = v.z; x[4 * q + 3] = v.w;
            }
#pragma unroll
            for (int d = 0; d < D; ++d) xn = fmaf(x[d], x[d], xn);
        } else {
#pragma unroll
            for (int d = 0; d < D; ++d) x[d] = 0.0f;
        }
        // bf16 operand: chunk kc of row `row` of group g at g*(128*DPAD*2) + kc*(128*16) + row*16
#pragma unroll
        for (int kc = 0; kc < KCH; ++kc) {
            float v[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) v[e] = (kc * 8 + e < D) ? x[kc * 8 + e] : 0.0f;
            const uint4 q = make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
            *reinterpret_cast<uint4*>(s_a + (size_t)g * 128 * DPAD * 2 + (size_t)kc * 128 * 16 + (size_t)row * 16) = q;
        }
        fence_async_smem();          // the tensor core reads shared memory through the async proxy
        fence_before_sync();
        __syncthreads();
        if (tid == 0 && healthy) {
            fence_after_sync();
#pragma unroll
            for (int gg = 0; gg < GROUPS; ++gg) {
#pragma unroll
                for (int ks = 0; ks < DPAD / 16; ++ks) {
                    const uint64_t ad = smem_desc(a_base + gg * 128 * DPAD * 2 + ks * 2 * 128 * 16, 128 * 16, 128);
                    const uint64_t bd = smem_desc(b_base + ks * 2 * npad * 16, npad * 16, 128);
                    mma_bf16(tmem_base + (uint32_t)(gg * npad), ad, bd, idesc, ks > 0 ? 1u : 0u);
                }
            }
            mma_commit(bar);         // the barrier completes when both accumulators are written
        }
        bool done = false;
        if (healthy) {
            for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
                if (mbar_try_wait(bar, phase)) { done = true; break; }
            }
        }
        done = __syncthreads_and(done) != 0;     // all threads take the same path
        healthy = done;
        phase ^= 1u;
        fence_after_sync();
        float m1 = __int_as_float(0x7f800000), m2 = m1;
        int kb = 0;
        if (done) {
            for (int ch = 0; ch < npad / 32; ++ch) {
                uint32_t dot[32];
                tmem_ld32(tmem_base + ((uint32_t)((w & 3) * 32) << 16) + (uint32_t)(g * npad + ch * 32), dot);
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const int k = ch * 32 + i;
                    const float v = fmaf(-2.0f, __uint_as_float(dot[i]), s_cn[k]);
                    const bool lt = v < m1;
                    m2 = fminf(m2, lt ? m1 : v);
                    kb = lt ? k : kb;
                    m1 = lt ? v : m1;
                }
            }
        } else if (tid == 0 && status != nullptr) {
            atomicOr(status, 1u);    // the tensor core did not answer in time: exact form from here on
        }
        fence_before_sync();         // accumulator reads are done before the next tile's MMA may overwrite it
        // rounding to bf16 perturbs v by at most 2^-7 |x||c| <= 2^-8 (|x|^2 + |c|max^2) per candidate
        const float tau = tau_scale * (xn + cmax);
        if (live && (!done || !(m2 - m1 > tau))) kb = exact_argmin_global<D>(x, centroids, K);
        if (live) labels[j] = kb;
        if (PARTIALS) {
            __syncthreads();                                   // (the operand tiles have been consumed: the MMA is complete)
            s_lab[tid] = live ? kb : -1;
#pragma unroll
            for (int d = 0; d < D; ++d) s_x[(size_t)tid * (D + 1) + d] = x[d];
            __syncthreads();
            float* acc = s_acc + (size_t)w * KD;
            int* cnt = s_cnt + w * K;
            for (int jj = 0; jj < 32; jj += 4) {
                int lab[4];
                float xv[4][(D + 31) / 32];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int pt = w * 32 + jj + u;
                    lab[u] = s_lab[pt];
#pragma unroll
                    for (int q = 0; q < (D + 31) / 32; ++q) {
                        const int d = lane + 32 * q;
                        xv[u][q] = d < D ? s_x[(size_t)pt * (D + 1) + d] : 0.0f;
                    }
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    if (lab[u] >= 0) {
#pragma unroll
                        for (int q = 0; q < (D + 31) / 32; ++q) {
                            const int d = lane + 32 * q;
                            if (d < D) acc[(size_t)lab[u] * D + d] = __fadd_rn(acc[(size_t)lab[u] * D + d], xv[u][q]);
                        }
                        if (lane == 0) cnt[lab[u]] += 1;
                    }
                }
            }
            __syncthreads();                                   // s_x is free again for the next tile's operands
        }
    }
    __syncthreads();
    if (PARTIALS) {
        const int stride = D + 4;
        float* dst = scratch + ((size_t)r * C + c) * (size_t)K * stride;
        for (size_t i = tid; i < (size_t)K * stride; i += THREADS) {
            const int kk = (int)(i / stride), d = (int)(i - (size_t)kk * stride);
            float val = 0.0f;
            if (d < D) {
                val = s_acc[(size_t)kk * D + d];
                for (int ww = 1; ww < WARPS; ++ww) val = __fadd_rn(val, s_acc[(size_t)ww * KD + (size_t)kk * D + d]);
            } else if (d == D) {
                int n = 0;
                for (int ww = 0; ww < WARPS; ++ww) n += s_cnt[ww * K + kk];
                val = (float)n;
            }
            dst[i] = val;
        }
    }
    fence_before_sync();
    __syncthreads();
    if (w == 0) tmem_dealloc(tmem_base, ncols);
}

}  // namespace tc
}  // namespace ec
