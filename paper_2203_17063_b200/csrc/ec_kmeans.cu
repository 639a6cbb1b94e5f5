// K-means driver on top of the eventually consistent allreduce.
//
// The paper's iterative-convergent ML workload (Sec. I, Sec. V) tolerates contributions that are
// missing or late; here Lloyd's iteration plays that role: every simulated rank assigns its shard
// of points, forms per-centroid partial sums, and the partial sums are combined by one allreduce
// epoch in which only the notified (rank, centroid-row) contributions take part.
//
// Kernels, fastest first (ec_kmeans_iterate takes the first that covers the shape):
//   tc::tc_fused_kernel   (ec_kmeans_tc.cuh) assignment and partial sums as two small GEMMs on the
//             tensor cores, exact fp32 re-decision of every point the bf16 search cannot separate;
//             D in {16, 32}, K <= 256.  After the first iteration it adds to the per-rank sums only
//             what changed since the labels were last written (every KM_REFRESH-th iteration sums
//             everything afresh).
//   fused_kernel          the same two steps on the fp32 pipes: one FMA per (point, centroid,
//             coordinate) proposes, the exact form decides inside the error bound; per-warp
//             shared-memory slabs collect the sums in a fixed order; D in {8, 16, 32, 64}.
//   assign_kernel / assign_generic_kernel, partials_kernel   one step each, any D that is a multiple
//             of 4: squared distance sum_d (x-c)^2 in fp32 with the point in registers; one warp
//             walks a run of points with lane = coordinate into its own [K][D] slab.  These also
//             serve ec_kmeans_partials (and ec_kmeans_assign for shapes the fused kernels skip).
//   partials_fold_kernel  folds the row blocks of a rank in index order;
//   update_kernel         centroid = sum / points where points > 0;
//   update_drift_kernel   the same in one block, and how far every centroid has moved in all (what the distance
//                         bounds of the tensor-core path rest on).
// No floating-point atomics on any of these paths: sums are the same bits run after run.

#include <mutex>
#include <new>

#include "ec_common.cuh"

namespace ec {
namespace {

constexpr int AS_THREADS = 256;
constexpr int PT_THREADS = 256;
constexpr int PT_WARPS = PT_THREADS / 32;
constexpr size_t SMEM_BUDGET = 200 * 1024;
constexpr int KM_REFRESH = 32;                  // iterations that sum only changes before a full pass
constexpr size_t ASSIGN_SMEM_MAX = 64 * 1024;   // centroid chunk staged by the assignment kernels

// ---------------------------------------------------------------------------------------------
// assignment
// ---------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(AS_THREADS)
assign_kernel(const float* __restrict__ points, size_t N, const float* __restrict__ centroids, int K, int kc,
              int32_t* __restrict__ labels) {
    extern __shared__ __align__(16) float s_c[];   // kc centroids of D floats
    const int tid = threadIdx.x;
    for (size_t base = (size_t)blockIdx.x * AS_THREADS; base < N; base += (size_t)gridDim.x * AS_THREADS) {
        const size_t j = base + tid;
        const bool live = j < N;
        float x[D];
        if (live) {
            const float4* row = reinterpret_cast<const float4*>(points + j * D);
#pragma unroll
            for (int q = 0; q < D / 4; ++q) {
                const float4 v = __ldg(row + q);
                x[4 * q] = v.x; x[4 * q + 1] = v.y; x[4 * q + 2] = v.z; x[4 * q + 3] = v.w;
            }
        } else {
#pragma unroll
            for (int d = 0; d < D; ++d) x[d] = 0.0f;
        }
        float best = __int_as_float(0x7f800000);
        int bi = 0;
        for (int k0 = 0; k0 < K; k0 += kc) {
            const int kn = K - k0 < kc ? K - k0 : kc;
            __syncthreads();                         // previous chunk fully consumed
            for (int i = tid; i < kn * D / 4; i += AS_THREADS)
                reinterpret_cast<float4*>(s_c)[i] = __ldg(reinterpret_cast<const float4*>(centroids + (size_t)k0 * D) + i);
            __syncthreads();
            int k = 0;
            for (; k + 1 < kn; k += 2) {             // two centroids at a time: two independent chains
                const float4* c0 = reinterpret_cast<const float4*>(s_c + (size_t)k * D);
                const float4* c1 = reinterpret_cast<const float4*>(s_c + (size_t)(k + 1) * D);
                float d0 = 0.0f, d1 = 0.0f;
#pragma unroll
                for (int q = 0; q < D / 4; ++q) {
                    const float4 a = c0[q], b = c1[q];
                    float t;
                    t = x[4 * q] - a.x; d0 = fmaf(t, t, d0);
                    t = x[4 * q + 1] - a.y; d0 = fmaf(t, t, d0);
                    t = x[4 * q + 2] - a.z; d0 = fmaf(t, t, d0);
                    t = x[4 * q + 3] - a.w; d0 = fmaf(t, t, d0);
                    t = x[4 * q] - b.x; d1 = fmaf(t, t, d1);
                    t = x[4 * q + 1] - b.y; d1 = fmaf(t, t, d1);
                    t = x[4 * q + 2] - b.z; d1 = fmaf(t, t, d1);
                    t = x[4 * q + 3] - b.w; d1 = fmaf(t, t, d1);
                }
                if (d0 < best) { best = d0; bi = k0 + k; }          // strict <: the lowest index wins a tie
                if (d1 < best) { best = d1; bi = k0 + k + 1; }
            }
            if (k < kn) {
                const float4* c0 = reinterpret_cast<const float4*>(s_c + (size_t)k * D);
                float d0 = 0.0f;
#pragma unroll
                for (int q = 0; q < D / 4; ++q) {
                    const float4 a = c0[q];
                    float t;
                    t = x[4 * q] - a.x; d0 = fmaf(t, t, d0);
                    t = x[4 * q + 1] - a.y; d0 = fmaf(t, t, d0);
                    t = x[4 * q + 2] - a.z; d0 = fmaf(t, t, d0);
                    t = x[4 * q + 3] - a.w; d0 = fmaf(t, t, d0);
                }
                if (d0 < best) { best = d0; bi = k0 + k; }
            }
        }
        if (live) labels[j] = bi;
    }
}

// Any D (multiple of 4, at most 128): coordinates are re-read from global memory (L1) per centroid chunk.
__global__ void __launch_bounds__(AS_THREADS)
assign_generic_kernel(const float* __restrict__ points, size_t N, int D, const float* __restrict__ centroids, int K,
                      int kc, int32_t* __restrict__ labels) {
    extern __shared__ __align__(16) float s_c[];
    const int tid = threadIdx.x;
    for (size_t base = (size_t)blockIdx.x * AS_THREADS; base < N; base += (size_t)gridDim.x * AS_THREADS) {
        const size_t j = base + tid;
        const bool live = j < N;
        const float* row = points + (live ? j : 0) * (size_t)D;
        float best = __int_as_float(0x7f800000);
        int bi = 0;
        for (int k0 = 0; k0 < K; k0 += kc) {
            const int kn = K - k0 < kc ? K - k0 : kc;
            __syncthreads();
            for (int i = tid; i < kn * D; i += AS_THREADS) s_c[i] = centroids[(size_t)k0 * D + i];
            __syncthreads();
            for (int k = 0; k < kn; ++k) {
                float d0 = 0.0f;
                for (int d = 0; d < D; ++d) {
                    const float t = row[d] - s_c[k * D + d];
                    d0 = fmaf(t, t, d0);
                }
                if (d0 < best) { best = d0; bi = k0 + k; }
            }
        }
        if (live) labels[j] = bi;
    }
}

// ---------------------------------------------------------------------------------------------
// per-rank partial sums
// ---------------------------------------------------------------------------------------------
// Block (r, c) covers the c-th of C equal runs of rank r's points; its `warps` warps split the run
// again.  out: [P][C][K][D+4] (scratch) - or the partials themselves when C == 1.
__global__ void __launch_bounds__(PT_THREADS)
partials_kernel(const float* __restrict__ points, const int32_t* __restrict__ labels, size_t N, int D, int K, int P,
                int C, int warps, float* __restrict__ out) {
    extern __shared__ __align__(16) float s_acc[];                  // [warps][K][D] sums, then [warps][K] counts
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int r = blockIdx.x / C, c = blockIdx.x - r * C;
    const size_t KD = (size_t)K * D;
    int* s_cnt = reinterpret_cast<int*>(s_acc + (size_t)warps * KD);
    for (size_t i = threadIdx.x; i < (size_t)warps * KD; i += blockDim.x) s_acc[i] = 0.0f;
    for (size_t i = threadIdx.x; i < (size_t)warps * K; i += blockDim.x) s_cnt[i] = 0;
    __syncthreads();
    const size_t j0 = (size_t)r * N / P, j1 = (size_t)(r + 1) * N / P;
    const size_t len = j1 - j0;
    const size_t b0 = j0 + len * c / C, b1 = j0 + len * (c + 1) / C;   // this block's run
    if (w < warps) {
        const size_t blen = b1 - b0;
        const size_t p0 = b0 + blen * w / warps, p1 = b0 + blen * (w + 1) / warps;
        float* acc = s_acc + (size_t)w * KD;
        int* cnt = s_cnt + (size_t)w * K;
        const int dims = (D + 31) / 32;                               // coordinates per lane
        size_t j = p0;
        for (; j + 4 <= p1; j += 4) {                                 // loads of four points in flight
            int lab[4];
            float v[4][4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                lab[u] = __ldg(labels + j + u);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int d = lane + 32 * q;
                    v[u][q] = (q < dims && d < D) ? __ldg(points + (j + u) * (size_t)D + d) : 0.0f;
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int k = lab[u];
                if ((unsigned)k < (unsigned)K) {
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int d = lane + 32 * q;
                        if (q < dims && d < D) acc[(size_t)k * D + d] = __fadd_rn(acc[(size_t)k * D + d], v[u][q]);
                    }
                    if (lane == 0) cnt[k] += 1;
                }
            }
        }
        for (; j < p1; ++j) {
            const int k = __ldg(labels + j);
            if ((unsigned)k < (unsigned)K) {
                for (int d = lane; d < D; d += 32)
                    acc[(size_t)k * D + d] = __fadd_rn(acc[(size_t)k * D + d], __ldg(points + j * (size_t)D + d));
                if (lane == 0) cnt[k] += 1;
            }
        }
    }
    __syncthreads();
    // fold the warps in index order and write rows of D+4
    const int stride = D + 4;
    float* dst = out + ((size_t)r * C + c) * (size_t)K * stride;
    for (size_t i = threadIdx.x; i < (size_t)K * stride; i += blockDim.x) {
        const int k = (int)(i / stride), d = (int)(i - (size_t)k * stride);
        float val = 0.0f;
        if (d < D) {
            val = s_acc[(size_t)k * D + d];
            for (int ww = 1; ww < warps; ++ww) val = __fadd_rn(val, s_acc[(size_t)ww * KD + (size_t)k * D + d]);
        } else if (d == D) {
            int n = 0;
            for (int ww = 0; ww < warps; ++ww) n += s_cnt[(size_t)ww * K + k];
            val = (float)n;                                            // exact: at most 2^24 points per block
        }
        dst[i] = val;
    }
}

// partials[r][k][d] = scratch[r][0][k][d] + scratch[r][1][k][d] + ... in index order, one warp per row (r, k).
// accumulate: the row blocks hold changes, which are added to what partials holds; only the row blocks that hold
// changes (dirty) were written.  The point counts stay exact integers under such updates, the coordinate sums
// collect rounding: a row whose count comes back to zero is an empty cluster and its sums are set to zero exactly.
__global__ void partials_fold_kernel(const float* __restrict__ scratch, int C, size_t row_elems, size_t total,
                                     float* __restrict__ partials, int stride, int accumulate = 0,
                                     const uint32_t* __restrict__ dirty = nullptr,
                                     const uint32_t* __restrict__ any_work = nullptr) {
    grid_dependency_wait();                                  // (launched ahead of its predecessor's end, see launch_dependent)
    if (any_work != nullptr && *any_work == 0u) return;      // the bounds check found no tile to search: nothing was written
    const int lane = threadIdx.x & 31;
    const size_t rows = total / (size_t)stride;
    const size_t per_rank = row_elems / (size_t)stride;      // K
    constexpr int U = 8;                                      // loads in flight per lane
    for (size_t row = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; row < rows; row += ((size_t)gridDim.x * blockDim.x) >> 5) {
        const size_t r = row / per_rank;
        const float* src = scratch + r * (size_t)C * row_elems + (row - r * per_rank) * (size_t)stride;
        float* dst = partials + row * (size_t)stride;
        if (accumulate) {
            // which row blocks of this rank hold changes: 32 flags per ballot (C is at most 64)
            unsigned long long mask = 0;
            for (int c0 = 0; c0 < C; c0 += 32) {
                const int c = c0 + lane;
                const unsigned m = __ballot_sync(0xffffffffu, c < C && dirty[r * (size_t)C + c] != 0u);
                mask |= (unsigned long long)m << c0;
            }
            if (mask == 0) continue;
            const int D = stride - 4;
            float cnt = dst[D];                               // every lane folds the count: it decides what the others write
            for (unsigned long long m = mask; m; m &= m - 1) cnt = __fadd_rn(cnt, src[(size_t)(__ffsll((long long)m) - 1) * row_elems + D]);
            __syncwarp();                                     // all lanes have read the old count before lane D % 32 replaces it
            for (int e = lane; e < stride; e += 32) {
                float v = dst[e];
                for (unsigned long long m = mask; m; m &= m - 1) v = __fadd_rn(v, src[(size_t)(__ffsll((long long)m) - 1) * row_elems + e]);
                dst[e] = (cnt == 0.0f && e < D) ? 0.0f : v;
            }
        } else {
            for (int e = lane; e < stride; e += 32) {
                float v = src[e];
                int c = 1;
                for (; c + U <= C; c += U) {                  // the loads of U row blocks together, the additions in index order
                    float t[U];
#pragma unroll
                    for (int u = 0; u < U; ++u) t[u] = src[(size_t)(c + u) * row_elems + e];
#pragma unroll
                    for (int u = 0; u < U; ++u) v = __fadd_rn(v, t[u]);
                }
                for (; c < C; ++c) v = __fadd_rn(v, src[(size_t)c * row_elems + e]);
                dst[e] = v;
            }
        }
    }
}

// |x|^2 of every point (four chains, the order the fused kernels used to take), once per context.
__global__ void point_norm_kernel(const float* __restrict__ points, size_t N, int D, float* __restrict__ xnorm) {
    for (size_t j = (size_t)blockIdx.x * blockDim.x + threadIdx.x; j < N; j += (size_t)gridDim.x * blockDim.x) {
        const float4* row = reinterpret_cast<const float4*>(points + j * D);
        float n0 = 0.0f, n1 = 0.0f, n2 = 0.0f, n3 = 0.0f;
        for (int q = 0; q < D / 4; ++q) {
            const float4 v = __ldg(row + q);
            n0 = fmaf(v.x, v.x, n0); n1 = fmaf(v.y, v.y, n1); n2 = fmaf(v.z, v.z, n2); n3 = fmaf(v.w, v.w, n3);
        }
        xnorm[j] = (n0 + n1) + (n2 + n3);
    }
}

__global__ void update_kernel(const float* __restrict__ reduced, int D, int K, float* __restrict__ centroids) {
    grid_dependency_wait();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= K * D) return;
    const int k = i / D, d = i - k * D;
    const float pts = reduced[(size_t)k * (D + 4) + D];
    if (pts > 0.0f) centroids[i] = __fdiv_rn(reduced[(size_t)k * (D + 4) + d], pts);
}

// The same update in one block, which also keeps the drift sums the assignment's distance bounds rest on:
// drift[k] += |c_k(new) - c_k(old)|, drift[K] += max_k of those moves.  Every rounding goes upwards, so the sums
// never understate how far a centroid has moved.  One warp per centroid, lanes over the coordinates.
constexpr int UD_THREADS = 1024;
__global__ void __launch_bounds__(UD_THREADS)
update_drift_kernel(const float* __restrict__ reduced, int D, int K, float* __restrict__ centroids, float* __restrict__ drift) {
    __shared__ float s_max[UD_THREADS / 32];
    grid_dependency_wait();
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    float wmax = 0.0f;
    for (int k = wid; k < K; k += UD_THREADS / 32) {
        const float pts = reduced[(size_t)k * (D + 4) + D];
        float sq = 0.0f;
        for (int d = lane; d < D; d += 32) {             // the loads do not wait for the count
            const float c_old = centroids[(size_t)k * D + d];
            const float sum = reduced[(size_t)k * (D + 4) + d];
            if (pts > 0.0f) {
                const float c_new = __fdiv_rn(sum, pts);
                centroids[(size_t)k * D + d] = c_new;
                const float diff = fmaxf(fabsf(__fsub_ru(c_new, c_old)), fabsf(__fsub_rd(c_new, c_old)));
                sq = __fadd_ru(sq, __fmul_ru(diff, diff));
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sq = __fadd_ru(sq, __shfl_xor_sync(0xffffffffu, sq, o));
        const float move = __fsqrt_ru(sq);
        if (lane == 0 && move > 0.0f) drift[k] = __fadd_ru(drift[k], move);
        wmax = fmaxf(wmax, move);
    }
    if (lane == 0) s_max[wid] = wmax;
    __syncthreads();
    if (threadIdx.x == 0) {
        float m = 0.0f;
        for (int w = 0; w < UD_THREADS / 32; ++w) m = fmaxf(m, s_max[w]);
        if (m > 0.0f) drift[K] = __fadd_ru(drift[K], m);
        reinterpret_cast<uint32_t*>(drift)[K + 1] = 0u;      // "some tile has to be searched": set by the next bounds check
    }
}

// ---------------------------------------------------------------------------------------------
// fused assignment + partial sums (the path ec_kmeans_iterate takes)
// ---------------------------------------------------------------------------------------------
// Candidate search: argmin_k |x-c_k|^2 = argmin_k v_k with v_k = |c_k|^2 - 2 x.c_k, one FMA per
// (point, centroid, coordinate) instead of a subtract and an FMA.  v_k cancels badly, so it only
// *proposes*: the smallest and second smallest v are tracked, and whenever they are closer than a
// bound on the rounding error of v (tau) the point is decided again by the exact form
// sum_d (x-c)^2 over all centroids.  A point that is not re-decided has a winner that leads by more
// than the error, hence is the winner of the exact form too.  Exact ties always re-decide, so the
// lowest index wins them.  Two points per thread share each centroid value read from shared memory.
//
// Partial sums: the block's points pass through shared memory once more, transposed, and each warp
// adds its 32 points one after the other into its own [K][D] slab with lane = coordinate: plain
// read-add-write in a fixed order.  Block (r, c) covers the c-th of C runs of rank r's points and
// writes one [K][D+4] row block of scratch; the rows of a rank are folded in order afterwards.
constexpr int FU_THREADS = 256;
constexpr int FU_PPT = 2;                       // points per thread
constexpr int FU_TILE = FU_THREADS * FU_PPT;    // points per tile
constexpr int FU_WARPS = FU_THREADS / 32;

__host__ __device__ inline size_t fused_smem_floats(int D, int K, bool partials) {
    size_t f = (size_t)K * D + (size_t)((K + 3) & ~3);                       // -2c and |c|^2
    if (partials) f += (size_t)FU_THREADS * (D + 1) + FU_THREADS             // transposed points, labels
                       + (size_t)FU_WARPS * K * D + (size_t)FU_WARPS * K;    // slabs and counts
    return f;
}

template <int D>
__device__ __forceinline__ void exact_argmin(const float (&x)[D], const float* s_c2, int K, int& kb) {
    float best = __int_as_float(0x7f800000);
    int bi = 0;
    for (int k = 0; k < K; ++k) {
        const float4* c = reinterpret_cast<const float4*>(s_c2 + (size_t)k * D);
        float d0 = 0.0f;
#pragma unroll
        for (int q = 0; q < D / 4; ++q) {
            const float4 a = c[q];                      // -2c: c = -0.5 * a exactly
            float t;
            t = x[4 * q] - (-0.5f * a.x); d0 = fmaf(t, t, d0);
            t = x[4 * q + 1] - (-0.5f * a.y); d0 = fmaf(t, t, d0);
            t = x[4 * q + 2] - (-0.5f * a.z); d0 = fmaf(t, t, d0);
            t = x[4 * q + 3] - (-0.5f * a.w); d0 = fmaf(t, t, d0);
        }
        if (d0 < best) { best = d0; bi = k; }           // strict <: the lowest index wins a tie
    }
    kb = bi;
}

#define EC_TRACK(v, k, b1, b2, kb)                 \
    do {                                           \
        const bool lt__ = (v) < (b1);              \
        (b2) = fminf((b2), lt__ ? (b1) : (v));     \
        (kb) = lt__ ? (k) : (kb);                  \
        (b1) = lt__ ? (v) : (b1);                  \
    } while (0)

template <int D, bool PARTIALS>
__global__ void __launch_bounds__(FU_THREADS, 2)
fused_kernel(const float* __restrict__ points, size_t N, int P, int C, const float* __restrict__ centroids, int K,
             int32_t* __restrict__ labels, float* __restrict__ scratch, float tau_scale) {
    extern __shared__ __align__(16) float smem[];
    float* s_c2 = smem;                                        // [K][D]   -2 c
    float* s_cn = s_c2 + (size_t)K * D;                        // [K]      |c|^2
    float* s_x = s_cn + ((K + 3) & ~3);                        // [256][D+1]
    int* s_lab = reinterpret_cast<int*>(s_x + (size_t)FU_THREADS * (D + 1));
    float* s_acc = reinterpret_cast<float*>(s_lab + FU_THREADS);          // [8][K][D]
    int* s_cnt = reinterpret_cast<int*>(s_acc + (size_t)FU_WARPS * K * D);  // [8][K]
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const size_t KD = (size_t)K * D;

    for (int i = tid; i < (int)KD; i += FU_THREADS) s_c2[i] = -2.0f * centroids[i];
    for (int k = tid; k < K; k += FU_THREADS) {
        float s = 0.0f;
        for (int d = 0; d < D; ++d) s = fmaf(centroids[(size_t)k * D + d], centroids[(size_t)k * D + d], s);
        s_cn[k] = s;
    }
    if (PARTIALS) {
        for (size_t i = tid; i < (size_t)FU_WARPS * KD; i += FU_THREADS) s_acc[i] = 0.0f;
        for (int i = tid; i < FU_WARPS * K; i += FU_THREADS) s_cnt[i] = 0;
    }
    __syncthreads();
    float cmax = 0.0f;
    for (int k = 0; k < K; ++k) cmax = fmaxf(cmax, s_cn[k]);

    const int r = blockIdx.x / C, c = blockIdx.x - r * C;
    const size_t j0 = (size_t)r * N / P, j1 = (size_t)(r + 1) * N / P;
    const size_t len = j1 - j0;
    const size_t b0 = j0 + len * c / C, b1 = j0 + len * (c + 1) / C;

    for (size_t base = b0; base < b1; base += FU_TILE) {
        float x[FU_PPT][D];
        bool live[FU_PPT];
        float xn[FU_PPT];
#pragma unroll
        for (int p = 0; p < FU_PPT; ++p) {
            const size_t j = base + (size_t)p * FU_THREADS + tid;
            live[p] = j < b1;
            xn[p] = 0.0f;
            if (live[p]) {
                const float4* row = reinterpret_cast<const float4*>(points + j * D);
#pragma unroll
                for (int q = 0; q < D / 4; ++q) {
                    const float4 v = __ldg(row + q);
                    x[p][4 * q] = v.x; x[p][4 * q + 1] = v.y; x[p][4 * q + 2] = v.z; x[p][4 * q + 3] = v.w;
                }
#pragma unroll
                for (int d = 0; d < D; ++d) xn[p] = fmaf(x[p][d], x[p][d], xn[p]);
            } else {
#pragma unroll
                for (int d = 0; d < D; ++d) x[p][d] = 0.0f;
            }
        }
        float m1[FU_PPT], m2[FU_PPT];
        int kb[FU_PPT];
#pragma unroll
        for (int p = 0; p < FU_PPT; ++p) { m1[p] = __int_as_float(0x7f800000); m2[p] = m1[p]; kb[p] = 0; }
        int k = 0;
        for (; k + 4 <= K; k += 4) {                 // four centroids x two points: eight independent chains
            float v[FU_PPT][4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const float cn = s_cn[k + u];
#pragma unroll
                for (int p = 0; p < FU_PPT; ++p) v[p][u] = cn;
            }
#pragma unroll
            for (int q = 0; q < D / 4; ++q) {
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const float4 a = reinterpret_cast<const float4*>(s_c2 + (size_t)(k + u) * D)[q];
#pragma unroll
                    for (int p = 0; p < FU_PPT; ++p) {
                        v[p][u] = fmaf(x[p][4 * q], a.x, v[p][u]);
                        v[p][u] = fmaf(x[p][4 * q + 1], a.y, v[p][u]);
                        v[p][u] = fmaf(x[p][4 * q + 2], a.z, v[p][u]);
                        v[p][u] = fmaf(x[p][4 * q + 3], a.w, v[p][u]);
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
#pragma unroll
                for (int p = 0; p < FU_PPT; ++p) EC_TRACK(v[p][u], k + u, m1[p], m2[p], kb[p]);
            }
        }
        for (; k < K; ++k) {
            const float cn = s_cn[k];
#pragma unroll
            for (int p = 0; p < FU_PPT; ++p) {
                float v = cn;
#pragma unroll
                for (int d = 0; d < D; ++d) v = fmaf(x[p][d], s_c2[(size_t)k * D + d], v);
                EC_TRACK(v, k, m1[p], m2[p], kb[p]);
            }
        }
#pragma unroll
        for (int p = 0; p < FU_PPT; ++p) {
            // |error of v| <= (D+3) u (|x| + |c|)^2 <= (D+3) u 2 (|x|^2 + |c|max^2); tau covers both candidates twice over
            const float tau = tau_scale * (xn[p] + cmax);
            if (live[p] && !(m2[p] - m1[p] > tau)) exact_argmin<D>(x[p], s_c2, K, kb[p]);
            if (live[p]) labels[base + (size_t)p * FU_THREADS + tid] = kb[p];
        }
        if (PARTIALS) {
#pragma unroll
            for (int p = 0; p < FU_PPT; ++p) {
                __syncthreads();                                   // the previous half has been consumed
                s_lab[tid] = live[p] ? kb[p] : -1;
#pragma unroll
                for (int d = 0; d < D; ++d) s_x[(size_t)tid * (D + 1) + d] = x[p][d];
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
            }
        }
    }
    if (PARTIALS) {
        __syncthreads();
        const int stride = D + 4;
        float* dst = scratch + ((size_t)r * C + c) * (size_t)K * stride;
        for (size_t i = tid; i < (size_t)K * stride; i += FU_THREADS) {
            const int kk = (int)(i / stride), d = (int)(i - (size_t)kk * stride);
            float val = 0.0f;
            if (d < D) {
                val = s_acc[(size_t)kk * D + d];
                for (int ww = 1; ww < FU_WARPS; ++ww) val = __fadd_rn(val, s_acc[(size_t)ww * KD + (size_t)kk * D + d]);
            } else if (d == D) {
                int n = 0;
                for (int ww = 0; ww < FU_WARPS; ++ww) n += s_cnt[ww * K + kk];
                val = (float)n;
            }
            dst[i] = val;
        }
    }
}
#undef EC_TRACK

}  // namespace
}  // namespace ec

#include "ec_kmeans_tc.cuh"
#include "ec_kmeans_ws.cuh"

namespace ec {
namespace {

int sm_count_km() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
    return n;
}

}  // namespace
}  // namespace ec

struct ec_kmeans {
    const float* points;
    size_t N;
    int D, K, P;
    void* ws;
    bool own_ws;
    // carved out of ws
    float* centroids;      // [K][D]
    int32_t* labels;       // [N]
    float* partials;       // [P][K][D+4]
    float* scratch;        // [P][C][K][D+4]
    float* reduced;        // [K][D+4]
    uint32_t* contrib;     // [K]
    void* ar_ws;
    ec_ctx_t* ar;
    const void* bufs[EC_MAX_RANKS];
    int sms, C, warps, kc;
    size_t assign_smem, part_smem;
    int Cf;                // runs per rank of the fused kernel; 0 = shape not covered by it
    size_t fused_smem, fused_assign_smem;
    bool tc_ok;            // the tensor-core candidate search covers this shape
    bool ws_ok;            // ... and so does its warp-specialised form (K <= 128, tensor map of the points made)
    CUtensorMap pmap;      // the points as a 2-D tensor [N][D] of fp32, tiles of 128 rows, swizzled rows
    ec::ws::Plan ws_plan, ws_plan_delta, ws_plan_assign;
    int path;              // 0 = automatic, 1 = fp32 fused kernel, 2 = tensor cores, 3 = tensor cores, register-staged form
    size_t tc_smem, tc_assign_smem;
    int tc_wave_full, tc_wave_delta, tc_wave_assign;   // resident blocks of the tensor-core kernels on the whole device
    uint32_t* tc_status;   // device word: nonzero if a wait on the tensor core ever gave up
    uint32_t* dirty;       // [P][Cf]: delta mode, which row blocks of scratch hold changes
    float2* bounds;        // [N]: distance bounds of every point (tensor-core path), see tc_fused_kernel
    float* xnorm;          // [N]: |x|^2 of every point, made once (the points do not change under a context)
    float* drift;          // [K + 1]: how far every centroid has moved in all, and the sum of the largest moves
    uint32_t* need;        // [P * Cf][need_words]: delta mode with bounds, which tiles have to be searched
    int need_words;
    bool skipped;          // the last pass of the tensor-core kernel ran behind a bounds check
    bool bounds_valid;     // the bounds belong to the labels and to the drift sums
    bool use_bounds;       // tiles whose bounds say that no label can change are skipped
    bool state_valid;      // labels and partials belong together (an iteration has run): changes can be summed
    int since_full;        // iterations since everything was summed afresh
    int refresh;           // every refresh-th iteration sums everything afresh (1: every iteration)
};

using namespace ec;

namespace {

struct KmLayout {
    size_t off_centroids, off_labels, off_partials, off_scratch, off_reduced, off_contrib, off_dirty, off_bounds, off_drift, off_need, off_xnorm, off_ar, total;
    int need_words;      // tiles of the longest run (0: the distance bounds are not kept)
    int C, warps;
    int Cf;   // runs per rank for the fused assignment+partials kernel, 0 if the shape is not covered
};

// Shapes the fused kernel is instantiated for and whose shared memory fits.
bool fused_capable(int D, int K) {
    if (D != 8 && D != 16 && D != 32 && D != 64) return false;
    return fused_smem_floats(D, K, true) * 4 <= SMEM_BUDGET;
}

// Shapes the tensor-core kernel covers: accumulators of both point groups fit in tensor memory.
bool tc_capable(int D, int K) {
    if (D != 16 && D != 32) return false;   // the point tile holds high parts, ones and low parts in 16 chunk columns
    if (tc::npad_of(K) > 256) return false;   // MMA width; search and sums accumulators (2 x npad columns) fit in tensor memory
    return tc::layout_of(D, K, true).total <= SMEM_BUDGET;
}

// Blocks per rank (C) and warps per block for the partials kernel, from the shape alone.
bool km_plan(size_t N, int D, int K, int P, int sms, KmLayout* L) {
    const size_t KD = (size_t)K * D;
    int warps = PT_WARPS;
    while (warps > 1 && (size_t)warps * (KD + K) * 4 > SMEM_BUDGET / 2) warps >>= 1;   // two blocks per SM if possible
    if ((size_t)warps * (KD + K) * 4 > SMEM_BUDGET) return false;
    const size_t smem = (size_t)warps * (KD + K) * 4;
    const int per_sm = (int)(SMEM_BUDGET / smem) < 2048 / PT_THREADS ? (int)(SMEM_BUDGET / smem) : 2048 / PT_THREADS;
    int C = (sms * (per_sm < 1 ? 1 : per_sm)) / P;          // one wave of resident blocks
    if (C < 1) C = 1;
    const size_t shard = N / (size_t)P > 0 ? N / (size_t)P : 1;
    while (C > 1 && shard / (size_t)C < 256) --C;            // keep runs long enough to be worth a block
    L->C = C;
    L->warps = warps;
    // fused kernels: runs of about 2048 points, their number rounded to whole waves of resident blocks
    // (four per SM) so that the last wave is as full as the others
    L->Cf = 0;
    if (fused_capable(D, K)) {
        const size_t slots = (size_t)sms * 4;
        const size_t target = N / 2048 > 0 ? N / 2048 : 1;
        size_t waves = (target + slots / 2) / slots;
        if (waves < 1) waves = 1;
        size_t cf = waves * slots / (size_t)P;
        while (cf > 1 && shard / cf < 512) --cf;            // keep runs long enough to be worth a block
        L->Cf = (int)(cf < 1 ? 1 : cf > 64 ? 64 : cf);
    }
    const size_t stride = (size_t)D + 4;
    size_t off = 0;
    L->off_centroids = off; off = align_up(off + KD * 4, 256);
    L->off_labels = off; off = align_up(off + N * 4, 256);
    L->off_partials = off; off = align_up(off + (size_t)P * K * stride * 4, 256);
    L->off_scratch = off; off = align_up(off + (size_t)P * (C > L->Cf ? C : L->Cf) * K * stride * 4, 256);
    L->off_reduced = off; off = align_up(off + (size_t)K * stride * 4, 256);
    L->off_contrib = off; off = align_up(off + (size_t)K * 4 + 256, 256);   // + a status word
    L->off_dirty = off; off = align_up(off + (size_t)P * (L->Cf > 0 ? L->Cf : 1) * 4, 256);   // change flags of the row blocks
    L->need_words = 0;
    if (L->Cf > 0 && tc_capable(D, K)) {
        const size_t maxrun = (N / (size_t)P + 1) / (size_t)L->Cf + 2;
        const size_t nw = (maxrun + 127) / 128 + 1;
        if (nw <= (size_t)tc::NEED_WORDS_MAX) L->need_words = (int)nw;     // longer runs: no bounds, every tile is searched
    }
    L->off_bounds = off; off = align_up(off + (L->need_words > 0 ? N * 8 : 0), 256);   // distance bounds of the points
    L->off_drift = off; off = align_up(off + ((size_t)K + 2) * 4, 256);    // drift sums, their maximum's sum, the check's flag word
    L->off_need = off; off = align_up(off + (size_t)P * (L->Cf > 0 ? L->Cf : 1) * (size_t)L->need_words * 4, 256);
    L->off_xnorm = off; off = align_up(off + ((L->Cf > 0 && tc_capable(D, K)) ? N * 4 : 0), 256);   // |x|^2 of every point
    L->off_ar = off; off = align_up(off + ec_allreduce_workspace_bytes(P, (size_t)K * stride, stride), 256);
    L->total = off;
    return true;
}

bool km_bad_shape(size_t N, int D, int K, int P) {
    return N == 0 || D < 1 || D > 128 || (D % 4) != 0 || K < 1 || K > 1024 || P < 1 || P > EC_MAX_RANKS ||
           (size_t)P > N;
}

float km_tau_scale(int D) { return 8.0f * (float)(D + 3) * 5.9604644775390625e-08f; }   // 8 (D+3) 2^-24

template <int D>
int km_fused_launch(ec_kmeans* km, bool partials, const float* centroids, int32_t* labels, cudaStream_t st) {
    if (partials) {
        fused_kernel<D, true><<<(unsigned)(km->P * km->Cf), FU_THREADS, km->fused_smem, st>>>(
            km->points, km->N, km->P, km->Cf, centroids, km->K, labels, km->Cf == 1 ? km->partials : km->scratch,
            km_tau_scale(D));
    } else {
        size_t runs = (km->N + 4 * FU_TILE - 1) / (4 * FU_TILE);
        if (runs > 0x7fffffffull) return EC_ERR_CAPACITY;
        fused_kernel<D, false><<<(unsigned)runs, FU_THREADS, km->fused_assign_smem, st>>>(
            km->points, km->N, 1, (int)runs, centroids, km->K, labels, nullptr, km_tau_scale(D));
    }
    EC_CUDA(cudaGetLastError());
    return EC_OK;
}

template <int D>
int km_tc_launch(ec_kmeans* km, bool partials, const float* centroids, int32_t* labels, cudaStream_t st, bool delta) {
    // 2^-6 + 2^-10: the bf16 search's two candidates are off by less than 2^-7 (|x|^2 + |c|^2) each (derivation at the
    // kernel's use of tau); the 2^-10 on top covers the fp32 accumulation and the split of |c|^2
    const float tau_scale = 0.015625f + 0.0009765625f;
    // the distance bounds describe the context's own labels against its own centroids: an iteration keeps them,
    // a stand-alone call on other arrays leaves them alone
    const bool own = centroids == km->centroids && labels == km->labels && km->bounds != nullptr && km->use_bounds;
    const bool skip = partials && delta && own && km->bounds_valid && km->use_bounds;
    if (skip) {      // which tiles can still change a label: one byte per 32 points
        EC_CUDA(launch_dependent(tc::bounds_check_kernel, (unsigned)(km->P * km->Cf), tc::BC_THREADS, 0, st,
                                 km->N, km->P, km->Cf, km->K, (const int32_t*)labels, (const float2*)km->bounds, (const float*)km->drift,
                                 km->need, km->need_words, km->dirty, reinterpret_cast<uint32_t*>(km->drift) + km->K + 1));
    }
    if (partials) {
        const unsigned gd = (unsigned)(km->P * km->Cf < km->tc_wave_delta ? km->P * km->Cf : km->tc_wave_delta);
        const unsigned gf = (unsigned)(km->P * km->Cf < km->tc_wave_full ? km->P * km->Cf : km->tc_wave_full);
        float* full_out = km->Cf == 1 ? km->partials : km->scratch;
        if (delta && own)
            tc::tc_fused_kernel<D, true, true, true><<<gd, tc::THREADS, km->tc_smem, st>>>(
                km->points, km->N, km->P, km->Cf, centroids, km->K, labels, km->scratch, tau_scale, km->tc_status, km->dirty,
                km->bounds, km->drift, skip ? km->need : nullptr, km->need_words);
        else if (delta)
            tc::tc_fused_kernel<D, true, true, false><<<gd, tc::THREADS, km->tc_smem, st>>>(
                km->points, km->N, km->P, km->Cf, centroids, km->K, labels, km->scratch, tau_scale, km->tc_status, km->dirty,
                nullptr, nullptr, nullptr, 0);
        else if (own)
            tc::tc_fused_kernel<D, true, false, true><<<gf, tc::THREADS, km->tc_smem, st>>>(
                km->points, km->N, km->P, km->Cf, centroids, km->K, labels, full_out, tau_scale, km->tc_status, km->dirty,
                km->bounds, km->drift, nullptr, 0);
        else
            tc::tc_fused_kernel<D, true, false, false><<<gf, tc::THREADS, km->tc_smem, st>>>(
                km->points, km->N, km->P, km->Cf, centroids, km->K, labels, full_out, tau_scale, km->tc_status, km->dirty,
                nullptr, nullptr, nullptr, 0);
    } else {
        size_t runs = (km->N + 2047) / 2048;
        if (runs > 0x7fffffffull) return EC_ERR_CAPACITY;
        tc::tc_fused_kernel<D, false, false, false><<<(unsigned)(runs < (size_t)km->tc_wave_assign ? runs : (size_t)km->tc_wave_assign), tc::THREADS, km->tc_assign_smem, st>>>(
            km->points, km->N, 1, (int)runs, centroids, km->K, labels, nullptr, tau_scale, km->tc_status, nullptr,
            nullptr, nullptr, nullptr, 0);
    }
    EC_CUDA(cudaGetLastError());
    km->skipped = skip;
    if (partials && own) km->bounds_valid = true;       // every tile searched in this launch has fresh bounds, the others kept valid ones
    return EC_OK;
}

// Raises the kernels' shared-memory limit and asks how many blocks of each stay resident on an SM: a launch is
// one wave of resident blocks that work through the runs in turn.
template <int D>
cudaError_t km_tc_attr(ec_kmeans* km) {
    cudaError_t e = cudaFuncSetAttribute(tc::tc_fused_kernel<D, true, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BUDGET);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(tc::tc_fused_kernel<D, true, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BUDGET);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(tc::tc_fused_kernel<D, true, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BUDGET);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(tc::tc_fused_kernel<D, true, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BUDGET);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(tc::tc_fused_kernel<D, false, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BUDGET);
    // Resident blocks per SM, from the kernels' own budgets (the occupancy query depends on the shared-memory
    // carve-out of the moment): 128 threads x 128 registers, shared memory + 1 KB per block, tensor-memory columns.
    auto per_sm = [](size_t smem, uint32_t cols) {
        int n = 65536 / (tc::THREADS * 128);
        const int by_smem = (int)(233472 / (smem + 1024)), by_tmem = (int)(512u / cols);
        if (by_smem < n) n = by_smem;
        if (by_tmem < n) n = by_tmem;
        return n < 1 ? 1 : n;
    };
    km->tc_wave_full = km->tc_wave_delta = km->sms * per_sm(km->tc_smem, tc::tmem_cols_of(D, km->K, true));
    km->tc_wave_assign = km->sms * per_sm(km->tc_assign_smem, tc::tmem_cols_of(D, km->K, false));
    return e;
}

// Shapes the warp-specialised tensor-core kernel covers: a row of D floats is one 64- or 128-byte swizzle span, the
// accumulators of at least two epilogue groups and of two runs fit in tensor memory, row indices fit the copy's int32.
bool ws_capable(size_t N, int D, int K) {
    if (D != 16 && D != 32) return false;
    if (tc::npad_of(K) > 128) return false;
    if (N >= 0x7fffff00ull) return false;
    return ws::plan_of(D, K, true, false).total <= 227 * 1024 && ws::plan_of(D, K, true, false).stages >= 3 &&
           ws::plan_of(D, K, true, true).total <= 227 * 1024;
}

// The tensor map of the points (driver entry point taken through the runtime: the library links no libcuda).
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
bool km_make_point_map(ec_kmeans* km) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres = cudaDriverEntryPointSymbolNotFound;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || fn == nullptr ||
        qres != cudaDriverEntryPointSuccess) {
        cudaGetLastError();
        return false;
    }
    const cuuint64_t dims[2] = {(cuuint64_t)km->D, (cuuint64_t)km->N};
    const cuuint64_t strides[1] = {(cuuint64_t)km->D * 4};
    const cuuint32_t box[2] = {(cuuint32_t)km->D, (cuuint32_t)ws::TILE};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = reinterpret_cast<EncodeTiledFn>(fn)(
        &km->pmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(km->points), dims, strides, box, estr,
        CU_TENSOR_MAP_INTERLEAVE_NONE, km->D == 32 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
        CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

template <int D>
cudaError_t km_ws_attr(ec_kmeans* km) {
    const int full = (int)km->ws_plan.total, asg = (int)km->ws_plan_assign.total;
    cudaError_t e = cudaFuncSetAttribute(ws::ws_fused_kernel<D, true, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(ws::ws_fused_kernel<D, true, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(ws::ws_fused_kernel<D, true, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(ws::ws_fused_kernel<D, true, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(ws::ws_fused_kernel<D, false, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    (void)full; (void)asg;
    return e;
}

template <int D>
int km_ws_launch(ec_kmeans* km, bool partials, const float* centroids, int32_t* labels, cudaStream_t st, bool delta) {
    const bool own = centroids == km->centroids && labels == km->labels && km->bounds != nullptr && km->use_bounds;
    const bool skip = partials && delta && own && km->bounds_valid && km->use_bounds;
    if (skip) {      // which tiles can still change a label: one byte per 32 points
        EC_CUDA(launch_dependent(tc::bounds_check_kernel, (unsigned)(km->P * km->Cf), tc::BC_THREADS, 0, st,
                                 km->N, km->P, km->Cf, km->K, (const int32_t*)labels, (const float2*)km->bounds, (const float*)km->drift,
                                 km->need, km->need_words, km->dirty, reinterpret_cast<uint32_t*>(km->drift) + km->K + 1));
    }
    if (partials) {
        const int runs = km->P * km->Cf;
        const unsigned grid = (unsigned)(runs < km->sms ? runs : km->sms);
        const ws::Plan& plan = delta ? km->ws_plan_delta : km->ws_plan;
        const unsigned thr = (unsigned)ws::threads_of(plan);
        const size_t smem = plan.total;
        float* full_out = km->Cf == 1 ? km->partials : km->scratch;
        if (delta && own)
            EC_CUDA(launch_dependent(ws::ws_fused_kernel<D, true, true, true>, grid, thr, smem, st,
                km->pmap, km->points, (const float*)km->xnorm, km->N, km->P, km->Cf, centroids, km->K, labels, km->scratch, km->tc_status, km->dirty,
                km->bounds, km->drift, skip ? km->need : nullptr, km->need_words));
        else if (delta)
            EC_CUDA(launch_dependent(ws::ws_fused_kernel<D, true, true, false>, grid, thr, smem, st,
                km->pmap, km->points, (const float*)km->xnorm, km->N, km->P, km->Cf, centroids, km->K, labels, km->scratch, km->tc_status, km->dirty,
                nullptr, nullptr, nullptr, 0));
        else if (own)
            EC_CUDA(launch_dependent(ws::ws_fused_kernel<D, true, false, true>, grid, thr, smem, st,
                km->pmap, km->points, (const float*)km->xnorm, km->N, km->P, km->Cf, centroids, km->K, labels, full_out, km->tc_status, km->dirty,
                km->bounds, km->drift, nullptr, 0));
        else
            EC_CUDA(launch_dependent(ws::ws_fused_kernel<D, true, false, false>, grid, thr, smem, st,
                km->pmap, km->points, (const float*)km->xnorm, km->N, km->P, km->Cf, centroids, km->K, labels, full_out, km->tc_status, km->dirty,
                nullptr, nullptr, nullptr, 0));
    } else {
        size_t runs = (km->N + 2047) / 2048;
        if (runs > 0x7fffffffull) return EC_ERR_CAPACITY;
        const unsigned grid = (unsigned)(runs < (size_t)km->sms ? runs : (size_t)km->sms);
        EC_CUDA(launch_dependent(ws::ws_fused_kernel<D, false, false, false>, grid, (unsigned)ws::threads_of(km->ws_plan_assign), km->ws_plan_assign.total, st,
                km->pmap, km->points, (const float*)km->xnorm, km->N, 1, (int)runs, centroids, km->K, labels, nullptr, km->tc_status, nullptr,
            nullptr, nullptr, nullptr, 0));
    }
    EC_CUDA(cudaGetLastError());
    km->skipped = skip;
    if (partials && own) km->bounds_valid = true;       // every tile searched in this launch has fresh bounds, the others kept valid ones
    return EC_OK;
}

int km_fused(ec_kmeans* km, bool partials, const float* centroids, int32_t* labels, cudaStream_t st, bool delta = false) {
    // Automatic choice between the two tensor-core kernels: the warp-specialised one for the assignment alone and for the
    // passes that sum only changes (config 5: 0.109 against 0.136 ms, 5980 against 4851 iterations/s), the register-staged
    // one for a pass that sums every point (0.253-0.268 against 0.313-0.320 ms: there every row has to be converted
    // for the sums GEMM anyway, and its four independent blocks per SM overlap that better than one block's slots do).
    const bool full_pass = partials && !delta;
    if (km->ws_ok && km->path != 1 && km->path != 3 && !(km->path == 0 && full_pass)) {
        switch (km->D) {
            case 16: return km_ws_launch<16>(km, partials, centroids, labels, st, delta);
            case 32: return km_ws_launch<32>(km, partials, centroids, labels, st, delta);
        }
    }
    if (km->tc_ok && km->path != 1) {
        switch (km->D) {
            case 16: return km_tc_launch<16>(km, partials, centroids, labels, st, delta);
            case 32: return km_tc_launch<32>(km, partials, centroids, labels, st, delta);
        }
    }
    switch (km->D) {
        case 8: return km_fused_launch<8>(km, partials, centroids, labels, st);
        case 16: return km_fused_launch<16>(km, partials, centroids, labels, st);
        case 32: return km_fused_launch<32>(km, partials, centroids, labels, st);
        case 64: return km_fused_launch<64>(km, partials, centroids, labels, st);
    }
    return EC_ERR_UNSUPPORTED;
}

template <int D>
cudaError_t km_fused_attr() {
    cudaError_t e = cudaFuncSetAttribute(fused_kernel<D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BUDGET);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(fused_kernel<D, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BUDGET);
    return e;
}

int km_assign(ec_kmeans* km, const float* centroids, int32_t* labels, cudaStream_t st) {
    if (km->Cf > 0) return km_fused(km, false, centroids, labels, st);
    const size_t tiles = (km->N + AS_THREADS - 1) / AS_THREADS;
    const size_t cap = (size_t)km->sms * 8;
    const unsigned grid = (unsigned)(tiles < cap ? tiles : cap);
    switch (km->D) {
#define EC_ASSIGN_CASE(DD)                                                                                   \
    case DD:                                                                                                  \
        assign_kernel<DD><<<grid, AS_THREADS, km->assign_smem, st>>>(km->points, km->N, centroids, km->K, km->kc, labels); \
        break;
        EC_ASSIGN_CASE(4)
        EC_ASSIGN_CASE(8)
        EC_ASSIGN_CASE(16)
        EC_ASSIGN_CASE(32)
        EC_ASSIGN_CASE(64)
#undef EC_ASSIGN_CASE
        default:
            assign_generic_kernel<<<grid, AS_THREADS, km->assign_smem, st>>>(km->points, km->N, km->D, centroids, km->K,
                                                                             km->kc, labels);
    }
    EC_CUDA(cudaGetLastError());
    return EC_OK;
}

int km_partials(ec_kmeans* km, const int32_t* labels, float* partials, cudaStream_t st) {
    float* first = km->C == 1 ? partials : km->scratch;
    partials_kernel<<<(unsigned)(km->P * km->C), PT_THREADS, km->part_smem, st>>>(km->points, labels, km->N, km->D, km->K,
                                                                                  km->P, km->C, km->warps, first);
    EC_CUDA(cudaGetLastError());
    if (km->C > 1) {
        const size_t row = (size_t)km->K * (km->D + 4), total = row * km->P;
        const unsigned grid = (unsigned)((total / (km->D + 4) * 32 + 255) / 256);   // one warp per row
        partials_fold_kernel<<<grid, 256, 0, st>>>(km->scratch, km->C, row, total, partials, km->D + 4);
        EC_CUDA(cudaGetLastError());
    }
    return EC_OK;
}

}  // namespace

extern "C" {

size_t ec_kmeans_workspace_bytes(size_t N, int D, int K, int P) {
    if (km_bad_shape(N, D, K, P)) return 0;
    KmLayout L;
    if (!km_plan(N, D, K, P, sm_count_km(), &L)) return 0;
    return L.total;
}

int ec_kmeans_init(ec_kmeans_t** out, const float* points, size_t N, int D, int K, int P, const float* init_centroids,
                   void* workspace, size_t workspace_bytes) {
    if (!out) return EC_ERR_INVALID;
    *out = nullptr;
    if (!points || !init_centroids || km_bad_shape(N, D, K, P)) return EC_ERR_INVALID;
    if (!aligned16(points)) return EC_ERR_INVALID;
    KmLayout L;
    const int sms = sm_count_km();
    if (!km_plan(N, D, K, P, sms, &L)) return EC_ERR_CAPACITY;
    if (workspace && (workspace_bytes < L.total || (reinterpret_cast<uintptr_t>(workspace) & 255u))) return EC_ERR_CAPACITY;
    ec_kmeans* km = new (std::nothrow) ec_kmeans();
    if (!km) return EC_ERR_INVALID;
    km->points = points; km->N = N; km->D = D; km->K = K; km->P = P;
    km->own_ws = workspace == nullptr;
    km->ws = workspace;
    km->ar = nullptr;
    if (km->own_ws) {
        cudaError_t e = cudaMalloc(&km->ws, L.total);
        if (e != cudaSuccess) { delete km; return cuda_fail(e); }
    }
    char* base = reinterpret_cast<char*>(km->ws);
    km->centroids = reinterpret_cast<float*>(base + L.off_centroids);
    km->labels = reinterpret_cast<int32_t*>(base + L.off_labels);
    km->partials = reinterpret_cast<float*>(base + L.off_partials);
    km->scratch = reinterpret_cast<float*>(base + L.off_scratch);
    km->reduced = reinterpret_cast<float*>(base + L.off_reduced);
    km->contrib = reinterpret_cast<uint32_t*>(base + L.off_contrib);
    km->ar_ws = base + L.off_ar;
    km->sms = sms; km->C = L.C; km->warps = L.warps;
    km->Cf = L.Cf;
    km->fused_smem = fused_smem_floats(D, K, true) * 4;
    km->fused_assign_smem = fused_smem_floats(D, K, false) * 4;
    km->tc_ok = km->Cf > 0 && tc_capable(D, K);
    km->path = 0;
    km->state_valid = false;
    km->since_full = 0;
    km->refresh = KM_REFRESH;
    km->tc_smem = tc::layout_of(D, K, true).total;
    km->tc_assign_smem = tc::layout_of(D, K, false).total;
    km->tc_status = reinterpret_cast<uint32_t*>(base + L.off_contrib + align_up((size_t)K * 4, 256));
    km->dirty = reinterpret_cast<uint32_t*>(base + L.off_dirty);
    km->bounds = km->tc_ok && L.need_words > 0 ? reinterpret_cast<float2*>(base + L.off_bounds) : nullptr;
    km->need = reinterpret_cast<uint32_t*>(base + L.off_need);
    km->xnorm = km->tc_ok ? reinterpret_cast<float*>(base + L.off_xnorm) : nullptr;
    km->need_words = L.need_words;
    km->drift = reinterpret_cast<float*>(base + L.off_drift);
    km->bounds_valid = false;
    km->use_bounds = true;
    // centroid chunk for the assignment: as many as fit in 64 KB, all of them if possible
    int kc = (int)((64 * 1024) / ((size_t)D * 4));
    if (kc > K) kc = K;
    if (kc > 1) kc &= ~1;
    if (kc < 1) kc = 1;
    km->kc = kc;
    km->assign_smem = (size_t)kc * D * 4;
    km->part_smem = (size_t)L.warps * ((size_t)K * D + K) * 4;
    const size_t stride = (size_t)D + 4;
    int rc = EC_OK;
    cudaError_t e = cudaSuccess;
    // The dynamic shared memory limit is a property of the kernel, not of this context: always raise it to
    // the largest size any shape can ask for, so that contexts of different shapes do not lower each other's.
    switch (D) {
        case 4: e = cudaFuncSetAttribute(assign_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ASSIGN_SMEM_MAX); break;
        case 8: e = cudaFuncSetAttribute(assign_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ASSIGN_SMEM_MAX); break;
        case 16: e = cudaFuncSetAttribute(assign_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ASSIGN_SMEM_MAX); break;
        case 32: e = cudaFuncSetAttribute(assign_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ASSIGN_SMEM_MAX); break;
        case 64: e = cudaFuncSetAttribute(assign_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ASSIGN_SMEM_MAX); break;
        default: e = cudaFuncSetAttribute(assign_generic_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ASSIGN_SMEM_MAX);
    }
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(partials_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BUDGET);
    if (e == cudaSuccess && km->Cf > 0)
        e = D == 8 ? km_fused_attr<8>() : D == 16 ? km_fused_attr<16>() : D == 32 ? km_fused_attr<32>() : km_fused_attr<64>();
    if (e == cudaSuccess && km->tc_ok)
        e = D == 16 ? km_tc_attr<16>(km) : km_tc_attr<32>(km);
    km->ws_ok = km->tc_ok && ws_capable(N, D, K) && km_make_point_map(km);
    if (km->ws_ok) {
        km->ws_plan = ws::plan_of(D, K, true, false);
        km->ws_plan_delta = ws::plan_of(D, K, true, true);
        km->ws_plan_assign = ws::plan_of(D, K, false, false);
        if (e == cudaSuccess) e = D == 16 ? km_ws_attr<16>(km) : km_ws_attr<32>(km);
    }
    if (e == cudaSuccess) e = cudaMemsetAsync(km->tc_status, 0, 4, 0);
    if (e == cudaSuccess) e = cudaMemsetAsync(km->drift, 0, ((size_t)K + 2) * 4, 0);
    if (e == cudaSuccess && km->xnorm != nullptr) {
        point_norm_kernel<<<(unsigned)(sms * 8), 256>>>(points, N, D, km->xnorm);
        e = cudaGetLastError();
    }
    if (e == cudaSuccess) e = cudaMemcpyAsync(km->centroids, init_centroids, (size_t)K * D * 4, cudaMemcpyDeviceToDevice, 0);
    if (e == cudaSuccess) e = cudaStreamSynchronize(0);
    if (e != cudaSuccess) rc = cuda_fail(e);
    if (rc == EC_OK)
        rc = ec_allreduce_init(&km->ar, P, (size_t)K * stride, EC_F32, EC_SUM, stride, EC_ORDER_FIXED, km->ar_ws,
                               ec_allreduce_workspace_bytes(P, (size_t)K * stride, stride));
    if (rc != EC_OK) {
        if (km->own_ws) cudaFree(km->ws);
        delete km;
        return rc;
    }
    for (int r = 0; r < P; ++r) km->bufs[r] = km->partials + (size_t)r * K * stride;
    allreduce_set_dependent_launch(km->ar, true);        // the small allreduce follows the fold kernel closely
    *out = km;
    return EC_OK;
}

int ec_kmeans_assign(ec_kmeans_t* km, const float* centroids, int32_t* labels, ec_stream_t stream) {
    if (!km || !centroids || !labels || !aligned16(centroids)) return EC_ERR_INVALID;
    return km_assign(km, centroids, labels, stream);
}

int ec_kmeans_partials(ec_kmeans_t* km, const int32_t* labels, float* partials, ec_stream_t stream) {
    if (!km || !labels || !partials) return EC_ERR_INVALID;
    return km_partials(km, labels, partials, stream);
}

namespace {
int km_iterate_rounds(ec_kmeans_t* km, const uint64_t* const* masks, int rounds, ec_stream_t stream);
}

int ec_kmeans_iterate(ec_kmeans_t* km, const uint64_t* arrival_mask, ec_stream_t stream) {
    if (!km) return EC_ERR_INVALID;
    const uint64_t* one[1] = {arrival_mask};
    return km_iterate_rounds(km, one, 1, stream);
}

int ec_kmeans_iterate_rounds(ec_kmeans_t* km, const uint64_t* const* arrival_masks, int rounds, ec_stream_t stream) {
    if (!km || !arrival_masks || rounds < 1 || rounds > 64) return EC_ERR_INVALID;
    return km_iterate_rounds(km, arrival_masks, rounds, stream);
}

namespace {
int km_iterate_rounds(ec_kmeans_t* km, const uint64_t* const* masks, int rounds, ec_stream_t stream) {
    int rc;
    if (km->Cf > 0) {
        // assignment and per-block partial sums in one pass over the points, then the rows of a rank in order
        // On the tensor-core path only the changes since the last iteration are summed (labels and per-rank sums
        // are kept between iterations); every KM_REFRESH-th iteration sums everything afresh, which bounds the
        // rounding that the running sums collect.
        const bool delta = km->tc_ok && km->path != 1 && km->state_valid && km->since_full + 1 < km->refresh;
        rc = km_fused(km, true, km->centroids, km->labels, stream, delta);
        if (rc != EC_OK) return rc;
        if (km->Cf > 1 || delta) {
            const size_t row = (size_t)km->K * (km->D + 4), total = row * km->P;
            EC_CUDA(launch_dependent(partials_fold_kernel, (unsigned)(((size_t)km->P * km->K * 32 + 255) / 256), 256, 0, stream,
                                     (const float*)km->scratch, km->Cf, row, total, km->partials, km->D + 4, delta ? 1 : 0,
                                     (const uint32_t*)km->dirty,
                                     delta && km->skipped ? reinterpret_cast<const uint32_t*>(km->drift) + km->K + 1 : (const uint32_t*)nullptr));
        }
        km->state_valid = true;
        km->since_full = delta ? km->since_full + 1 : 0;
    } else {
        rc = km_assign(km, km->centroids, km->labels, stream);
        if (rc != EC_OK) return rc;
        rc = km_partials(km, km->labels, km->partials, stream);
        if (rc != EC_OK) return rc;
    }
    rc = ec_allreduce_reset(km->ar, stream);
    if (rc != EC_OK) return rc;
    const size_t stride = (size_t)km->D + 4;
    for (int t = 0; t < rounds; ++t) {     // one epoch: the first round builds the partial result, the others fold late rows in
        rc = ec_allreduce_apply(km->ar, km->bufs, km->P, (size_t)km->K * stride, EC_F32, EC_SUM, stride, masks[t],
                                km->reduced, km->contrib, stream);
        if (rc != EC_OK) return rc;
    }
    if (km->bounds != nullptr && km->use_bounds) {   // (bounds switched on again later are all renewed first: no drift sums needed meanwhile)
        EC_CUDA(launch_dependent(update_drift_kernel, 1, UD_THREADS, 0, stream, (const float*)km->reduced, km->D, km->K, km->centroids, km->drift));
    } else {
        const int total = km->K * km->D;
        EC_CUDA(launch_dependent(update_kernel, (unsigned)((total + 255) / 256), 256, 0, stream, (const float*)km->reduced, km->D, km->K, km->centroids));
    }
    EC_CUDA(cudaGetLastError());
    return EC_OK;
}
}  // namespace

int ec_kmeans_set_centroids(ec_kmeans_t* km, const float* centroids, ec_stream_t stream) {
    if (!km || !centroids) return EC_ERR_INVALID;
    EC_CUDA(cudaMemcpyAsync(km->centroids, centroids, (size_t)km->K * km->D * 4, cudaMemcpyDeviceToDevice, stream));
    km->bounds_valid = false;       // the centroids moved without the drift sums knowing: the next iteration searches every tile
    return EC_OK;
}

int ec_kmeans_get(ec_kmeans_t* km, float* centroids, int32_t* labels, float* reduced, uint32_t* contrib_count,
                  ec_stream_t stream) {
    if (!km) return EC_ERR_INVALID;
    if (centroids) EC_CUDA(cudaMemcpyAsync(centroids, km->centroids, (size_t)km->K * km->D * 4, cudaMemcpyDeviceToDevice, stream));
    if (labels) EC_CUDA(cudaMemcpyAsync(labels, km->labels, km->N * 4, cudaMemcpyDeviceToDevice, stream));
    if (reduced) EC_CUDA(cudaMemcpyAsync(reduced, km->reduced, (size_t)km->K * (km->D + 4) * 4, cudaMemcpyDeviceToDevice, stream));
    if (contrib_count) EC_CUDA(cudaMemcpyAsync(contrib_count, km->contrib, (size_t)km->K * 4, cudaMemcpyDeviceToDevice, stream));
    return EC_OK;
}

int ec_kmeans_set_refresh(ec_kmeans_t* km, int every) {
    if (!km || every < 1) return EC_ERR_INVALID;
    km->refresh = every;
    km->state_valid = false;        // the next iteration sums everything afresh
    return EC_OK;
}

int ec_kmeans_set_bounds(ec_kmeans_t* km, int enable) {
    if (!km) return EC_ERR_INVALID;
    km->use_bounds = enable != 0;
    km->bounds_valid = false;       // kept only while they are in use: the next iteration searches every tile and renews them
    return EC_OK;
}

int ec_kmeans_set_path(ec_kmeans_t* km, int path) {
    if (!km || path < 0 || path > 3) return EC_ERR_INVALID;
    if ((path == 2 || path == 3) && !km->tc_ok) return EC_ERR_UNSUPPORTED;
    if (path == 1 && km->Cf == 0) return EC_ERR_UNSUPPORTED;
    km->path = path;
    km->state_valid = false;        // the next iteration sums everything afresh
    return EC_OK;
}

int ec_kmeans_tc_status(ec_kmeans_t* km, uint32_t* device_out, ec_stream_t stream) {
    if (!km || !device_out) return EC_ERR_INVALID;
    EC_CUDA(cudaMemcpyAsync(device_out, km->tc_status, 4, cudaMemcpyDeviceToDevice, stream));
    return EC_OK;
}

int ec_kmeans_destroy(ec_kmeans_t* km) {
    if (!km) return EC_ERR_INVALID;
    int rc = EC_OK;
    if (km->ar) ec_allreduce_destroy(km->ar);
    if (km->own_ws && km->ws) {
        cudaError_t e = cudaFree(km->ws);
        if (e != cudaSuccess) rc = cuda_fail(e);
    }
    delete km;
    return rc;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// Per-rank partial sums for callers that must not allocate device memory
// ---------------------------------------------------------------------------------------------
// Same two kernels as ec_kmeans_partials, but the per-block partial sums go to a fixed array that
// is part of the library image instead of a workspace.  Every GPU that loads the library carries
// these 8 MiB until the process exits, whether or not the entry point is ever called.
namespace {

constexpr size_t STATIC_SCRATCH_BYTES = 8u << 20;
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
struct StaticDeviceState {
    bool ready;
    float* scratch;   // device address of g_static_scratch on that device
    int sms;
};
StaticDeviceState g_static_state[MAX_DEVICES];   // host side, indexed by device ordinal; zero-initialised
std::mutex g_static_mutex;                        // host threads making their first calls at the same time take turns

// Once per device, with that device current.  In host code `g_static_scratch` is only a handle of
// the symbol, not an address the GPU understands: the device address has to be asked for.
int static_setup(int dev, StaticDeviceState** out) {
    if (dev < 0 || dev >= MAX_DEVICES) return EC_ERR_CAPACITY;
    StaticDeviceState* st = &g_static_state[dev];
    std::lock_guard<std::mutex> guard(g_static_mutex);
    if (!st->ready) {
        void* addr = nullptr;
        EC_CUDA(cudaGetSymbolAddress(&addr, g_static_scratch));
        int sms = 0;
        EC_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        EC_CUDA(cudaFuncSetAttribute(partials_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BUDGET));
        st->scratch = reinterpret_cast<float*>(addr);
        st->sms = sms > 0 ? sms : 148;
        st->ready = true;
    }
    *out = st;
    return EC_OK;
}

}  // namespace

extern "C" int ec_kmeans_partials_static(const float* points, const int32_t* labels, size_t N, int D, int K, int P,
                                         float* partials, ec_stream_t stream) {
    if (!points || !labels || !partials || km_bad_shape(N, D, K, P)) return EC_ERR_INVALID;
    int dev = 0;
    EC_CUDA(cudaGetDevice(&dev));
    StaticDeviceState* st = nullptr;
    const int rc = static_setup(dev, &st);
    if (rc != EC_OK) return rc;
    KmLayout L;
    if (!km_plan(N, D, K, P, st->sms, &L)) return EC_ERR_CAPACITY;
    const size_t row = (size_t)K * ((size_t)D + 4);
    if (L.C > 1 && (size_t)P * L.C * row * sizeof(float) > STATIC_SCRATCH_BYTES) return EC_ERR_CAPACITY;
    const size_t smem = (size_t)L.warps * ((size_t)K * D + K) * 4;
    // Every element of the scratch that the fold reads was written by the first kernel of this
    // same call, so nothing left over from an earlier call can leak in and nothing needs clearing.
    float* first = L.C == 1 ? partials : st->scratch;
    partials_kernel<<<(unsigned)(P * L.C), PT_THREADS, smem, stream>>>(points, labels, N, D, K, P, L.C, L.warps, first);
    EC_CUDA(cudaGetLastError());
    if (L.C > 1) {
        const size_t total = row * P;
        partials_fold_kernel<<<(unsigned)(((size_t)P * K * 32 + 255) / 256), 256, 0, stream>>>(st->scratch, L.C, row, total, partials, D + 4);
        EC_CUDA(cudaGetLastError());
    }
    return EC_OK;
}
