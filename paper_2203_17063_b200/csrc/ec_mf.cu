// Matrix factorisation trained by gradient steps whose item gradients are combined by the
// stale-synchronous allreduce (the experiment of Sec. V: allreduce_SSP inside an ML solver).
//
// r_ui ~ <p_u, q_i>.  Rank r owns a contiguous block of users with all their ratings, so user factors
// are updated locally; the item factors are shared, and every rank contributes the gradient
// G_r[i] = sum over its ratings of e_ui * p_u.  The P gradients live as rank buffers in device memory
// with one logical clock per (item segment, rank); an iteration recomputes only the contributions that
// are delivered fresh (or have become too stale: Algorithm 1's wait), reduces all buffers with
// ec_allreduce_ssp_apply and takes the step.  One warp owns one row (an item of one rank, or a user):
// it walks the row's ratings in storage order, four groups of eight lanes taking one rating each with
// the factor vector spread over the group's lanes, so every sum has a fixed shape and results repeat bit
// for bit from run to run.

#include <new>

#include "ec_common.cuh"

namespace ec {
namespace {

constexpr int MF_THREADS = 256;
constexpr int MF_WARPS = MF_THREADS / 32;
#ifndef EC_MF_INFLIGHT
#define EC_MF_INFLIGHT 4     // measured: 1, 2, 4, 8 in flight give 2363, 2389, 2507, 1572 iterations per second
#endif
constexpr int MF_INFLIGHT = EC_MF_INFLIGHT;   // ratings a group of eight lanes keeps in flight
#ifndef EC_MF_ROWS
#define EC_MF_ROWS 1         // measured: 1, 2, 4, 8 rows per warp give 2680, 2161, 2011, 1741 iterations per second
#endif
constexpr int MF_ROWS = EC_MF_ROWS;           // consecutive rows a warp works through (at most 32)

struct MfArgs {
    const int64_t* user_ptr; const int32_t* user_item; const float* user_val;
    const int64_t* rank_item_ptr; const int32_t* item_user; const float* item_val;
    float* pu; float* qi; float* grad; const float* reduced;
    uint32_t* notif_clock; uint8_t* refreshed; const uint64_t* refresh;
    double* sse_partial; double* sse;
    size_t seg_rows, S;
    int U, I, P, W;
    uint32_t clock, min_ok;
    float lr, lam;
    int sse_blocks;
};

// which contributions are recomputed in this iteration, and their new clocks
__global__ void mf_decide_kernel(const MfArgs a) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= a.S * (size_t)a.P) return;
    const size_t s = i / (size_t)a.P;
    const int r = (int)(i - s * (size_t)a.P);
    bool want = true;
    if (a.refresh != nullptr) want = (a.refresh[s * (size_t)a.W + (r >> 6)] >> (r & 63)) & 1ull;
    const uint32_t c = a.notif_clock[i];
    const bool fresh = want || c == 0u || c < a.min_ok;      // never delivered, or too stale: it is waited for
    a.refreshed[i] = fresh ? 1 : 0;
    if (fresh) a.notif_clock[i] = a.clock;
}

// A warp works through MF_ROWS consecutive rows (one by default).  SIDE 0: row = (rank r, item i), other = users,
// writes G_r[i].  SIDE 1: row = user u, other = items, takes the user step in place and adds up e^2.
// Rows are short (tens of ratings), so a row is a chain of dependent loads (extent -> ratings -> factor rows).
// With several rows per warp the extents of all of them are read at once and the first ratings and the factor
// vector of the next row while the current one is computed; that measured slower than one row per warp and
// more warps, so it is off.
// The warp works as four groups of eight lanes: a group takes one rating at a time (ratings t, t+4, t+8, ... of
// the row go to group t mod 4), each of its lanes holds V = k/8 entries of the factor vectors, so one 128-bit
// load per lane fetches the 128-byte factor row of the rating and the inner product needs three shuffle steps.
// The four partial gradients are added at the end of the row ((g0+g1)+(g2+g3)): a fixed shape, the same bits
// every run.  V4 = float4 per lane (k = 32 * V4).
template <int V4, int SIDE>
__global__ void __launch_bounds__(MF_THREADS) mf_row_kernel(const MfArgs a) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int grp = lane >> 3, sub = lane & 7;
    constexpr int k = 32 * V4;
    const size_t rows = SIDE == 0 ? (size_t)a.P * a.I : (size_t)a.U;
    const size_t first = ((size_t)blockIdx.x * MF_WARPS + wid) * MF_ROWS;      // the warp's rows: first .. first + MF_ROWS - 1
    const int32_t* idx = SIDE == 0 ? a.item_user : a.user_item;
    const float* val = SIDE == 0 ? a.item_val : a.user_val;
    const float* own = SIDE == 0 ? a.qi : a.pu;          // the rows' factors
    const float* oth = SIDE == 0 ? a.pu : a.qi;          // the factors their ratings point at
    __shared__ float s_sse[MF_WARPS];
    float sse = 0.0f;
    // Lane l < MF_ROWS looks up row first + l (its extent in the rating arrays, whether it is to be computed), so
    // the warp pays the latency of these dependent loads once for all its rows.
    long long l_beg = 0, l_end = 0, l_self = 0;
    int l_r = 0, l_active = 0;
    if (lane < MF_ROWS && first + lane < rows) {
        const size_t row = first + lane;
        size_t self = row;                       // index of the row's own factor vector
        bool active = true;
        if (SIDE == 0) {
            l_r = (int)(row / (size_t)a.I);
            self = row - (size_t)l_r * a.I;
            active = a.refreshed[(self / a.seg_rows) * (size_t)a.P + l_r] != 0;
        }
        l_self = (long long)self;
        l_active = active ? 1 : 0;
        // the extent is read whether or not the row is recomputed: the two loads then do not wait for the flag
        const int64_t* ptr = SIDE == 0 ? a.rank_item_ptr + (size_t)l_r * (a.I + 1) + self : a.user_ptr + self;
        l_beg = ptr[0];
        l_end = ptr[1];
    }
    // The first 32 ratings and the factor vector of the next row are fetched while the current row is computed.
    int nxt_i = 0;
    float nxt_v = 0.0f;
    float4 nxt_mine[V4];
    auto prefetch = [&](int rr) {
        const long long beg = __shfl_sync(0xffffffffu, l_beg, rr), end = __shfl_sync(0xffffffffu, l_end, rr);
        const long long self = __shfl_sync(0xffffffffu, l_self, rr);
        const int active = __shfl_sync(0xffffffffu, l_active, rr);
        nxt_i = 0;
        nxt_v = 0.0f;
        if (active) {
            if (beg + lane < end) {
                nxt_i = idx[beg + lane];
                nxt_v = val[beg + lane];
            }
#pragma unroll
            for (int c = 0; c < V4; ++c) nxt_mine[c] = *reinterpret_cast<const float4*>(own + (size_t)self * k + c * 32 + sub * 4);
        }
    };
    prefetch(0);
#pragma unroll 1
    for (int rr = 0; rr < MF_ROWS; ++rr) {
        const long long beg = __shfl_sync(0xffffffffu, l_beg, rr), end = __shfl_sync(0xffffffffu, l_end, rr);
        const size_t self = (size_t)__shfl_sync(0xffffffffu, l_self, rr);
        const int r = __shfl_sync(0xffffffffu, l_r, rr);
        const bool active = __shfl_sync(0xffffffffu, l_active, rr) != 0;
        int my_i = nxt_i;
        float my_v = nxt_v;
        // lane `sub` of every group holds entries [c*32 + sub*4, +4) of a factor vector, c < V4
        float4 mine[V4], g[V4];
#pragma unroll
        for (int c = 0; c < V4; ++c) {
            mine[c] = nxt_mine[c];
            g[c] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        }
        if (rr + 1 < MF_ROWS) prefetch(rr + 1);
        if (!active) continue;                   // warp-uniform: a row that is not recomputed, or past the last one
        for (long long j0 = beg; j0 < end; j0 += 32) {
            const int cnt = end - j0 < 32 ? (int)(end - j0) : 32;
            if (j0 != beg) {
                my_i = lane < cnt ? idx[j0 + lane] : 0;
                my_v = lane < cnt ? val[j0 + lane] : 0.0f;
            }
            for (int t0 = 0; t0 < cnt; t0 += 4 * MF_INFLIGHT) {   // MF_INFLIGHT ratings per group in flight
                float4 x[MF_INFLIGHT][V4];
                float dot[MF_INFLIGHT], v[MF_INFLIGHT];
                bool ok[MF_INFLIGHT];
#pragma unroll
                for (int h = 0; h < MF_INFLIGHT; ++h) {
                    const int t = t0 + h * 4 + grp;
                    ok[h] = t < cnt;
                    const int o = __shfl_sync(0xffffffffu, my_i, t & 31);
                    v[h] = __shfl_sync(0xffffffffu, my_v, t & 31);
                    dot[h] = 0.0f;
#pragma unroll
                    for (int c = 0; c < V4; ++c) {
                        x[h][c] = ok[h] ? __ldg(reinterpret_cast<const float4*>(oth + (size_t)o * k + c * 32 + sub * 4))
                                        : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                        dot[h] = fmaf(x[h][c].x, mine[c].x, dot[h]);
                        dot[h] = fmaf(x[h][c].y, mine[c].y, dot[h]);
                        dot[h] = fmaf(x[h][c].z, mine[c].z, dot[h]);
                        dot[h] = fmaf(x[h][c].w, mine[c].w, dot[h]);
                    }
                }
#pragma unroll
                for (int d = 1; d < 8; d <<= 1) {
#pragma unroll
                    for (int h = 0; h < MF_INFLIGHT; ++h) dot[h] += __shfl_xor_sync(0xffffffffu, dot[h], d);
                }
#pragma unroll
                for (int h = 0; h < MF_INFLIGHT; ++h) {
                    const float e = ok[h] ? v[h] - dot[h] : 0.0f;
#pragma unroll
                    for (int c = 0; c < V4; ++c) {
                        g[c].x = fmaf(e, x[h][c].x, g[c].x);
                        g[c].y = fmaf(e, x[h][c].y, g[c].y);
                        g[c].z = fmaf(e, x[h][c].z, g[c].z);
                        g[c].w = fmaf(e, x[h][c].w, g[c].w);
                    }
                    if (SIDE == 1) sse = fmaf(e, e, sse);
                }
            }
        }
        // the four groups' partial sums: (g0 + g1) + (g2 + g3), the same in every lane
#pragma unroll
        for (int d = 8; d < 32; d <<= 1) {
#pragma unroll
            for (int c = 0; c < V4; ++c) {
                g[c].x += __shfl_xor_sync(0xffffffffu, g[c].x, d);
                g[c].y += __shfl_xor_sync(0xffffffffu, g[c].y, d);
                g[c].z += __shfl_xor_sync(0xffffffffu, g[c].z, d);
                g[c].w += __shfl_xor_sync(0xffffffffu, g[c].w, d);
            }
        }
        if (grp == 0) {
#pragma unroll
            for (int c = 0; c < V4; ++c) {
                if (SIDE == 0) {
                    *reinterpret_cast<float4*>(a.grad + ((size_t)r * a.I + self) * k + c * 32 + sub * 4) = g[c];
                } else {
                    float4 p = mine[c];
                    p.x += a.lr * (g[c].x - a.lam * p.x);
                    p.y += a.lr * (g[c].y - a.lam * p.y);
                    p.z += a.lr * (g[c].z - a.lam * p.z);
                    p.w += a.lr * (g[c].w - a.lam * p.w);
                    *reinterpret_cast<float4*>(a.pu + self * k + c * 32 + sub * 4) = p;
                }
            }
        }
    }
    if (SIDE == 1) {
        // e^2 of the warp's rows: every group added up its own ratings; (s0 + s1) + (s2 + s3), then the warps in order
#pragma unroll
        for (int d = 8; d < 32; d <<= 1) sse += __shfl_xor_sync(0xffffffffu, sse, d);
        if (lane == 0) s_sse[wid] = sse;
        __syncthreads();
        if (threadIdx.x == 0) {
            double t = 0.0;
            for (int w = 0; w < MF_WARPS; ++w) t += (double)s_sse[w];
            a.sse_partial[blockIdx.x] = t;
        }
    }
}

// q_i += lr * (R_i - lam * q_i); the first block also adds up the per-block error sums in a fixed order
__global__ void __launch_bounds__(MF_THREADS) mf_item_step_kernel(const MfArgs a, size_t n) {
    const size_t i = (size_t)blockIdx.x * MF_THREADS + threadIdx.x;
    if (i < n) {
        const float q = a.qi[i];
        a.qi[i] = q + a.lr * (a.reduced[i] - a.lam * q);
    }
    if (blockIdx.x == 0) {
        __shared__ double s[MF_THREADS];
        double t = 0.0;
        for (int b = threadIdx.x; b < a.sse_blocks; b += MF_THREADS) t += a.sse_partial[b];
        s[threadIdx.x] = t;
        __syncthreads();
        for (int d = MF_THREADS / 2; d > 0; d >>= 1) {
            if (threadIdx.x < d) s[threadIdx.x] += s[threadIdx.x + d];
            __syncthreads();
        }
        if (threadIdx.x == 0) *a.sse = s[0];
    }
}

struct MfLayout {
    size_t pu, qi, grad, reduced, notif, seg_clock, count, wait, refreshed, sse_partial, sse, ar, total;
    int sse_blocks;
};

bool mf_plan(int U, int I, int k, int P, size_t seg_rows, MfLayout* L) {
    if (U < 1 || I < 1 || P < 1 || P > EC_MAX_RANKS || P > U || seg_rows == 0 || (k != 32 && k != 64)) return false;
    const size_t S = ((size_t)I + seg_rows - 1) / seg_rows;
    size_t off = 0;
    L->pu = off; off = align_up(off + (size_t)U * k * 4, 256);
    L->qi = off; off = align_up(off + (size_t)I * k * 4, 256);
    L->grad = off; off = align_up(off + (size_t)P * I * k * 4, 256);
    L->reduced = off; off = align_up(off + (size_t)I * k * 4, 256);
    L->notif = off; off = align_up(off + S * P * 4, 256);
    L->seg_clock = off; off = align_up(off + S * 4, 256);
    L->count = off; off = align_up(off + S * 4, 256);
    L->wait = off; off = align_up(off + S * 4, 256);
    L->refreshed = off; off = align_up(off + S * P, 256);
    L->sse_blocks = (U + MF_WARPS * MF_ROWS - 1) / (MF_WARPS * MF_ROWS);
    L->sse_partial = off; off = align_up(off + (size_t)L->sse_blocks * 8, 256);
    L->sse = off; off = align_up(off + 8, 256);
    L->ar = off; off = align_up(off + ec_allreduce_workspace_bytes(P, (size_t)I * k, seg_rows * k), 256);
    L->total = off;
    return true;
}

}  // namespace
}  // namespace ec

using namespace ec;

struct ec_mf {
    MfArgs a;
    MfLayout L;
    int k;
    void* ws;
    bool own_ws;
    ec_ctx_t* ar;
    uint32_t* seg_clock; uint32_t* count; uint32_t* wait;
    const void* bufs[EC_MAX_RANKS];
};

extern "C" {

size_t ec_mf_workspace_bytes(int n_users, int n_items, int k, int P, size_t segment_rows) {
    MfLayout L;
    if (!mf_plan(n_users, n_items, k, P, segment_rows, &L)) return 0;
    return L.total;
}

int ec_mf_init(ec_mf_t** out, int n_users, int n_items, int k, int P, const int64_t* user_ptr, const int32_t* user_item,
               const float* user_val, const int64_t* rank_item_ptr, const int32_t* item_user, const float* item_val,
               const float* user_factors, const float* item_factors, float lr, float lambda, size_t segment_rows,
               void* workspace, size_t workspace_bytes) {
    if (!out) return EC_ERR_INVALID;
    *out = nullptr;
    if (!user_ptr || !user_item || !user_val || !rank_item_ptr || !item_user || !item_val || !user_factors || !item_factors)
        return EC_ERR_INVALID;
    if (n_users < 1 || n_items < 1 || P < 1 || P > EC_MAX_RANKS || P > n_users || segment_rows == 0) return EC_ERR_INVALID;
    if (k != 32 && k != 64) return EC_ERR_UNSUPPORTED;
    MfLayout L;
    if (!mf_plan(n_users, n_items, k, P, segment_rows, &L)) return EC_ERR_INVALID;
    if (workspace && (workspace_bytes < L.total || (reinterpret_cast<uintptr_t>(workspace) & 255u))) return EC_ERR_CAPACITY;
    ec_mf* m = new (std::nothrow) ec_mf();
    if (!m) return EC_ERR_INVALID;
    m->own_ws = workspace == nullptr;
    m->ws = workspace;
    if (m->own_ws) {
        cudaError_t e = cudaMalloc(&m->ws, L.total);
        if (e != cudaSuccess) { delete m; return cuda_fail(e); }
    }
    char* base = static_cast<char*>(m->ws);
    m->L = L;
    m->k = k;
    MfArgs& a = m->a;
    a.user_ptr = user_ptr; a.user_item = user_item; a.user_val = user_val;
    a.rank_item_ptr = rank_item_ptr; a.item_user = item_user; a.item_val = item_val;
    a.pu = reinterpret_cast<float*>(base + L.pu);
    a.qi = reinterpret_cast<float*>(base + L.qi);
    a.grad = reinterpret_cast<float*>(base + L.grad);
    a.reduced = reinterpret_cast<float*>(base + L.reduced);
    a.notif_clock = reinterpret_cast<uint32_t*>(base + L.notif);
    a.refreshed = reinterpret_cast<uint8_t*>(base + L.refreshed);
    a.refresh = nullptr;
    a.sse_partial = reinterpret_cast<double*>(base + L.sse_partial);
    a.sse = reinterpret_cast<double*>(base + L.sse);
    a.seg_rows = segment_rows;
    a.S = ((size_t)n_items + segment_rows - 1) / segment_rows;
    a.U = n_users; a.I = n_items; a.P = P; a.W = (P + 63) / 64;
    a.clock = 0; a.min_ok = 1;
    a.lr = lr; a.lam = lambda;
    a.sse_blocks = L.sse_blocks;
    m->seg_clock = reinterpret_cast<uint32_t*>(base + L.seg_clock);
    m->count = reinterpret_cast<uint32_t*>(base + L.count);
    m->wait = reinterpret_cast<uint32_t*>(base + L.wait);
    for (int r = 0; r < P; ++r) m->bufs[r] = a.grad + (size_t)r * n_items * k;
    // clocks 0 = nothing delivered yet; gradients and sums start at zero
    cudaError_t e = cudaMemsetAsync(base + L.grad, 0, L.ar - L.grad, 0);
    if (e == cudaSuccess) e = cudaMemcpyAsync(a.pu, user_factors, (size_t)n_users * k * 4, cudaMemcpyDeviceToDevice, 0);
    if (e == cudaSuccess) e = cudaMemcpyAsync(a.qi, item_factors, (size_t)n_items * k * 4, cudaMemcpyDeviceToDevice, 0);
    if (e == cudaSuccess) e = cudaStreamSynchronize(0);
    int rc = e == cudaSuccess ? EC_OK : cuda_fail(e);
    if (rc == EC_OK)
        rc = ec_allreduce_init(&m->ar, P, (size_t)n_items * k, EC_F32, EC_SUM, segment_rows * k, EC_ORDER_FIXED, base + L.ar,
                               L.total - L.ar);
    if (rc != EC_OK) {
        if (m->own_ws) cudaFree(m->ws);
        delete m;
        return rc;
    }
    *out = m;
    return EC_OK;
}

int ec_mf_iterate(ec_mf_t* m, const uint64_t* refresh_mask, uint32_t slack, ec_stream_t stream) {
    if (!m) return EC_ERR_INVALID;
    MfArgs& a = m->a;
    a.clock += 1;
    a.min_ok = a.clock > slack ? a.clock - slack : 1u;
    a.refresh = refresh_mask;
    const size_t pairs = a.S * (size_t)a.P;
    mf_decide_kernel<<<(unsigned)((pairs + 255) / 256), 256, 0, stream>>>(a);
    const size_t item_rows = (size_t)a.P * a.I;
    const unsigned gi = (unsigned)((item_rows + MF_WARPS * MF_ROWS - 1) / (MF_WARPS * MF_ROWS)), gu = (unsigned)a.sse_blocks;
    if (m->k == 32) mf_row_kernel<1, 0><<<gi, MF_THREADS, 0, stream>>>(a);
    else mf_row_kernel<2, 0><<<gi, MF_THREADS, 0, stream>>>(a);
    EC_CUDA(cudaGetLastError());
    const size_t n = (size_t)a.I * m->k;
    int rc = ec_allreduce_ssp_apply(m->ar, m->bufs, a.P, n, EC_F32, EC_SUM, a.seg_rows * m->k, a.notif_clock, a.clock, slack,
                                    const_cast<float*>(a.reduced), m->count, m->seg_clock, m->wait, stream);
    if (rc != EC_OK) return rc;
    if (m->k == 32) mf_row_kernel<1, 1><<<gu, MF_THREADS, 0, stream>>>(a);
    else mf_row_kernel<2, 1><<<gu, MF_THREADS, 0, stream>>>(a);
    mf_item_step_kernel<<<(unsigned)((n + MF_THREADS - 1) / MF_THREADS), MF_THREADS, 0, stream>>>(a, n);
    EC_CUDA(cudaGetLastError());
    return EC_OK;
}

int ec_mf_set_factors(ec_mf_t* m, const float* user_factors, const float* item_factors, ec_stream_t stream) {
    if (!m || !user_factors || !item_factors) return EC_ERR_INVALID;
    EC_CUDA(cudaMemcpyAsync(m->a.pu, user_factors, (size_t)m->a.U * m->k * 4, cudaMemcpyDeviceToDevice, stream));
    EC_CUDA(cudaMemcpyAsync(m->a.qi, item_factors, (size_t)m->a.I * m->k * 4, cudaMemcpyDeviceToDevice, stream));
    return EC_OK;
}

int ec_mf_get(ec_mf_t* m, float* user_factors, float* item_factors, double* sse, uint32_t* seg_clock, uint32_t* notif_clock,
              uint32_t* wait_count, ec_stream_t stream) {
    if (!m) return EC_ERR_INVALID;
    const MfArgs& a = m->a;
    if (user_factors) EC_CUDA(cudaMemcpyAsync(user_factors, a.pu, (size_t)a.U * m->k * 4, cudaMemcpyDeviceToDevice, stream));
    if (item_factors) EC_CUDA(cudaMemcpyAsync(item_factors, a.qi, (size_t)a.I * m->k * 4, cudaMemcpyDeviceToDevice, stream));
    if (sse) EC_CUDA(cudaMemcpyAsync(sse, a.sse, 8, cudaMemcpyDeviceToDevice, stream));
    if (seg_clock) EC_CUDA(cudaMemcpyAsync(seg_clock, m->seg_clock, a.S * 4, cudaMemcpyDeviceToDevice, stream));
    if (notif_clock) EC_CUDA(cudaMemcpyAsync(notif_clock, a.notif_clock, a.S * a.P * 4, cudaMemcpyDeviceToDevice, stream));
    if (wait_count) EC_CUDA(cudaMemcpyAsync(wait_count, m->wait, a.S * 4, cudaMemcpyDeviceToDevice, stream));
    return EC_OK;
}

int ec_mf_destroy(ec_mf_t* m) {
    if (!m) return EC_ERR_INVALID;
    int rc = EC_OK;
    if (m->ar) rc = ec_allreduce_destroy(m->ar);
    if (m->own_ws && m->ws) {
        cudaError_t e = cudaFree(m->ws);
        if (e != cudaSuccess) rc = cuda_fail(e);
    }
    delete m;
    return rc;
}

}  // extern "C"
