// Eventually consistent Broadcast (Sec. III-B): the root ships only a leading share of its data, the
// threshold, and every receiver is told through notifications which segments it now holds.
//
// On one device the binomial spanning tree of the paper (root -> children -> their children, one
// write_notify per edge) collapses into one pass: every tile of the delivered prefix is read once
// and written into the receive buffer of every rank.  Segments beyond the threshold are not
// touched - a receiver keeps whatever it had there - and their notification bits are 0, so a
// consumer (ec_allreduce_apply with these words as its arrival mask, for instance) never reads them.

#include "ec_common.cuh"

namespace ec {
namespace {

constexpr int BC_THREADS = 256;
constexpr int BC_VPT = 2;                                  // 16-byte vectors per thread
constexpr size_t BC_TILE = (size_t)BC_THREADS * BC_VPT * 16;   // bytes of the source per block

struct BcastArgs {
    const char* src;
    uint64_t* notify;        // [S][W] or nullptr
    size_t keep_bytes;       // delivered prefix of the source
    size_t S, keep_segments;
    int P, W, root;
};

template <int CAP>
struct DstTable {
    void* p[CAP];            // nullptr: this rank receives nothing
};

template <int CAP, bool VECTOR>
__global__ void __launch_bounds__(BC_THREADS)
bcast_kernel(const BcastArgs a, const __grid_constant__ DstTable<CAP> t) {
    const int tid = threadIdx.x;
    // notification words: bit r of segment s = rank r holds segment s after this call
    if (a.notify != nullptr) {
        const size_t words = a.S * (size_t)a.W;
        for (size_t i = (size_t)blockIdx.x * BC_THREADS + tid; i < words; i += (size_t)gridDim.x * BC_THREADS) {
            const size_t s = i / (size_t)a.W;
            const int w = (int)(i - s * (size_t)a.W);
            uint64_t word = 0;
            if (s < a.keep_segments) {
                for (int b = 0; b < 64; ++b) {
                    const int r = w * 64 + b;
                    if (r < a.P && (t.p[r] != nullptr || r == a.root)) word |= 1ull << b;
                }
            }
            a.notify[i] = word;
        }
    }
    const uint64_t pol_ld = evict_first_policy();
    const uint64_t pol_st = result_policy(2);              // P copies of the data: they stream out
    for (size_t base = (size_t)blockIdx.x * BC_TILE; base < a.keep_bytes; base += (size_t)gridDim.x * BC_TILE) {
        if (VECTOR) {
            uint4 v[BC_VPT];
            bool have[BC_VPT];
#pragma unroll
            for (int q = 0; q < BC_VPT; ++q) {
                const size_t off = base + ((size_t)q * BC_THREADS + tid) * 16;
                have[q] = off + 16 <= a.keep_bytes;
                if (have[q]) v[q] = ld_stream16(a.src + off, pol_ld);
            }
            for (int r = 0; r < a.P; ++r) {
                char* dst = reinterpret_cast<char*>(t.p[r]);
                if (dst == nullptr || dst == a.src) continue;          // absent, or the root's own buffer
#pragma unroll
                for (int q = 0; q < BC_VPT; ++q)
                    if (have[q]) st_hint16(dst + base + ((size_t)q * BC_THREADS + tid) * 16, v[q], pol_st);
            }
            // bytes of the prefix after its last whole vector (a prefix that is not a multiple of 16 bytes)
            const size_t tail0 = a.keep_bytes & ~(size_t)15;
            if (base <= tail0 && tail0 < base + BC_TILE && tid < (int)(a.keep_bytes - tail0)) {
                const char c = a.src[tail0 + tid];
                for (int r = 0; r < a.P; ++r) {
                    char* dst = reinterpret_cast<char*>(t.p[r]);
                    if (dst != nullptr && dst != a.src) dst[tail0 + tid] = c;
                }
            }
        } else {
            for (size_t off = base + tid; off < base + BC_TILE && off < a.keep_bytes; off += BC_THREADS) {
                const char c = a.src[off];
                for (int r = 0; r < a.P; ++r) {
                    char* dst = reinterpret_cast<char*>(t.p[r]);
                    if (dst != nullptr && dst != a.src) dst[off] = c;
                }
            }
        }
    }
}

template <int CAP>
int launch(const BcastArgs& a, void* const* dsts, bool vector, unsigned grid, cudaStream_t st) {
    DstTable<CAP> t;
    for (int r = 0; r < CAP; ++r) t.p[r] = r < a.P ? dsts[r] : nullptr;
    if (vector) bcast_kernel<CAP, true><<<grid, BC_THREADS, 0, st>>>(a, t);
    else bcast_kernel<CAP, false><<<grid, BC_THREADS, 0, st>>>(a, t);
    EC_CUDA(cudaGetLastError());
    return EC_OK;
}

}  // namespace
}  // namespace ec

using namespace ec;

extern "C" int ec_bcast(const void* src, void* const* dst_bufs, int P, int root, size_t n, ec_dtype_t dtype,
                        size_t segment_size, double data_fraction, uint64_t* notify, ec_stream_t stream) {
    if (!src || !dst_bufs || P < 1 || P > EC_MAX_RANKS || root < 0 || root >= P || n == 0 || segment_size == 0)
        return EC_ERR_INVALID;
    if ((int)dtype < 0 || (int)dtype > EC_F64 || !(data_fraction >= 0.0) || data_fraction > 1.0) return EC_ERR_INVALID;
    const size_t es = in_bytes(dtype);
    const size_t S = (n + segment_size - 1) / segment_size;
    size_t keep = (size_t)(data_fraction * (double)S);
    if ((double)keep < data_fraction * (double)S) ++keep;      // ceil: the same rule as ec_mask_data_fraction
    if (keep > S) keep = S;
    size_t keep_elems = keep * segment_size;
    if (keep_elems > n) keep_elems = n;
    bool vector = aligned16(src);
    for (int r = 0; r < P; ++r) {
        if (dst_bufs[r] && dst_bufs[r] != src) {
            const uintptr_t d0 = reinterpret_cast<uintptr_t>(dst_bufs[r]), s0 = reinterpret_cast<uintptr_t>(src);
            if (d0 < s0 + n * es && s0 < d0 + n * es) return EC_ERR_INVALID;      // partial overlap with the source
        }
        vector = vector && aligned16(dst_bufs[r]);
    }
    BcastArgs a;
    a.src = reinterpret_cast<const char*>(src);
    a.notify = notify;
    a.keep_bytes = keep_elems * es;
    a.S = S; a.keep_segments = keep;
    a.P = P; a.W = (P + 63) / 64; a.root = root;
    size_t tiles = (a.keep_bytes + BC_TILE - 1) / BC_TILE;
    if (tiles < 1) tiles = 1;                                   // the notification words are still written
    const unsigned grid = (unsigned)(tiles < 0x7fffffffull ? tiles : 0x7fffffffull);
    if (P <= 64) return launch<64>(a, dst_bufs, vector, grid, stream);
    return launch<EC_MAX_RANKS>(a, dst_bufs, vector, grid, stream);
}
