// Eventually consistent allgatherv: exclusive prefix sum of the counts and packed copy of the
// ranks that have arrived, in one launch.
//
// Every rank owns a fixed slot (the placement rule of the ring's Allgather stage, Sec. IV-A, and
// of the AlltoAll's one-target-per-writer, Sec. IV-B), so the displacements come from the counts
// of all ranks.  Every block recomputes the scan of the (at most 1024) counts in shared memory -
// 8 KB of reads that stay in L2 - which removes any ordering between blocks.  The flattened output
// range is cut into equal chunks; a block finds the first rank of its chunk by binary search in
// the displacements and walks the ranks that overlap the chunk.

#include "ec_common.cuh"

namespace ec {
namespace {

constexpr int GV_THREADS = 256;
constexpr size_t GV_CHUNK_BYTES = 16384;

struct GatherArgs {
    const int64_t* counts;
    const uint64_t* arrival;   // [W] or nullptr
    int64_t* displs;           // [P+1]
    char* out;
    uint32_t* status;
    size_t capacity;           // elements
    int P, esize;              // element size in bytes
};

template <int CAP>
__global__ void __launch_bounds__(GV_THREADS)
allgatherv_kernel(const GatherArgs a, const __grid_constant__ PtrTable<CAP> tbl) {
    __shared__ long long s_scan[2][CAP];      // double-buffered inclusive scan
    __shared__ long long s_displs[CAP + 1];
    __shared__ uint64_t s_arr[CAP / 64];
    __shared__ int s_bad;
    const int tid = threadIdx.x;
    const int P = a.P;

    if (tid == 0) s_bad = 0;
    __syncthreads();
    for (int r = tid; r < CAP; r += GV_THREADS) {
        long long c = 0;
        if (r < P) {
            c = a.counts[r];
            if (c < 0) { s_bad = 1; c = 0; }
        }
        s_scan[0][r] = c;
    }
    for (int w = tid; w < CAP / 64; w += GV_THREADS) {
        uint64_t word = 0;
        if (w * 64 < P) {
            word = a.arrival ? a.arrival[w] : ~0ull;
            if (P - w * 64 < 64) word &= (1ull << (P - w * 64)) - 1;
        }
        s_arr[w] = word;
    }
    __syncthreads();
    int cur = 0;
    for (int d = 1; d < CAP; d <<= 1) {          // Hillis-Steele inclusive scan
        for (int r = tid; r < CAP; r += GV_THREADS)
            s_scan[cur ^ 1][r] = s_scan[cur][r] + (r >= d ? s_scan[cur][r - d] : 0);
        cur ^= 1;
        __syncthreads();
    }
    for (int r = tid; r <= P; r += GV_THREADS) s_displs[r] = r == 0 ? 0 : s_scan[cur][r - 1];
    __syncthreads();
    const long long total = s_displs[P];
    const bool bad = s_bad != 0 || (unsigned long long)total > (unsigned long long)a.capacity;
    if (blockIdx.x == 0) {
        for (int r = tid; r <= P; r += GV_THREADS) a.displs[r] = s_displs[r];
        if (tid == 0) *a.status = bad ? 1u : 0u;
    }
    if (bad) return;

    const int es = a.esize;
    const uint64_t pol = evict_first_policy();
    const long long chunk = (long long)(GV_CHUNK_BYTES / (size_t)es);
    for (long long c0 = (long long)blockIdx.x * chunk; c0 < total; c0 += (long long)gridDim.x * chunk) {
        const long long c1 = c0 + chunk < total ? c0 + chunk : total;
        // first rank whose slot reaches into the chunk: the last r with displs[r] <= c0
        int lo = 0, hi = P;                       // invariant: displs[lo] <= c0 < displs[hi] (displs[P] = total > c0)
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (s_displs[mid] <= c0) lo = mid; else hi = mid;
        }
        for (int r = lo; r < P && s_displs[r] < c1; ++r) {
            if (!((s_arr[r >> 6] >> (r & 63)) & 1ull)) continue;     // not notified: never read, slot untouched
            const long long d0 = s_displs[r], d1 = s_displs[r + 1];
            const long long b = d0 > c0 ? d0 : c0, e = d1 < c1 ? d1 : c1;
            if (b >= e) continue;                                    // empty contribution
            const char* src = reinterpret_cast<const char*>(tbl.p[r]) + (size_t)(b - d0) * es;
            char* dst = a.out + (size_t)b * es;
            size_t bytes = (size_t)(e - b) * es;
            if (((reinterpret_cast<uintptr_t>(src) ^ reinterpret_cast<uintptr_t>(dst)) & 15u) == 0) {
                // same phase modulo 16: element-wise head up to the boundary, 128-bit body, element-wise tail
                size_t head = (16 - (reinterpret_cast<uintptr_t>(dst) & 15u)) & 15u;
                if (head > bytes) head = bytes;
                const size_t body = (bytes - head) / 16;
                const size_t tail0 = head + body * 16;
                for (size_t o = (size_t)tid * es; o < head; o += (size_t)GV_THREADS * es) {
                    if (es == 8) *reinterpret_cast<uint64_t*>(dst + o) = *reinterpret_cast<const uint64_t*>(src + o);
                    else if (es == 4) *reinterpret_cast<uint32_t*>(dst + o) = *reinterpret_cast<const uint32_t*>(src + o);
                    else *reinterpret_cast<uint16_t*>(dst + o) = *reinterpret_cast<const uint16_t*>(src + o);
                }
                for (size_t v = tid; v < body; v += GV_THREADS)
                    st_plain16(dst + head + v * 16, ld_stream16(src + head + v * 16, pol));
                for (size_t o = tail0 + (size_t)tid * es; o < bytes; o += (size_t)GV_THREADS * es) {
                    if (es == 8) *reinterpret_cast<uint64_t*>(dst + o) = *reinterpret_cast<const uint64_t*>(src + o);
                    else if (es == 4) *reinterpret_cast<uint32_t*>(dst + o) = *reinterpret_cast<const uint32_t*>(src + o);
                    else *reinterpret_cast<uint16_t*>(dst + o) = *reinterpret_cast<const uint16_t*>(src + o);
                }
            } else {
                const size_t cnt = (size_t)(e - b);
                if (es == 8) {
                    const uint64_t* s8 = reinterpret_cast<const uint64_t*>(src);
                    uint64_t* d8 = reinterpret_cast<uint64_t*>(dst);
                    for (size_t i = tid; i < cnt; i += GV_THREADS) d8[i] = s8[i];
                } else if (es == 4) {
                    const uint32_t* s4 = reinterpret_cast<const uint32_t*>(src);
                    uint32_t* d4 = reinterpret_cast<uint32_t*>(dst);
                    for (size_t i = tid; i < cnt; i += GV_THREADS) d4[i] = s4[i];
                } else {
                    const uint16_t* s2 = reinterpret_cast<const uint16_t*>(src);
                    uint16_t* d2 = reinterpret_cast<uint16_t*>(dst);
                    for (size_t i = tid; i < cnt; i += GV_THREADS) d2[i] = s2[i];
                }
            }
        }
    }
}

int sm_count() {
    static thread_local int cached_dev = -1, cached = 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (dev != cached_dev) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached = n;
        cached_dev = dev;
    }
    return cached;
}

}  // namespace
}  // namespace ec

using namespace ec;

extern "C" int ec_allgatherv(const void* const* bufs, const int64_t* counts, int P, ec_dtype_t dtype,
                             const uint64_t* arrival_mask, int64_t* displs, void* out, size_t out_capacity_elems,
                             uint32_t* status, ec_stream_t stream) {
    if (!bufs || !counts || !displs || !status || P < 1 || P > EC_MAX_RANKS) return EC_ERR_INVALID;
    if ((int)dtype < 0 || (int)dtype > EC_F64) return EC_ERR_INVALID;
    if (!out && out_capacity_elems != 0) return EC_ERR_INVALID;
    const int es = (int)in_bytes(dtype);
    if (reinterpret_cast<uintptr_t>(out) % (uintptr_t)es) return EC_ERR_INVALID;
    for (int r = 0; r < P; ++r)
        if (reinterpret_cast<uintptr_t>(bufs[r]) % (uintptr_t)es) return EC_ERR_INVALID;
    // A NULL entry is legal for a rank that is not notified or whose count is 0 (counts live on the
    // device, so this cannot be checked here); the kernel dereferences neither.
    GatherArgs a;
    a.counts = counts; a.arrival = arrival_mask; a.displs = displs; a.out = reinterpret_cast<char*>(out);
    a.status = status; a.capacity = out_capacity_elems; a.P = P; a.esize = es;
    // enough blocks for every chunk the capacity allows, at most four per SM (the blocks loop)
    size_t chunks = (out_capacity_elems * (size_t)es + GV_CHUNK_BYTES - 1) / GV_CHUNK_BYTES;
    if (chunks < 1) chunks = 1;
    const size_t cap_blocks = (size_t)sm_count() * 4;
    const unsigned grid = (unsigned)(chunks < cap_blocks ? chunks : cap_blocks);
    if (P <= 64) {
        PtrTable<64> tbl;
        for (int r = 0; r < 64; ++r) tbl.p[r] = r < P ? bufs[r] : nullptr;
        allgatherv_kernel<64><<<grid, GV_THREADS, 0, stream>>>(a, tbl);
    } else {
        PtrTable<EC_MAX_RANKS> tbl;
        for (int r = 0; r < EC_MAX_RANKS; ++r) tbl.p[r] = r < P ? bufs[r] : nullptr;
        allgatherv_kernel<EC_MAX_RANKS><<<grid, GV_THREADS, 0, stream>>>(a, tbl);
    }
    EC_CUDA(cudaGetLastError());
    return EC_OK;
}
