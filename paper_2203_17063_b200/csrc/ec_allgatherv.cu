// Eventually consistent allgatherv: exclusive prefix sum of the counts and packed copy of the
// ranks that have arrived, in one launch.
//
// Every rank owns a fixed slot (the placement rule of the ring's Allgather stage, Sec. IV-A, and
// of the AlltoAll's one-target-per-writer, Sec. IV-B), so the displacements come from the counts
// of all ranks.  Every block recomputes the scan of the (at most 1024) counts - a few KB that stay
// in L2 - with warp shuffles, which removes any ordering between blocks.  The flattened output
// range is cut into equal chunks; a block finds the first rank of its chunk by binary search in
// the displacements and walks the ranks that overlap the chunk.  Measured on 256 ranks of int64 (counts 1024..65536 and
// the same times 8, 80 % notified): chunks of 64 KB with evict-first stores 24.9 / 172.9 us, chunks of 16 KB with plain
// stores 27.4 / 183.3 us; putting the 16-byte stores of slots whose phase differs from their source together by lane
// shuffles, or from element loads, was slower than the element-wise path (38.8 / 211.7 and 34.7 / 214.0 us); a plain
// device copy of the same bytes takes 28.0 / 151.8 us.

#include <type_traits>

#include "ec_common.cuh"

namespace ec {
namespace {

#ifndef EC_GV_BATCH
#define EC_GV_BATCH 4
#endif
#ifndef EC_GV_CHUNK
#define EC_GV_CHUNK 65536
#endif
#ifndef EC_GV_THREADS
#define EC_GV_THREADS 256
#endif
constexpr int GV_THREADS = EC_GV_THREADS;
constexpr size_t GV_CHUNK_BYTES = EC_GV_CHUNK;
constexpr int GV_BATCH = EC_GV_BATCH;  // loads in flight per thread before the stores
constexpr unsigned GV_MAX_BLOCKS = 16384;

struct GatherArgs {
    const int64_t* counts;
    const uint64_t* arrival;   // [W] or nullptr
    int64_t* displs;           // [P+1]
    char* out;
    uint32_t* status;
    size_t capacity;           // elements
    int P, esize;              // element size in bytes
    int compact;               // 1: only the ranks that have arrived get a slot
};

template <class T>
__device__ __forceinline__ void copy_elems(T* __restrict__ dst, const T* __restrict__ src, size_t cnt, int tid) {
    for (size_t i0 = tid; i0 < cnt; i0 += (size_t)GV_THREADS * GV_BATCH) {
        T v[GV_BATCH];
#pragma unroll
        for (int b = 0; b < GV_BATCH; ++b) {
            const size_t i = i0 + (size_t)b * GV_THREADS;
            if (i < cnt) v[b] = src[i];
        }
#pragma unroll
        for (int b = 0; b < GV_BATCH; ++b) {
            const size_t i = i0 + (size_t)b * GV_THREADS;
            if (i < cnt) dst[i] = v[b];
        }
    }
}

__device__ __forceinline__ void copy_vec16(char* __restrict__ dst, const char* __restrict__ src, size_t nvec, int tid,
                                           uint64_t pol) {
    for (size_t v0 = tid; v0 < nvec; v0 += (size_t)GV_THREADS * GV_BATCH) {
        uint4 r[GV_BATCH];
#pragma unroll
        for (int b = 0; b < GV_BATCH; ++b) {
            const size_t v = v0 + (size_t)b * GV_THREADS;
            if (v < nvec) r[b] = ld_stream16(src + v * 16, pol);
        }
#pragma unroll
        for (int b = 0; b < GV_BATCH; ++b) {
            const size_t v = v0 + (size_t)b * GV_THREADS;
            if (v < nvec) st_hint16(dst + v * 16, r[b], pol);     // written once, not read again here: evict-first like the loads
        }
    }
}

template <int ES>
__device__ __forceinline__ void copy_small(char* dst, const char* src, size_t bytes, int tid) {
    typedef typename std::conditional<ES == 8, uint64_t, typename std::conditional<ES == 4, uint32_t, uint16_t>::type>::type T;
    copy_elems<T>(reinterpret_cast<T*>(dst), reinterpret_cast<const T*>(src), bytes / ES, tid);
}

template <int CAP>
__global__ void __launch_bounds__(GV_THREADS)
allgatherv_kernel(const GatherArgs a, const __grid_constant__ PtrTable<CAP> tbl) {
    constexpr int ITEMS = CAP >= GV_THREADS ? CAP / GV_THREADS : 1;   // consecutive counts per thread
    __shared__ long long s_displs[CAP + 1];
    __shared__ long long s_warp[GV_THREADS / 32];
    __shared__ uint64_t s_arr[(CAP + 63) / 64];
    __shared__ int s_bad;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int P = a.P;

    if (tid == 0) s_bad = 0;
    // the counts and the arrival words are fetched together (one trip to memory, not two in a row)
    long long cnt[ITEMS];
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) {
        const int r = tid * ITEMS + i;
        cnt[i] = (r < P && r < CAP) ? a.counts[r] : 0;
    }
    for (int w = tid; w < (CAP + 63) / 64; w += GV_THREADS) {
        uint64_t word = 0;
        if (w * 64 < P) {
            word = a.arrival ? a.arrival[w] : ~0ull;
            if (P - w * 64 < 64) word &= (1ull << (P - w * 64)) - 1;       // bits >= P mean nothing
        }
        s_arr[w] = word;
    }
    __syncthreads();
    // exclusive scan: thread-local prefix, warp shuffle scan of the thread totals, scan of the warp totals
    long long local = 0;
    bool neg = false;
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) {
        const int r = tid * ITEMS + i;
        long long c = cnt[i];
        if (a.compact && r < P && !((s_arr[r >> 6] >> (r & 63)) & 1ull)) c = 0;   // compact reading: no slot for a missing rank
        if (c < 0) { neg = true; c = 0; }
        cnt[i] = c;
        local += c;
    }
    if (neg) s_bad = 1;
    long long incl = local;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const long long y = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += y;
    }
    if (lane == 31) s_warp[wid] = incl;
    __syncthreads();
    long long warp_off = 0;
    for (int w = 0; w < wid; ++w) warp_off += s_warp[w];
    long long run = warp_off + incl - local;                               // exclusive prefix of this thread's first item
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) {
        const int r = tid * ITEMS + i;
        if (r <= P && r < CAP) s_displs[r] = run;
        run += cnt[i];
        if (r + 1 == P) s_displs[P] = run;                                 // the total
    }
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
            const size_t bytes = (size_t)(e - b) * es;
            if (((reinterpret_cast<uintptr_t>(src) ^ reinterpret_cast<uintptr_t>(dst)) & 15u) == 0) {
                // same phase modulo 16: element-wise head up to the boundary, 128-bit body, element-wise tail
                size_t head = (16 - (reinterpret_cast<uintptr_t>(dst) & 15u)) & 15u;
                if (head > bytes) head = bytes;
                const size_t body = (bytes - head) / 16;
                const size_t tail0 = head + body * 16;
                if (head) {
                    if (es == 8) copy_small<8>(dst, src, head, tid);
                    else if (es == 4) copy_small<4>(dst, src, head, tid);
                    else copy_small<2>(dst, src, head, tid);
                }
                copy_vec16(dst + head, src + head, body, tid, pol);
                if (bytes > tail0) {
                    if (es == 8) copy_small<8>(dst + tail0, src + tail0, bytes - tail0, tid);
                    else if (es == 4) copy_small<4>(dst + tail0, src + tail0, bytes - tail0, tid);
                    else copy_small<2>(dst + tail0, src + tail0, bytes - tail0, tid);
                }
            } else {
                if (es == 8) copy_small<8>(dst, src, bytes, tid);
                else if (es == 4) copy_small<4>(dst, src, bytes, tid);
                else copy_small<2>(dst, src, bytes, tid);
            }
        }
    }
}

template <int CAP>
void launch(const GatherArgs& a, const void* const* bufs, unsigned grid, cudaStream_t stream) {
    PtrTable<CAP> tbl;
    for (int r = 0; r < CAP; ++r) tbl.p[r] = r < a.P ? bufs[r] : nullptr;
    allgatherv_kernel<CAP><<<grid, GV_THREADS, 0, stream>>>(a, tbl);
}

}  // namespace
}  // namespace ec

using namespace ec;

namespace {
int gather_common(const void* const* bufs, const int64_t* counts, int P, ec_dtype_t dtype, const uint64_t* arrival_mask,
                  int64_t* displs, void* out, size_t out_capacity_elems, uint32_t* status, int compact, cudaStream_t stream) {
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
    a.status = status; a.capacity = out_capacity_elems; a.P = P; a.esize = es; a.compact = compact;
    // One block per chunk the capacity allows; beyond GV_MAX_BLOCKS chunks the blocks loop.
    size_t chunks = (out_capacity_elems * (size_t)es + GV_CHUNK_BYTES - 1) / GV_CHUNK_BYTES;
    if (chunks < 1) chunks = 1;
    const unsigned grid = (unsigned)(chunks < (size_t)GV_MAX_BLOCKS ? chunks : (size_t)GV_MAX_BLOCKS);
    if (P <= 64) launch<64>(a, bufs, grid, stream);
    else if (P <= 256) launch<256>(a, bufs, grid, stream);
    else launch<EC_MAX_RANKS>(a, bufs, grid, stream);
    EC_CUDA(cudaGetLastError());
    return EC_OK;
}
}  // namespace

extern "C" int ec_allgatherv(const void* const* bufs, const int64_t* counts, int P, ec_dtype_t dtype,
                             const uint64_t* arrival_mask, int64_t* displs, void* out, size_t out_capacity_elems,
                             uint32_t* status, ec_stream_t stream) {
    return gather_common(bufs, counts, P, dtype, arrival_mask, displs, out, out_capacity_elems, status, 0, stream);
}

extern "C" int ec_allgatherv_compact(const void* const* bufs, const int64_t* counts, int P, ec_dtype_t dtype,
                                     const uint64_t* arrival_mask, int64_t* displs, void* out,
                                     size_t out_capacity_elems, uint32_t* status, ec_stream_t stream) {
    return gather_common(bufs, counts, P, dtype, arrival_mask, displs, out, out_capacity_elems, status, 1, stream);
}
