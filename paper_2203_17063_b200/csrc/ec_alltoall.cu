// Eventually consistent AlltoAll (Sec. IV-B): every rank writes one block into the memory of every
// other rank, each write with a notification of its own; the receiver consumes whatever has been
// notified and knows the collective is complete once all P blocks have arrived.
//
// On one device: recv[d] block s  <-  send[s] block d  for every (destination d, source s) whose
// notification bit is set; blocks whose bit is clear are left untouched (a late block is one more
// call).  recv_count[d] = number of blocks notified for destination d.  Stateless, one launch.
// The flattened receive space (P * P * block_bytes) is walked with 128-bit copies when blocks and
// pointers allow, so consecutive threads touch consecutive bytes whatever the block size.

#include "ec_common.cuh"

namespace ec {
namespace {

struct A2AArgs {
    const uint64_t* arrival;   // [P dst][W], bit = source rank; nullptr = all
    uint32_t* recv_count;      // [P] or nullptr
    size_t block_bytes;
    int P, W;
};

template <int CAP>
struct A2ATables {
    const void* send[CAP];
    void* recv[CAP];
};

template <int CAP, int VB>   // VB = bytes per copy: 16 or 1
__global__ void __launch_bounds__(256)
alltoall_kernel(const A2AArgs a, const __grid_constant__ A2ATables<CAP> t) {
    const int P = a.P;
    if (blockIdx.x == 0 && a.recv_count != nullptr) {
        for (int d = threadIdx.x; d < P; d += blockDim.x) {
            unsigned c = 0;
            for (int w = 0; w < a.W; ++w) {
                uint64_t word = a.arrival ? a.arrival[(size_t)d * a.W + w] : ~0ull;
                const int hi = P - w * 64;
                if (hi < 64) word &= hi <= 0 ? 0ull : (1ull << hi) - 1;        // bits >= P mean nothing
                c += (unsigned)__popcll(word);
            }
            a.recv_count[d] = c;
        }
    }
    const uint64_t pol = evict_first_policy();
    const size_t bv = a.block_bytes / VB;                  // copies per block
    const size_t per_dst = bv * (size_t)P;
    const size_t total = per_dst * (size_t)P;
    for (size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x; g < total; g += (size_t)gridDim.x * blockDim.x) {
        const size_t d = g / per_dst, rem = g - d * per_dst;
        const size_t s = rem / bv, off = (rem - s * bv) * VB;
        if (a.arrival) {
            const uint64_t word = a.arrival[d * (size_t)a.W + (s >> 6)];
            if (!((word >> (s & 63)) & 1ull)) continue;    // not notified: never read, block untouched
        }
        const char* src = reinterpret_cast<const char*>(t.send[s]) + d * a.block_bytes + off;
        char* dst = reinterpret_cast<char*>(t.recv[d]) + s * a.block_bytes + off;
        if (VB == 16) st_plain16(dst, ld_stream16(src, pol));
        else *dst = *src;
    }
}

// Blocks of at least a few KB: one thread block copies one 8 KB piece of one (destination, source) block,
// so the index arithmetic happens once per piece and every thread keeps two 128-bit loads in flight.
constexpr size_t A2A_PIECE = 8192;

template <int CAP>
__global__ void __launch_bounds__(256)
alltoall_piece_kernel(const A2AArgs a, const __grid_constant__ A2ATables<CAP> t) {
    const int P = a.P;
    if (blockIdx.x == 0 && a.recv_count != nullptr) {
        for (int d = threadIdx.x; d < P; d += blockDim.x) {
            unsigned c = 0;
            for (int w = 0; w < a.W; ++w) {
                uint64_t word = a.arrival ? a.arrival[(size_t)d * a.W + w] : ~0ull;
                const int hi = P - w * 64;
                if (hi < 64) word &= hi <= 0 ? 0ull : (1ull << hi) - 1;
                c += (unsigned)__popcll(word);
            }
            a.recv_count[d] = c;
        }
    }
    const uint64_t pol = evict_first_policy();
    const size_t pieces = (a.block_bytes + A2A_PIECE - 1) / A2A_PIECE;
    const size_t items = pieces * (size_t)P * (size_t)P;
    for (size_t it = blockIdx.x; it < items; it += gridDim.x) {
        const size_t pair = it / pieces, piece = it - pair * pieces;
        const size_t d = pair / (size_t)P, s = pair - d * (size_t)P;
        if (a.arrival) {
            const uint64_t word = a.arrival[d * (size_t)a.W + (s >> 6)];
            if (!((word >> (s & 63)) & 1ull)) continue;    // not notified: never read, block untouched
        }
        const size_t off = piece * A2A_PIECE;
        const size_t len = a.block_bytes - off < A2A_PIECE ? a.block_bytes - off : A2A_PIECE;   // multiple of 16
        const char* src = reinterpret_cast<const char*>(t.send[s]) + d * a.block_bytes + off;
        char* dst = reinterpret_cast<char*>(t.recv[d]) + s * a.block_bytes + off;
        const size_t nvec = len / 16;
        const size_t v0 = threadIdx.x, v1 = threadIdx.x + 256;
        uint4 r0, r1;
        if (v0 < nvec) r0 = ld_stream16(src + v0 * 16, pol);
        if (v1 < nvec) r1 = ld_stream16(src + v1 * 16, pol);
        if (v0 < nvec) st_plain16(dst + v0 * 16, r0);
        if (v1 < nvec) st_plain16(dst + v1 * 16, r1);
    }
}

template <int CAP>
int launch(const A2AArgs& a, const void* const* send, void* const* recv, bool vec, cudaStream_t st) {
    A2ATables<CAP> t;
    for (int r = 0; r < CAP; ++r) {
        t.send[r] = r < a.P ? send[r] : nullptr;
        t.recv[r] = r < a.P ? recv[r] : nullptr;
    }
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const size_t copies = (a.block_bytes / (vec ? 16 : 1)) * (size_t)a.P * (size_t)a.P;
    size_t blocks = (copies + 255) / 256;
    const size_t cap = (size_t)sms * 16;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    if (vec && a.block_bytes >= 2048) {
        const size_t items = ((a.block_bytes + A2A_PIECE - 1) / A2A_PIECE) * (size_t)a.P * (size_t)a.P;
        size_t pb = items < (size_t)sms * 32 ? items : (size_t)sms * 32;
        alltoall_piece_kernel<CAP><<<(unsigned)pb, 256, 0, st>>>(a, t);
    } else if (vec) alltoall_kernel<CAP, 16><<<(unsigned)blocks, 256, 0, st>>>(a, t);
    else alltoall_kernel<CAP, 1><<<(unsigned)blocks, 256, 0, st>>>(a, t);
    EC_CUDA(cudaGetLastError());
    return EC_OK;
}

}  // namespace
}  // namespace ec

using namespace ec;

extern "C" int ec_alltoall(const void* const* send_bufs, void* const* recv_bufs, int P, size_t block_bytes,
                           const uint64_t* arrival_mask, uint32_t* recv_count, ec_stream_t stream) {
    if (!send_bufs || !recv_bufs || P < 1 || P > EC_MAX_RANKS || block_bytes == 0) return EC_ERR_INVALID;
    bool vec = block_bytes % 16 == 0;
    for (int r = 0; r < P; ++r) {
        if (!send_bufs[r] || !recv_bufs[r]) return EC_ERR_INVALID;
        vec = vec && aligned16(send_bufs[r]) && aligned16(recv_bufs[r]);
        for (int q = 0; q < P; ++q)
            if (send_bufs[r] == recv_bufs[q]) return EC_ERR_INVALID;     // not an in-place collective
    }
    A2AArgs a;
    a.arrival = arrival_mask; a.recv_count = recv_count; a.block_bytes = block_bytes; a.P = P; a.W = (P + 63) / 64;
    return P <= 64 ? launch<64>(a, send_bufs, recv_bufs, vec, stream) : launch<EC_MAX_RANKS>(a, send_bufs, recv_bufs, vec, stream);
}
