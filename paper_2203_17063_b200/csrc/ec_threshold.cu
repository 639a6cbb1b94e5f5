// Threshold variants of Reduce / Broadcast (Sec. III-B) as notification-word generators, and the
// threshold test on the status output.
//
// The paper offers two ways to make a Reduce eventually consistent: ship only a fraction of the
// data, or ship all data but leave processes out by their position in the binomial spanning tree so
// that at least the threshold share of processes takes part.  On one device both are a choice of
// notification words for ec_allreduce_apply: which segments, or which ranks, count as arrived.
// The binomial tree works in stages that double the number of involved processes (stage k brings in
// ranks 2^k .. 2^(k+1)-1, children of ranks 0 .. 2^k-1), so the share that can be reached is a power
// of two over P; the last stage alone adds half of the processes, which is why thresholds of 75 %
// and 100 % select the same set.

#include "ec_common.cuh"

namespace ec {
namespace {

__global__ void count_ready_kernel(const uint32_t* __restrict__ contrib_count, size_t S, uint32_t need,
                                   uint32_t* __restrict__ ready) {
    __shared__ unsigned s_part[32];
    unsigned local = 0;
    for (size_t s = threadIdx.x; s < S; s += blockDim.x) local += contrib_count[s] >= need ? 1u : 0u;
    for (int d = 16; d > 0; d >>= 1) local += __shfl_xor_sync(0xffffffffu, local, d);
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = local;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned total = 0;
        for (unsigned w = 0; w < (blockDim.x + 31) / 32; ++w) total += s_part[w];   // one block: no atomics, no clearing needed
        *ready = total;
    }
}

int ranks_for_share(int P, double fraction) {
    if (fraction <= 0.0) return 0;
    double need = fraction * (double)P;
    int involved = 1;                        // the root
    while (involved < P && (double)involved < need) involved *= 2;   // one more stage of the tree
    return involved < P ? involved : P;
}

}  // namespace
}  // namespace ec

using namespace ec;

extern "C" {

int ec_mask_data_fraction(int P, size_t S, double fraction, uint64_t* host_mask) {
    if (P < 1 || P > EC_MAX_RANKS || S == 0 || !host_mask || !(fraction >= 0.0) || fraction > 1.0) return EC_ERR_INVALID;
    const size_t W = (size_t)(P + 63) / 64;
    size_t keep = (size_t)(fraction * (double)S);
    if ((double)keep < fraction * (double)S) ++keep;          // ceil
    if (keep > S) keep = S;
    for (size_t s = 0; s < S; ++s)
        for (size_t w = 0; w < W; ++w) {
            uint64_t word = 0;
            if (s < keep) {
                const int hi = P - (int)w * 64;
                word = hi >= 64 ? ~0ull : (1ull << hi) - 1;
            }
            host_mask[s * W + w] = word;
        }
    return EC_OK;
}

int ec_mask_process_threshold(int P, size_t S, double fraction, uint64_t* host_mask, int* ranks_included) {
    if (P < 1 || P > EC_MAX_RANKS || S == 0 || !host_mask || !(fraction >= 0.0) || fraction > 1.0) return EC_ERR_INVALID;
    const size_t W = (size_t)(P + 63) / 64;
    const int involved = ranks_for_share(P, fraction);
    for (size_t s = 0; s < S; ++s)
        for (size_t w = 0; w < W; ++w) {
            const int hi = involved - (int)w * 64;
            host_mask[s * W + w] = hi <= 0 ? 0ull : hi >= 64 ? ~0ull : (1ull << hi) - 1;
        }
    if (ranks_included) *ranks_included = involved;
    return EC_OK;
}

int ec_threshold_segments(const uint32_t* contrib_count, size_t S, uint32_t need, uint32_t* ready_segments,
                          ec_stream_t stream) {
    if (!contrib_count || !ready_segments || S == 0) return EC_ERR_INVALID;
    count_ready_kernel<<<1, 1024, 0, stream>>>(contrib_count, S, need, ready_segments);
    EC_CUDA(cudaGetLastError());
    return EC_OK;
}

}  // extern "C"
