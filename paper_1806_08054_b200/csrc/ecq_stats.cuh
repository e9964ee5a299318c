// Message statistics: how often each of the 2s+1 levels occurs in a code stream.  With the
// counts d_k the entropy-coded length of a message is at most sum_k d_k log2(d / d_k) bits
// (paragraph after Eq. 9), the figure behind every "# of bits" the paper reports.
#pragma once

#include "ecq_common.cuh"

namespace ecq {

constexpr int kHistThreads = 256;
constexpr uint32_t kHistLaneBins = 33;      // up to here every lane keeps its own column
constexpr uint32_t kHistSharedBins = 1025;  // up to here one shared-memory table per CTA

// One thread per run of 32 consecutive codes (= r whole words).  Small alphabets: a
// [bin][lane] table per warp, so increments need no atomics and hit distinct banks.
// Larger ones: one table per CTA with shared-memory atomics; beyond that, global atomics.
__global__ void __launch_bounds__(kHistThreads)
code_histogram_kernel(const CodecParams P, const uint32_t* __restrict__ codes,
                      unsigned long long* __restrict__ counts) {
    extern __shared__ uint32_t hsm[];
    const uint32_t r = P.r, mask = (1u << r) - 1u;
    const uint32_t nbins = 2 * P.s + 1;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int mode = nbins <= kHistLaneBins ? 0 : (nbins <= kHistSharedBins ? 1 : 2);
    uint32_t* mine = hsm;
    if (mode == 0) {
        mine = hsm + warp * (nbins * 32);
        for (uint32_t k = lane; k < nbins * 32; k += 32) mine[k] = 0;
        __syncwarp();
    } else if (mode == 1) {
        for (uint32_t k = threadIdx.x; k < nbins; k += kHistThreads) hsm[k] = 0;
        __syncthreads();
    }
    const uint64_t n_rows = (P.d + 31) >> 5;
    for (uint64_t row = (uint64_t)blockIdx.x * kHistThreads + threadIdx.x; row < n_rows;
         row += (uint64_t)gridDim.x * kHistThreads) {
        const uint64_t e0 = row << 5;
        const uint32_t nv = (uint32_t)((P.d - e0 < 32) ? (P.d - e0) : 32);
        const uint32_t* w = codes + row * r;
        const uint32_t nw = (nv * r + 31) >> 5;             // words that exist for this run
        uint64_t acc = 0;
        uint32_t have = 0, kw = 0;
        for (uint32_t j = 0; j < nv; ++j) {
            if (have < r) { acc |= (uint64_t)(kw < nw ? __ldg(w + kw) : 0u) << have; ++kw; have += 32; }
            const uint32_t c = (uint32_t)acc & mask;
            acc >>= r; have -= r;
            if (c < nbins) {
                if (mode == 0) mine[c * 32 + lane] += 1;
                else if (mode == 1) atomicAdd(hsm + c, 1u);
                else atomicAdd(counts + c, 1ull);
            }
        }
    }
    if (mode == 0) {
        __syncwarp();
        for (uint32_t b = 0; b < nbins; ++b) {
            uint32_t v = mine[b * 32 + lane];
            v = __reduce_add_sync(0xFFFFFFFFu, v);
            if (lane == 0 && v) atomicAdd(counts + b, (unsigned long long)v);
        }
    } else if (mode == 1) {
        __syncthreads();
        for (uint32_t k = threadIdx.x; k < nbins; k += kHistThreads)
            if (hsm[k]) atomicAdd(counts + k, (unsigned long long)hsm[k]);
    }
}

}  // namespace ecq
