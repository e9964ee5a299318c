// Receiver-side kernel: unpack -> dequantise -> W-way mean (Eq. 4; Algorithm 1,
// "compute global gradients").
#pragma once

#include "ecq_common.cuh"

namespace ecq {

struct MessageTable {
    const uint32_t* codes[64];
    const float* scales[64];
};

// Entries per thread: the shortest run whose codes fill whole 32-bit words.
template <int R> struct DecodeGroup {
    static constexpr int kElems = (R % 8 == 0) ? 4 : (R % 4 == 0) ? 8 : (R % 2 == 0) ? 16 : 32;
    static constexpr int kWords = kElems * R / 32;
};

// out_i = (1/W) sum_w q_{w,i} * (scale_{w,b}/s), summed in ascending w with one
// fused multiply-add per term.
template <int R>
__global__ void __launch_bounds__(256)
decode_mean_kernel(const CodecParams P, const uint32_t W, const __grid_constant__ MessageTable tab,
                   float* __restrict__ out, const uint64_t n_groups, const uint64_t n_words,
                   const float w_recip, const int w_pow2) {
    constexpr int G = DecodeGroup<R>::kElems;
    constexpr int NW = DecodeGroup<R>::kWords;
    constexpr uint32_t mask = (1u << R) - 1u;
    const float magic = 8388608.f + (float)P.s;          // exact: s < 2^15
    for (uint64_t gi = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; gi < n_groups;
         gi += (uint64_t)gridDim.x * blockDim.x) {
        const uint64_t i0 = gi * G;
        const uint64_t b = i0 / P.bucket;
        const uint64_t w0 = gi * NW;
        float acc[G];
#pragma unroll
        for (int j = 0; j < G; ++j) acc[j] = 0.f;
        for (uint32_t w = 0; w < W; ++w) {
            const float a = __fdiv_rn(__ldg(tab.scales[w] + b), P.sf);
            uint32_t cw[NW + 1];
#pragma unroll
            for (int q = 0; q < NW; ++q)
                cw[q] = (w0 + q < n_words) ? __ldg(tab.codes[w] + w0 + q) : 0u;
            cw[NW] = 0u;
#pragma unroll
            for (int j = 0; j < G; ++j) {
                const int bit = j * R, wi = bit >> 5, sh = bit & 31;
                const uint32_t c = (sh + R <= 32) ? ((cw[wi] >> sh) & mask)
                                                  : (__funnelshift_r(cw[wi], cw[wi + 1], sh) & mask);
                // (float)(c - s) without a conversion: 2^23 + c is exact in fp32
                const float q = __fsub_rn(__uint_as_float(0x4B000000u | c), magic);
                acc[j] = __fmaf_rn(q, a, acc[j]);
            }
        }
#pragma unroll
        for (int j = 0; j < G; ++j)
            acc[j] = w_pow2 ? __fmul_rn(acc[j], w_recip) : __fdiv_rn(acc[j], (float)W);
        if (i0 + G <= P.d) {
#pragma unroll
            for (int j = 0; j < G; j += 4)
                *reinterpret_cast<float4*>(out + i0 + j) =
                    make_float4(acc[j], acc[j + 1], acc[j + 2], acc[j + 3]);
        } else {
#pragma unroll
            for (int j = 0; j < G; ++j)
                if (i0 + j < P.d) out[i0 + j] = acc[j];
        }
    }
}

// Any code width (r up to 16): 32 entries per thread, run-time shifts.
__global__ void __launch_bounds__(256)
decode_mean_generic_kernel(const CodecParams P, const uint32_t W,
                           const __grid_constant__ MessageTable tab, float* __restrict__ out,
                           const uint64_t n_groups, const uint64_t n_words, const float w_recip,
                           const int w_pow2) {
    const uint32_t r = P.r, mask = (1u << r) - 1u;
    const float magic = 8388608.f + (float)P.s;
    for (uint64_t gi = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; gi < n_groups;
         gi += (uint64_t)gridDim.x * blockDim.x) {
        const uint64_t i0 = gi * 32;
        const uint64_t b = i0 / P.bucket;
        const uint64_t w0 = gi * r;
        for (int j = 0; j < 32 && i0 + j < P.d; ++j) {
            const uint32_t bit = j * r, wi = bit >> 5, sh = bit & 31;
            float acc = 0.f;
            for (uint32_t w = 0; w < W; ++w) {
                const float a = __fdiv_rn(__ldg(tab.scales[w] + b), P.sf);
                const uint32_t lo = __ldg(tab.codes[w] + w0 + wi);
                const uint32_t hi = (sh + r > 32 && w0 + wi + 1 < n_words)
                                        ? __ldg(tab.codes[w] + w0 + wi + 1) : 0u;
                const uint32_t c = __funnelshift_r(lo, hi, sh) & mask;
                const float q = __fsub_rn(__uint_as_float(0x4B000000u | c), magic);
                acc = __fmaf_rn(q, a, acc);
            }
            out[i0 + j] = w_pow2 ? __fmul_rn(acc, w_recip) : __fdiv_rn(acc, (float)W);
        }
    }
}

}  // namespace ecq
