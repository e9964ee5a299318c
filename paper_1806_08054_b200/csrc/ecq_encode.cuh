// Sender-side kernels: compensate (Eq. 7) -> per-bucket l-infinity scale (Eq. 8)
// -> stochastic rounding (Eq. 9) -> error-accumulator update (Eq. 6) -> r-bit pack.
#pragma once

#include <cuda.h>

#include "ecq_common.cuh"

namespace ecq {

// ===========================================================================
// Any-shape path: one CTA per bucket, two passes over the bucket (the second
// one hits L1/L2).  Serves bucket sizes the tiled kernel does not take (not a
// power of two, or above 4096) and the ragged end of a vector.
// ===========================================================================
template <int NT>
__device__ void encode_bucket_generic(const CodecParams& P, uint64_t b, uint32_t worker,
                                      uint32_t step, const float* __restrict__ g, float* h,
                                      uint32_t* __restrict__ codes, float* __restrict__ scales,
                                      uint32_t* status, uint32_t* s_red, int tid) {
    const uint64_t lo = b * (uint64_t)P.bucket;
    const uint64_t hi = (lo + P.bucket < P.d) ? lo + P.bucket : P.d;
    const uint32_t n = (uint32_t)(hi - lo);
    const float* gb = g + lo;
    float* hb = h + lo;

    // pass 1: max |g + alpha h| over the bucket, as an integer max of the
    // sign-cleared bit patterns (exact, order-free, NaN/Inf sort on top)
    uint32_t m = 0;
    for (uint32_t idx = tid * 4; idx < n; idx += NT * 4) {
        if (idx + 4 <= n) {
            const float4 g4 = *reinterpret_cast<const float4*>(gb + idx);
            const float4 h4 = *reinterpret_cast<const float4*>(hb + idx);
            m = max(m, __float_as_uint(__fmaf_rn(P.alpha, h4.x, g4.x)) & 0x7FFFFFFFu);
            m = max(m, __float_as_uint(__fmaf_rn(P.alpha, h4.y, g4.y)) & 0x7FFFFFFFu);
            m = max(m, __float_as_uint(__fmaf_rn(P.alpha, h4.z, g4.z)) & 0x7FFFFFFFu);
            m = max(m, __float_as_uint(__fmaf_rn(P.alpha, h4.w, g4.w)) & 0x7FFFFFFFu);
        } else {
            for (uint32_t j = idx; j < n; ++j)
                m = max(m, __float_as_uint(__fmaf_rn(P.alpha, hb[j], gb[j])) & 0x7FFFFFFFu);
        }
    }
    m = __reduce_max_sync(0xFFFFFFFFu, m);
    if ((tid & 31) == 0) s_red[tid >> 5] = m;
    __syncthreads();
    m = 0;
#pragma unroll
    for (int w = 0; w < NT / 32; ++w) m = max(m, s_red[w]);
    const BucketScale bs = bucket_scale(m, P.sf);
    if (tid == 0) {
        scales[b] = bs.scale;
        if (bs.kind == 2) atomicOr(status, kStatusNonFinite);
    }

    // pass 2: one thread per run of 32 consecutive entries (= r whole words)
    const uint32_t nrows = (n + 31) >> 5;
    const uint64_t word0 = (lo >> 5) * P.r;
    for (uint32_t row = tid; row < nrows; row += NT) {
        const uint32_t e0 = row * 32;
        const uint32_t nv = min(32u, n - e0);
        const uint64_t blk0 = (lo + e0) >> 2;
        uint32_t* cw = codes + word0 + (uint64_t)row * P.r;
        uint64_t acc = 0;
        uint32_t nbits = 0, kw = 0;
        for (uint32_t c = 0; c < 8 && 4 * c < nv; ++c) {
            float gv[4], hv[4], hn[4];
            const uint32_t e = e0 + 4 * c;
            const uint32_t cnt = min(4u, nv - 4 * c);
            if (cnt == 4) {
                const float4 g4 = *reinterpret_cast<const float4*>(gb + e);
                const float4 h4 = *reinterpret_cast<const float4*>(hb + e);
                gv[0] = g4.x; gv[1] = g4.y; gv[2] = g4.z; gv[3] = g4.w;
                hv[0] = h4.x; hv[1] = h4.y; hv[2] = h4.z; hv[3] = h4.w;
            } else {
                for (uint32_t j = 0; j < 4; ++j) {
                    gv[j] = (j < cnt) ? gb[e + j] : 0.f;
                    hv[j] = (j < cnt) ? hb[e + j] : 0.f;
                }
            }
            uint32_t R[4];
            const uint64_t blk = blk0 + c;
            philox4x32_10(P, (uint32_t)blk, (uint32_t)(blk >> 32), worker, step, R);
#pragma unroll
            for (uint32_t j = 0; j < 4; ++j) {
                const float v = __fmaf_rn(P.alpha, hv[j], gv[j]);
                uint32_t code = P.s;
                if (bs.kind == 0) code = quantise_entry(gv[j], hv[j], v, R[j], bs, P, hn[j]);
                else if (bs.kind == 1) hn[j] = __fmaf_rn(P.beta, hv[j], P.mode ? v : gv[j]);
                else hn[j] = hv[j];
                if (j < cnt) {
                    acc |= (uint64_t)code << nbits;
                    nbits += P.r;
                    if (nbits >= 32) { cw[kw++] = (uint32_t)acc; acc >>= 32; nbits -= 32; }
                }
            }
            if (cnt == 4) {
                *reinterpret_cast<float4*>(hb + e) = make_float4(hn[0], hn[1], hn[2], hn[3]);
            } else {
                for (uint32_t j = 0; j < cnt; ++j) hb[e + j] = hn[j];
            }
        }
        if (nbits > 0) cw[kw] = (uint32_t)acc;      // zero-padded last word of the stream
    }
    __syncthreads();   // s_red is reused by the next bucket
}

template <int NT>
__global__ void __launch_bounds__(NT)
encode_generic_kernel(CodecParams P, uint32_t worker, uint32_t step, const float* __restrict__ g,
                      float* h, uint32_t* __restrict__ codes, float* __restrict__ scales,
                      uint32_t* status, uint64_t first_bucket, uint64_t n_buckets) {
    __shared__ uint32_t s_red[NT / 32];
    for (uint64_t b = blockIdx.x; b < n_buckets; b += gridDim.x)
        encode_bucket_generic<NT>(P, first_bucket + b, worker, step, g, h, codes, scales, status,
                                  s_red, threadIdx.x);
}

// ===========================================================================
// Tiled path.  The vector is seen as a matrix of 128-byte rows (32 floats).  A
// tile is 128 rows = 4096 entries = a whole number of buckets (bucket a power
// of two <= 4096).  A persistent CTA streams its tiles through an NSTAGES ring
// in shared memory:
//   producer lane : TMA loads of the g and h tiles (128-byte swizzle) ->
//                   full[s];  after the consumers are done with a stage it
//                   issues the TMA store of the updated h tile and a linear
//                   bulk store of the tile's code words, then refills the stage
//   128 consumers : one thread per row.  The swizzle makes a thread's eight
//                   16-byte chunks of its row conflict-free across the warp.
//                   Pass 1 takes the row max, the rows of a bucket are combined
//                   by shuffles (and one shared-memory hop above 1024 entries);
//                   pass 2 re-reads the row, draws Philox per 4 entries, rounds,
//                   updates h in place and packs the 32 codes into R words.
// g and h are read from HBM once, h is written once; v never leaves the SM.
// ===========================================================================
constexpr int kTileRows = 128;
constexpr int kTileElems = kTileRows * 32;          // 4096
constexpr int kTileBytes = kTileElems * 4;          // 16 KiB per operand
constexpr int kConsumers = kTileRows;               // one thread per row
constexpr int kEncodeThreads = kConsumers + 32;     // + producer warp

template <int R, int NSTAGES>
struct EncodeSmem {
    static constexpr int kCodeBytes = R * (kTileElems / 8);       // R * 512
    static constexpr int kStageBytes = 2 * kTileBytes;
    static constexpr int kCodesOff = NSTAGES * kStageBytes;
    static constexpr int kBarOff = kCodesOff + NSTAGES * kCodeBytes;
    static constexpr int kMiscOff = kBarOff + 2 * NSTAGES * 8;
    static constexpr int kTotal = kMiscOff + 64 + 1024;           // + alignment slack
};

template <int R, int NSTAGES>
__global__ void __launch_bounds__(kEncodeThreads)
encode_tiled_kernel(const __grid_constant__ CUtensorMap tm_g, const __grid_constant__ CUtensorMap tm_h,
                    const CodecParams P, const uint32_t worker, const uint32_t step,
                    const float* __restrict__ g, float* h, uint32_t* __restrict__ codes,
                    float* __restrict__ scales, uint32_t* status, const uint32_t n_tiles) {
    using L = EncodeSmem<R, NSTAGES>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* const sm = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bar_full = base + L::kBarOff;
    const uint32_t bar_done = bar_full + NSTAGES * 8;
    volatile uint32_t* s_abort = reinterpret_cast<volatile uint32_t*>(sm + L::kMiscOff);
    uint32_t* s_wmax = reinterpret_cast<uint32_t*>(sm + L::kMiscOff + 16);   // 4 warps x 2 parities

    const int tid = threadIdx.x;
    if (tid == 0) {
        for (int s = 0; s < NSTAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_done + 8 * s, kConsumers);
        }
        *s_abort = 0;
        fence_mbar_init();
    }
    __syncthreads();

    const uint32_t n_my = (n_tiles > blockIdx.x)
                              ? (n_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    const uint32_t rpb = P.bucket >> 5;              // rows per bucket, power of two <= 128

    if (tid >= kConsumers) {
        // ------------------------------ producer ------------------------------
        if (tid == kConsumers) {
            auto issue_load = [&](uint32_t k) {
                const uint32_t s = k % NSTAGES;
                const uint32_t tile = blockIdx.x + k * gridDim.x;
                const uint32_t bar = bar_full + 8 * s;
                mbar_arrive_expect_tx(bar, 2 * kTileBytes);
                tma_load_2d(base + s * L::kStageBytes, &tm_g, 0, (int)(tile * kTileRows), bar);
                tma_load_2d(base + s * L::kStageBytes + kTileBytes, &tm_h, 0,
                            (int)(tile * kTileRows), bar);
            };
            uint32_t issued = 0;
            for (; issued < n_my && issued < (uint32_t)NSTAGES; ++issued) issue_load(issued);
            bool ok = true;
            for (uint32_t k = 0; k < n_my; ++k) {
                const uint32_t s = k % NSTAGES;
                if (*s_abort || !mbar_wait(bar_done + 8 * s, (k / NSTAGES) & 1u)) { ok = false; break; }
                const uint32_t tile = blockIdx.x + k * gridDim.x;
                tma_store_2d(&tm_h, 0, (int)(tile * kTileRows),
                             base + s * L::kStageBytes + kTileBytes);
                bulk_store_1d(codes + (uint64_t)tile * (R * kTileRows),
                              base + L::kCodesOff + s * L::kCodeBytes, L::kCodeBytes);
                bulk_commit();
                if (issued < n_my) {
                    bulk_wait_read0();               // the stage is free once the stores have read it
                    issue_load(issued++);
                }
            }
            if (!ok) {
                *s_abort = 1;
                atomicOr(status, kStatusTimeout);
                // let the loads still in flight land before the CTA gives up its shared memory
                const uint32_t first = issued > (uint32_t)NSTAGES ? issued - NSTAGES : 0;
                for (uint32_t j = first; j < issued; ++j)
                    mbar_wait(bar_full + 8 * (j % NSTAGES), (j / NSTAGES) & 1u);
            }
            bulk_wait_all();
        }
    } else {
        // ------------------------------ consumers -----------------------------
        const int row = tid;
        const int lane = tid & 31;
        const int warp = tid >> 5;
        const uint32_t sw = (uint32_t)(row & 7) << 4;
        const uint32_t buckets_per_tile = kTileElems / P.bucket;
        for (uint32_t k = 0; k < n_my; ++k) {
            const uint32_t s = k % NSTAGES;
            const uint32_t tile = blockIdx.x + k * gridDim.x;
            bool ok = mbar_wait(bar_full + 8 * s, (k / NSTAGES) & 1u);
            if (!ok) { *s_abort = 1; atomicOr(status, kStatusTimeout); }
            const uint8_t* gs = sm + s * L::kStageBytes + row * 128;
            uint8_t* hs = sm + s * L::kStageBytes + kTileBytes + row * 128;

            // pass 1: row max of |g + alpha h|
            uint32_t m = 0;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const uint32_t off = ((uint32_t)c << 4) ^ sw;
                const float4 g4 = *reinterpret_cast<const float4*>(gs + off);
                const float4 h4 = *reinterpret_cast<const float4*>(hs + off);
                m = max(m, __float_as_uint(__fmaf_rn(P.alpha, h4.x, g4.x)) & 0x7FFFFFFFu);
                m = max(m, __float_as_uint(__fmaf_rn(P.alpha, h4.y, g4.y)) & 0x7FFFFFFFu);
                m = max(m, __float_as_uint(__fmaf_rn(P.alpha, h4.z, g4.z)) & 0x7FFFFFFFu);
                m = max(m, __float_as_uint(__fmaf_rn(P.alpha, h4.w, g4.w)) & 0x7FFFFFFFu);
            }
            // combine the rows of a bucket
            for (uint32_t o = 1; o < rpb && o < 32; o <<= 1)
                m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
            if (rpb > 32) {
                uint32_t* wm = s_wmax + (k & 1u) * 4;
                if (lane == 0) wm[warp] = m;
                named_bar_sync(1, kConsumers);
                if (rpb == 64) m = max(wm[warp & ~1], wm[warp | 1]);
                else m = max(max(wm[0], wm[1]), max(wm[2], wm[3]));
                if (*s_abort) break;                 // uniform: read after the barrier
            } else {
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;                      // warp-uniform
            }
            const BucketScale bs = bucket_scale(m, P.sf);
            if ((row & (rpb - 1)) == 0) {
                scales[(uint64_t)tile * buckets_per_tile + row / rpb] = bs.scale;
                if (bs.kind == 2) atomicOr(status, kStatusNonFinite);
            }

            // pass 2: round, update h in place, pack 32 codes into R words
            const uint64_t blk0 = (uint64_t)tile * (kTileElems / 4) + (uint32_t)row * 8;
            uint32_t wout[R];
            uint64_t acc = 0;
            int nbits = 0, kw = 0;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const uint32_t off = ((uint32_t)c << 4) ^ sw;
                const float4 g4 = *reinterpret_cast<const float4*>(gs + off);
                const float4 h4 = *reinterpret_cast<const float4*>(hs + off);
                const float gv[4] = {g4.x, g4.y, g4.z, g4.w};
                const float hv[4] = {h4.x, h4.y, h4.z, h4.w};
                float hn[4];
                uint32_t code[4];
                if (bs.kind == 0) {
                    uint32_t Rw[4];
                    const uint64_t blk = blk0 + c;
                    philox4x32_10(P, (uint32_t)blk, (uint32_t)(blk >> 32), worker, step, Rw);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float v = __fmaf_rn(P.alpha, hv[j], gv[j]);
                        code[j] = quantise_entry(gv[j], hv[j], v, Rw[j], bs, P, hn[j]);
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float v = __fmaf_rn(P.alpha, hv[j], gv[j]);
                        code[j] = P.s;
                        hn[j] = (bs.kind == 1) ? __fmaf_rn(P.beta, hv[j], P.mode ? v : gv[j]) : hv[j];
                    }
                }
                *reinterpret_cast<float4*>(hs + off) = make_float4(hn[0], hn[1], hn[2], hn[3]);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    acc |= (uint64_t)code[j] << nbits;
                    nbits += R;
                    if (nbits >= 32) { wout[kw++] = (uint32_t)acc; acc >>= 32; nbits -= 32; }
                }
            }
            uint32_t* cs = reinterpret_cast<uint32_t*>(sm + L::kCodesOff + s * L::kCodeBytes) + row * R;
            if constexpr (R % 4 == 0) {
#pragma unroll
                for (int q = 0; q < R / 4; ++q)
                    reinterpret_cast<uint4*>(cs)[q] =
                        make_uint4(wout[4 * q], wout[4 * q + 1], wout[4 * q + 2], wout[4 * q + 3]);
            } else if constexpr (R % 2 == 0) {
#pragma unroll
                for (int q = 0; q < R / 2; ++q)
                    reinterpret_cast<uint2*>(cs)[q] = make_uint2(wout[2 * q], wout[2 * q + 1]);
            } else {
#pragma unroll
                for (int q = 0; q < R; ++q) cs[q] = wout[q];
            }
            fence_proxy_async_smem();               // my writes -> visible to the TMA stores
            mbar_arrive(bar_done + 8 * s);
        }
    }

    __syncthreads();
    if (*s_abort) return;

    // ragged end: the buckets after the last whole tile, spread over the CTAs
    // from the back of the grid (those own one tile fewer)
    const uint64_t tail_first = (uint64_t)n_tiles * (kTileElems / P.bucket);
    const uint64_t nb_total = (P.d + P.bucket - 1) / P.bucket;
    uint32_t* s_red = reinterpret_cast<uint32_t*>(sm);   // the ring is idle now
    for (uint64_t b = tail_first + (gridDim.x - 1 - blockIdx.x); b < nb_total; b += gridDim.x)
        encode_bucket_generic<kEncodeThreads>(P, b, worker, step, g, h, codes, scales, status,
                                              s_red, tid);
}

}  // namespace ecq
