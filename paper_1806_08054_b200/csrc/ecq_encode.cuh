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
// Tiled path.  The vector is seen as a matrix of 128-byte rows (32 floats); a
// tile is 128 rows = 4096 entries = a whole number of buckets (bucket a power
// of two <= 4096).  A persistent CTA of 128 threads (four per SM) owns one
// 32 KiB load buffer and one store staging buffer and walks its tiles:
//   * thread 0 issues two 16 KiB TMA loads (g and h tile, 128-byte swizzle);
//     measured on B200, a TMA operation costs ~200 cycles of issue time
//     whatever its size, so tiles are moved with few large operations;
//   * every thread copies its row of g and h to registers (the swizzle makes
//     the eight 16-byte chunks of a row conflict-free across the warp); after
//     one CTA barrier the buffer is refilled with the next tile, which lands
//     while this one is being computed;
//   * the row max of |g + alpha h| is combined over the rows of a bucket by
//     shuffles (and through shared memory when a bucket spans 2 or 4 warps);
//   * each thread draws Philox per 4 entries, rounds, forms the new h row in
//     registers and packs its 32 codes into R words; both go to the staging
//     buffer, from which thread 0 issues one TMA store (h tile) and one linear
//     bulk store (code words).
// g and h are read from HBM once, h is written once; v never leaves the SM.
// ===========================================================================
constexpr int kTileRows = 128;
constexpr int kTileElems = kTileRows * 32;          // 4096
constexpr int kTileBytes = kTileElems * 4;          // 16 KiB per operand
constexpr int kEncodeThreads = kTileRows;           // one thread per row
constexpr int kEncodeCtasPerSm = 4;
constexpr uint32_t kMaxTiledBucket = kTileElems;    // largest bucket of the tiled path

template <int R>
struct EncodeSmem {
    static constexpr int kCodeBytes = R * (kTileElems / 8);       // R * 512 per tile
    static constexpr int kLoadOff = 0;                            // g tile, h tile
    static constexpr int kHoutOff = 2 * kTileBytes;               // staged new h tile
    static constexpr int kCoutOff = 3 * kTileBytes;               // staged code words
    static constexpr int kBarOff = kCoutOff + kCodeBytes;
    static constexpr int kMiscOff = kBarOff + 16;
    static constexpr int kTotal = kMiscOff + 48 + 1024;           // + alignment slack
};

// max(m, |a|, |b|) that returns NaN if any input is NaN
__device__ __forceinline__ float max3_abs_nan(float m, float a, float b) {
    float r;
    asm("max.NaN.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(m), "f"(fabsf(a)), "f"(fabsf(b)));
    return r;
}

template <int R>
__global__ void __launch_bounds__(kEncodeThreads, kEncodeCtasPerSm)
encode_tiled_kernel(const __grid_constant__ CUtensorMap tm_g, const __grid_constant__ CUtensorMap tm_h,
                    const CodecParams P, const uint32_t worker, const uint32_t step,
                    const float* __restrict__ g, float* h, uint32_t* __restrict__ codes,
                    float* __restrict__ scales, uint32_t* status, const uint32_t n_tiles) {
    using L = EncodeSmem<R>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* const sm = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bar_full = base + L::kBarOff;
    volatile uint32_t* s_abort = reinterpret_cast<volatile uint32_t*>(sm + L::kMiscOff);
    uint32_t* s_wmax = reinterpret_cast<uint32_t*>(sm + L::kMiscOff + 16);   // one per warp

    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    auto issue_load = [&](uint32_t tile) {
        mbar_arrive_expect_tx(bar_full, 2 * kTileBytes);
        tma_load_2d(base + L::kLoadOff, &tm_g, 0, (int)(tile * kTileRows), bar_full);
        tma_load_2d(base + L::kLoadOff + kTileBytes, &tm_h, 0, (int)(tile * kTileRows), bar_full);
    };
    if (tid == 0) {
        mbar_init(bar_full, 1);
        *s_abort = 0;
        fence_mbar_init();
        if (blockIdx.x < n_tiles) issue_load(blockIdx.x);
    }
    __syncthreads();

    const uint32_t sw = (uint32_t)(tid & 7) << 4;
    const uint32_t rpb = P.bucket >> 5;                    // rows per bucket, power of two <= 128
    const uint32_t buckets_per_tile = kTileElems / P.bucket;
    const float magic_code = 12582912.f + P.sf;            // 1.5*2^23 + s, exact
    const uint8_t* const g_row = sm + L::kLoadOff + tid * 128;
    const uint8_t* const h_row = g_row + kTileBytes;
    uint8_t* const hout_row = sm + L::kHoutOff + tid * 128;
    uint32_t* const cout_row = reinterpret_cast<uint32_t*>(sm + L::kCoutOff) + tid * R;

    uint32_t parity = 0;
    for (uint32_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, parity ^= 1u) {
        if (!mbar_wait(bar_full, parity)) { *s_abort = 1; atomicOr(status, kStatusTimeout); }

        // my row of g and h -> registers
        float4 G[8], H[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const uint32_t off = ((uint32_t)c << 4) ^ sw;
            G[c] = *reinterpret_cast<const float4*>(g_row + off);
            H[c] = *reinterpret_cast<const float4*>(h_row + off);
        }
        // row max of |g + alpha h| (NaN-propagating), then over the rows of the bucket
        float mf = 0.f;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            mf = max3_abs_nan(mf, __fmaf_rn(P.alpha, H[c].x, G[c].x), __fmaf_rn(P.alpha, H[c].y, G[c].y));
            mf = max3_abs_nan(mf, __fmaf_rn(P.alpha, H[c].z, G[c].z), __fmaf_rn(P.alpha, H[c].w, G[c].w));
        }
        // non-negative floats and NaN (0x7FFFFFFF) order like their bit patterns
        uint32_t m = __float_as_uint(mf) & 0x7FFFFFFFu;
        for (uint32_t o = 1; o < rpb && o < 32; o <<= 1)
            m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
        if (rpb > 32 && lane == 0) s_wmax[warp] = m;
        // the stores of the previous tile must have read the staging buffer
        if (tid == 0) bulk_wait_read0();
        __syncthreads();                                   // load buffer and staging are free
        if (*s_abort) break;                               // uniform: set before the barrier
        if (tid == 0 && tile + gridDim.x < n_tiles) issue_load(tile + gridDim.x);
        if (rpb == 64) m = max(s_wmax[warp & ~1], s_wmax[warp | 1]);
        if (rpb == 128) m = max(max(s_wmax[0], s_wmax[1]), max(s_wmax[2], s_wmax[3]));
        const BucketScale bs = bucket_scale(m, P.sf);
        if ((tid & (rpb - 1)) == 0) {
            scales[(uint64_t)tile * buckets_per_tile + tid / rpb] = bs.scale;
            if (bs.kind == 2) atomicOr(status, kStatusNonFinite);
        }

        // round, new h (kept in H), pack 32 codes into R words.  The codes enter a
        // 64-bit window as (float bits of q + s + 1.5*2^23) << pos; the constant
        // high bits are removed once per output word.
        const uint64_t blk0 = (uint64_t)tile * (kTileElems / 4) + (uint32_t)tid * 8;
        uint32_t wout[R];
        uint64_t acc = 0, junk = 0;
        int nbits = 0, kw = 0;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const float gv[4] = {G[c].x, G[c].y, G[c].z, G[c].w};
            const float hv[4] = {H[c].x, H[c].y, H[c].z, H[c].w};
            float hn[4];
            uint32_t cb[4];
            if (bs.kind == 0) {
                uint32_t Rw[4];
                const uint64_t blk = blk0 + c;
                philox4x32_10(P, (uint32_t)blk, (uint32_t)(blk >> 32), worker, step, Rw);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float v = __fmaf_rn(P.alpha, hv[j], gv[j]);
                    const uint32_t sgn = __float_as_uint(v) & 0x80000000u;
                    const float x = fminf(__fmul_rn(fabsf(v), bs.inv), P.sf);
                    const float lf = __fsub_rn(__fadd_rz(x, 8388608.f), 8388608.f);   // floor
                    const float f = __fsub_rn(x, lf);
                    const float u = __fmul_rn(__uint2float_rn(Rw[j] >> 8), 0x1p-24f);
                    const float mlev = __fadd_rn(lf, (u < f) ? 1.f : 0.f);
                    // work on sgn(v)*g so that the level stays non-negative: negation
                    // commutes with rounding, and a zero level leaves g untouched
                    const float gsn = __uint_as_float(__float_as_uint(P.mode ? v : gv[j]) ^ sgn);
                    const float esn = __fsub_rn(gsn, __fmul_rn(mlev, bs.a));
                    const float e = __uint_as_float(__float_as_uint(esn) ^ sgn);
                    hn[j] = __fmaf_rn(P.beta, hv[j], e);
                    const float q = __uint_as_float(__float_as_uint(mlev) ^ sgn);
                    cb[j] = __float_as_uint(__fadd_rn(q, magic_code));     // 0x4B400000 + q + s
                }
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float v = __fmaf_rn(P.alpha, hv[j], gv[j]);
                    cb[j] = 0x4B400000u + P.s;
                    hn[j] = (bs.kind == 1) ? __fmaf_rn(P.beta, hv[j], P.mode ? v : gv[j]) : hv[j];
                }
            }
            *reinterpret_cast<float4*>(hout_row + (((uint32_t)c << 4) ^ sw)) =
                make_float4(hn[0], hn[1], hn[2], hn[3]);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                acc += (uint64_t)cb[j] * (uint64_t)(1u << nbits);
                junk += (uint64_t)0x4B400000u << nbits;
                nbits += R;
                if (nbits >= 32) {
                    acc -= junk; junk = 0;
                    wout[kw++] = (uint32_t)acc;
                    acc >>= 32;
                    nbits -= 32;
                }
            }
        }
        if constexpr (R % 4 == 0) {
#pragma unroll
            for (int q = 0; q < R / 4; ++q)
                reinterpret_cast<uint4*>(cout_row)[q] =
                    make_uint4(wout[4 * q], wout[4 * q + 1], wout[4 * q + 2], wout[4 * q + 3]);
        } else if constexpr (R % 2 == 0) {
#pragma unroll
            for (int q = 0; q < R / 2; ++q)
                reinterpret_cast<uint2*>(cout_row)[q] = make_uint2(wout[2 * q], wout[2 * q + 1]);
        } else {
#pragma unroll
            for (int q = 0; q < R; ++q) cout_row[q] = wout[q];
        }
        fence_proxy_async_smem();               // my writes -> visible to the TMA stores
        __syncthreads();
        if (tid == 0) {
            tma_store_2d(&tm_h, 0, (int)(tile * kTileRows), base + L::kHoutOff);
            bulk_store_1d(codes + (uint64_t)tile * (R * kTileRows), base + L::kCoutOff, L::kCodeBytes);
            bulk_commit();
        }
    }
    if (tid == 0) {
        if (*s_abort) mbar_wait(bar_full, parity);   // let a load still in flight land
        bulk_wait_all();
    }
    __syncthreads();
    if (*s_abort) return;

    // ragged end: the buckets after the last whole tile, spread over the CTAs from
    // the back of the grid
    const uint64_t tail_first = (uint64_t)n_tiles * buckets_per_tile;
    const uint64_t nb_total = (P.d + P.bucket - 1) / P.bucket;
    uint32_t* s_red = reinterpret_cast<uint32_t*>(sm);   // the buffers are idle now
    for (uint64_t b = tail_first + (gridDim.x - 1 - blockIdx.x); b < nb_total; b += gridDim.x)
        encode_bucket_generic<kEncodeThreads>(P, b, worker, step, g, h, codes, scales, status,
                                              s_red, tid);
}

}  // namespace ecq
