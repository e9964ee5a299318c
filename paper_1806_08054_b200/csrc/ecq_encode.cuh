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
constexpr uint32_t kMaxL2Runs = 1024;       // any-shape path: l2 buckets of up to 32768 entries

template <int NT>
__device__ void encode_bucket_generic(const CodecParams& P, uint64_t b, uint32_t worker,
                                      uint32_t step, const float* __restrict__ g, float* h,
                                      uint32_t* __restrict__ codes, float* __restrict__ scales,
                                      uint32_t* status, uint32_t* s_red, float* s_runs, int tid) {
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
    if (P.norm == 1 && m < 0x7F800000u) {
        // l2 scale in the stated order: every run of 32 entries front to back with one fma
        // per entry, then the run sums pairwise in index order, level by level (ping-pong
        // between the two halves of s_runs; at most kMaxL2Runs runs)
        const uint32_t n_runs = (n + 31) >> 5;
        for (uint32_t run = tid; run < n_runs; run += NT) {
            float acc = 0.f;
            const uint32_t e0 = run * 32, e1 = min(n, e0 + 32);
            for (uint32_t j = e0; j < e1; ++j) {
                const float v = __fmaf_rn(P.alpha, hb[j], gb[j]);
                acc = __fmaf_rn(v, v, acc);
            }
            s_runs[run] = acc;
        }
        __syncthreads();
        uint32_t cnt = n_runs, src = 0;
        while (cnt > 1) {
            const uint32_t up = (cnt + 1) >> 1, dst = src ^ kMaxL2Runs;
            for (uint32_t k = tid; k < up; k += NT)
                s_runs[dst + k] = (2 * k + 1 < cnt) ? __fadd_rn(s_runs[src + 2 * k], s_runs[src + 2 * k + 1])
                                                    : s_runs[src + 2 * k];
            __syncthreads();
            cnt = up; src = dst;
        }
        m = __float_as_uint(s_runs[src]) & 0x7FFFFFFFu;
        __syncthreads();
    }
    const BucketScale bs = bucket_scale(m, P.sf, P.norm);
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
    __shared__ float s_runs[2 * kMaxL2Runs];
    for (uint64_t b = blockIdx.x; b < n_buckets; b += gridDim.x)
        encode_bucket_generic<NT>(P, first_bucket + b, worker, step, g, h, codes, scales, status,
                                  s_red, s_runs, threadIdx.x);
}

// ===========================================================================
// Tiled path.  The vector is seen as a matrix of 128-byte rows (32 floats); a
// tile is 256 rows = 8192 entries = a whole number of buckets (bucket a power
// of two <= 4096).  A persistent CTA of 256 threads (two per SM) owns one
// 64 KiB load buffer and one store staging buffer and walks its tiles:
//   * thread 0 issues two 32 KiB TMA loads (g and h tile, 128-byte swizzle);
//     measured on B200, a TMA operation costs ~200 cycles of issue time
//     whatever its size, so tiles are moved with few, maximal operations (a box
//     of 256 rows is the largest a tensor map allows; 16 KiB boxes with four
//     CTAs per SM ran 7 % slower);
//   * every thread copies its row of g and h to registers (the swizzle makes
//     the eight 16-byte chunks of a row conflict-free across the warp); after
//     one CTA barrier the buffer is refilled with the next tile, which lands
//     while this one is being computed;
//   * the scale of the bucket (max of |g + alpha h|, or its l2 norm) is combined
//     over the rows of a bucket by shuffles (and through shared memory when a
//     bucket spans 2 or 4 warps);
//   * each thread draws Philox per 4 entries, rounds, forms the new h row in
//     registers and packs its 32 codes into R words; both go to the staging
//     buffer, from which thread 0 issues one TMA store (h tile) and one linear
//     bulk store (code words).
// g and h are read from HBM once, h is written once; v never leaves the SM.
// ===========================================================================
// Two tile shapes share the code: 256 rows (32 KiB operations, two CTAs per SM) and 128 rows
// (16 KiB operations, four CTAs per SM).  Measured on B200: the large shape is 5-8 % faster
// in launches of up to a few milliseconds (6.5 vs 6.1 TB/s), the small one sustains 3 % more
// in launches long enough to run into the board's power cap (6.0 vs 5.85 TB/s).
template <int ROWS> struct EncodeTile {
    static constexpr int kRows = ROWS;
    static constexpr int kElems = ROWS * 32;        // one thread per row of 32 entries
    static constexpr int kBytes = kElems * 4;       // per operand
    static constexpr int kThreads = ROWS;
    static constexpr int kCtasPerSm = 512 / ROWS;
};
constexpr uint32_t kMaxTiledBucket = 4096;          // largest bucket of the tiled path (4 warps)

template <int R, int ROWS>
struct EncodeSmem {
    static constexpr int kTileBytes = EncodeTile<ROWS>::kBytes;
    static constexpr int kCodeBytes = R * (EncodeTile<ROWS>::kElems / 8);
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

// The buffers of the workers that one launch serves (a batch may hold one worker).
constexpr int kMaxBatch = 64;
struct alignas(64) EncodeBatch {
    CUtensorMap tm_g[kMaxBatch];    // tiled views of grad (loads)
    CUtensorMap tm_h[kMaxBatch];    // tiled views of err (loads and stores)
    const float* g[kMaxBatch];
    float* h[kMaxBatch];
    uint32_t* codes[kMaxBatch];
    float* scales[kMaxBatch];
};

// One launch walks the tiles of n_workers vectors: global tile T is tile T % n_tiles
// of batch entry T / n_tiles, whose Philox stream is that of worker worker_base + entry.
template <int R, bool MODE1, int ROWS>
__global__ void __launch_bounds__(EncodeTile<ROWS>::kThreads, EncodeTile<ROWS>::kCtasPerSm)
encode_tiled_kernel(const __grid_constant__ EncodeBatch bt, const CodecParams P,
                    const uint32_t worker_base, const uint32_t n_workers, const uint32_t step,
                    uint32_t* status, const uint32_t n_tiles, const uint32_t wait_limit) {
    using L = EncodeSmem<R, ROWS>;
    constexpr int kTileRows = ROWS, kTileElems = EncodeTile<ROWS>::kElems;
    constexpr int kTileBytes = EncodeTile<ROWS>::kBytes, kEncodeThreads = ROWS;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* const sm = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bar_full = base + L::kBarOff;
    volatile uint32_t* s_abort = reinterpret_cast<volatile uint32_t*>(sm + L::kMiscOff);
    uint32_t* s_wmax = reinterpret_cast<uint32_t*>(sm + L::kMiscOff + 16);   // one per warp

    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    const uint32_t total_tiles = n_workers * n_tiles;       // < 2^32: checked by the host
    auto issue_load = [&](uint32_t T) {
        const uint32_t e = T / n_tiles, tile = T - e * n_tiles;
        mbar_arrive_expect_tx(bar_full, 2 * kTileBytes);
        tma_load_2d(base + L::kLoadOff, &bt.tm_g[e], 0, (int)(tile * kTileRows), bar_full);
        tma_load_2d(base + L::kLoadOff + kTileBytes, &bt.tm_h[e], 0, (int)(tile * kTileRows), bar_full);
    };
    griddep_launch();
    griddep_wait();
    if (tid == 0) {
        mbar_init(bar_full, 1);
        *s_abort = 0;
        fence_mbar_init();
        if (blockIdx.x < total_tiles) issue_load(blockIdx.x);
    }
    __syncthreads();

    const uint32_t sw = (uint32_t)(tid & 7) << 4;
    const uint32_t rpb = P.bucket >> 5;                    // rows per bucket, power of two <= 128
    const uint32_t buckets_per_tile = kTileElems / P.bucket;
    const float magic_code = 12582912.f + P.sf;            // 1.5*2^23 + s, exact
    const uint64_t magic2 = pack2(magic_code, magic_code);
    const uint64_t alpha2 = pack2(P.alpha, P.alpha), beta2 = pack2(P.beta, P.beta);
    const uint64_t two23_2 = pack2(8388608.f, 8388608.f), ulp24_2 = pack2(0x1p-24f, 0x1p-24f);
    const uint8_t* const g_row = sm + L::kLoadOff + tid * 128;
    const uint8_t* const h_row = g_row + kTileBytes;
    uint8_t* const hout_row = sm + L::kHoutOff + tid * 128;
    uint32_t* const cout_row = reinterpret_cast<uint32_t*>(sm + L::kCoutOff) + tid * R;

    uint32_t parity = 0;
    for (uint32_t T = blockIdx.x; T < total_tiles; T += gridDim.x, parity ^= 1u) {
        const uint32_t entry = T / n_tiles, tile = T - entry * n_tiles;
        const uint32_t worker = worker_base + entry;
        if (!mbar_wait_n(bar_full, parity, wait_limit)) { *s_abort = 1; atomicOr(status, kStatusTimeout); }

        // my row of g and h -> registers
        float4 G[8], H[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const uint32_t off = ((uint32_t)c << 4) ^ sw;
            G[c] = *reinterpret_cast<const float4*>(g_row + off);
            H[c] = *reinterpret_cast<const float4*>(h_row + off);
        }
        // Eq. 8 scale.  l-infinity: row max of |g + alpha h| (NaN-propagating), then the max
        // over the rows of the bucket.  l2: the row's sum of squares front to back with one
        // fma per entry, then the row sums pairwise in index order (the xor butterfly is that
        // tree, and addition commutes).  Both travel as sign-cleared bit patterns.
        uint32_t m;
        if (P.norm == 0) {
            float mf = 0.f;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                float v0, v1, v2, v3;
                unpack2(fma2(alpha2, pack2(H[c].x, H[c].y), pack2(G[c].x, G[c].y)), v0, v1);
                unpack2(fma2(alpha2, pack2(H[c].z, H[c].w), pack2(G[c].z, G[c].w)), v2, v3);
                mf = max3_abs_nan(mf, v0, v1);
                mf = max3_abs_nan(mf, v2, v3);
            }
            // non-negative floats and NaN (0x7FFFFFFF) order like their bit patterns
            m = __float_as_uint(mf) & 0x7FFFFFFFu;
            for (uint32_t o = 1; o < rpb && o < 32; o <<= 1)
                m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
        } else {
            float ss = 0.f;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                float v0, v1, v2, v3;
                unpack2(fma2(alpha2, pack2(H[c].x, H[c].y), pack2(G[c].x, G[c].y)), v0, v1);
                unpack2(fma2(alpha2, pack2(H[c].z, H[c].w), pack2(G[c].z, G[c].w)), v2, v3);
                ss = __fmaf_rn(v0, v0, ss); ss = __fmaf_rn(v1, v1, ss);
                ss = __fmaf_rn(v2, v2, ss); ss = __fmaf_rn(v3, v3, ss);
            }
            for (uint32_t o = 1; o < rpb && o < 32; o <<= 1)
                ss = __fadd_rn(ss, __shfl_xor_sync(0xFFFFFFFFu, ss, o));
            m = __float_as_uint(ss);
        }
        if (rpb > 32 && lane == 0) s_wmax[warp] = m;
        // The barrier below hands the load buffer to the next tile's copy, so every thread's
        // shared loads of G and H must have completed by then, which the barrier itself does not
        // wait for.  m depends on all of them, and the shuffles above consume it; with one row
        // per bucket there is no shuffle, so one is made here (it returns m).
        if (rpb == 1) m = __shfl_sync(0xFFFFFFFFu, m, lane);
        __syncthreads();                                   // the load buffer is free
        if (*s_abort) break;                               // uniform: set before the barrier
        if (tid == 0 && T + gridDim.x < total_tiles) issue_load(T + gridDim.x);
        if (P.norm == 0) {
            if (rpb == 64) m = max(s_wmax[warp & ~1], s_wmax[warp | 1]);
            if (rpb == 128) { const int w0 = warp & ~3; m = max(max(s_wmax[w0], s_wmax[w0 + 1]), max(s_wmax[w0 + 2], s_wmax[w0 + 3])); }
        } else {
            const float* wf = reinterpret_cast<const float*>(s_wmax);
            float ss = __uint_as_float(m);
            if (rpb == 64) ss = __fadd_rn(wf[warp & ~1], wf[warp | 1]);
            if (rpb == 128) { const int w0 = warp & ~3; ss = __fadd_rn(__fadd_rn(wf[w0], wf[w0 + 1]), __fadd_rn(wf[w0 + 2], wf[w0 + 3])); }
            m = __float_as_uint(ss) & 0x7FFFFFFFu;
        }
        const BucketScale bs = bucket_scale(m, P.sf, P.norm);
        if ((tid & (rpb - 1)) == 0) {
            bt.scales[entry][(uint64_t)tile * buckets_per_tile + tid / rpb] = bs.scale;
            if (bs.kind == 2) atomicOr(status, kStatusNonFinite);
        }

        // round, new h (written over H), pack 32 codes into R words.  The codes enter
        // a 64-bit window as (float bits of q + s + 1.5*2^23) << pos; the constant high
        // bits are removed once per output word.  The fp32 steps run as packed fp32x2
        // instructions on two neighbouring entries (each half is the same IEEE
        // operation as in the scalar form).
        const uint64_t blk0 = (uint64_t)tile * (kTileElems / 4) + (uint32_t)tid * 8;
        uint32_t wout[R];
        uint64_t acc = 0, junk = 0;
        int nbits = 0, kw = 0;
        if (bs.kind == 0) {
            const uint64_t inv2 = pack2(bs.inv, bs.inv);
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                uint32_t Rw[4];
                const uint64_t blk = blk0 + c;
                philox4x32_10(P, (uint32_t)blk, (uint32_t)(blk >> 32), worker, step, Rw);
                uint32_t cb[4];
                float hn[4];
#pragma unroll
                for (int hlf = 0; hlf < 2; ++hlf) {
                    const uint64_t g2 = hlf ? pack2(G[c].z, G[c].w) : pack2(G[c].x, G[c].y);
                    const uint64_t h2 = hlf ? pack2(H[c].z, H[c].w) : pack2(H[c].x, H[c].y);
                    const uint64_t v2 = fma2(alpha2, h2, g2);                       // Eq. 7
                    const uint64_t sgn2 = v2 & 0x8000000080000000ull;
                    float xs0, xs1;
                    unpack2(mul2(v2, inv2), xs0, xs1);                              // |v| s/scale, signed
                    const uint64_t x2 = pack2(fminf(fabsf(xs0), P.sf), fminf(fabsf(xs1), P.sf));
                    const uint64_t lf2 = sub2(add2_rz(x2, two23_2), two23_2);       // floor
                    float f0, f1, u0, u1;
                    unpack2(sub2(x2, lf2), f0, f1);
                    unpack2(mul2(pack2(__uint2float_rn(Rw[2 * hlf] >> 8),
                                       __uint2float_rn(Rw[2 * hlf + 1] >> 8)), ulp24_2), u0, u1);
                    const uint64_t m2 = add2(lf2, pack2((u0 < f0) ? 1.f : 0.f, (u1 < f1) ? 1.f : 0.f));
                    // work on sgn(v)*g so that the level stays non-negative: negation
                    // commutes with rounding, and a zero level leaves g untouched
                    const uint64_t gsn2 = (MODE1 ? v2 : g2) ^ sgn2;
                    // (the product stays scalar: ptxas contracts a packed multiply with a
                    // following packed subtract into one fused operation, which would drop
                    // the rounding of g~ that Eq. 6 books)
                    float m0, m1;
                    unpack2(m2, m0, m1);
                    const uint64_t e2 = sub2(gsn2, pack2(__fmul_rn(m0, bs.a), __fmul_rn(m1, bs.a))) ^ sgn2;
                    unpack2(fma2(beta2, h2, e2), hn[2 * hlf], hn[2 * hlf + 1]);     // Eq. 6
                    const uint64_t c2 = add2(m2 ^ sgn2, magic2);                    // 0x4B400000 + q + s
                    cb[2 * hlf] = (uint32_t)c2;
                    cb[2 * hlf + 1] = (uint32_t)(c2 >> 32);
                }
                H[c] = make_float4(hn[0], hn[1], hn[2], hn[3]);
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
        } else {
            // all levels zero (code s): an all-zero bucket books beta*h + g, a non-finite one
            // keeps h
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                if (bs.kind == 1) {
                    const float gv[4] = {G[c].x, G[c].y, G[c].z, G[c].w};
                    const float hv[4] = {H[c].x, H[c].y, H[c].z, H[c].w};
                    float hn[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        hn[j] = __fmaf_rn(P.beta, hv[j], MODE1 ? __fmaf_rn(P.alpha, hv[j], gv[j]) : gv[j]);
                    H[c] = make_float4(hn[0], hn[1], hn[2], hn[3]);
                }
            }
            uint64_t zacc = 0;
            int zbits = 0, zk = 0;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                zacc |= (uint64_t)P.s << zbits;
                zbits += R;
                if (zbits >= 32) { wout[zk++] = (uint32_t)zacc; zacc >>= 32; zbits -= 32; }
            }
        }
        (void)acc; (void)junk; (void)nbits; (void)kw;

        // the stores of the previous tile must have read the staging buffer
        if (tid == 0) bulk_wait_read0();
        __syncthreads();
#pragma unroll
        for (int c = 0; c < 8; ++c)
            *reinterpret_cast<float4*>(hout_row + (((uint32_t)c << 4) ^ sw)) = H[c];
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
            tma_store_2d(&bt.tm_h[entry], 0, (int)(tile * kTileRows), base + L::kHoutOff);
            bulk_store_1d(bt.codes[entry] + (uint64_t)tile * (R * kTileRows), base + L::kCoutOff,
                          L::kCodeBytes);
            bulk_commit();
        }
    }
    if (tid == 0) {
        if (*s_abort) mbar_wait(bar_full, parity);   // let a load still in flight land
        bulk_wait_all();
    }
    __syncthreads();
    if (*s_abort) return;

    // ragged ends: the buckets after the last whole tile of every vector, spread over the
    // CTAs from the back of the grid
    const uint64_t tail_first = (uint64_t)n_tiles * buckets_per_tile;
    const uint64_t nb_total = (P.d + P.bucket - 1) / P.bucket;
    const uint64_t n_tail = nb_total - tail_first;
    uint32_t* s_red = reinterpret_cast<uint32_t*>(sm);   // the buffers are idle now
    float* s_runs = reinterpret_cast<float*>(sm + 64);
    for (uint64_t k = gridDim.x - 1 - blockIdx.x; k < n_tail * n_workers; k += gridDim.x) {
        const uint32_t e = (uint32_t)(k / n_tail);
        encode_bucket_generic<kEncodeThreads>(P, tail_first + (k - e * n_tail), worker_base + e, step,
                                              bt.g[e], bt.h[e], bt.codes[e], bt.scales[e], status,
                                              s_red, s_runs, tid);
    }
}

}  // namespace ecq
