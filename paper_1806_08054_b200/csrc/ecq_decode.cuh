// Receiver-side kernel: unpack -> dequantise -> W-way mean (Eq. 4; Algorithm 1, phase 2,
// global-gradient step).
#pragma once

#include "ecq_common.cuh"

namespace ecq {

struct MessageTable {
    const uint32_t* codes[64];
    const float* scales[64];
};

// Where a decoded mean goes: to `out` (may be null), and, for the fused model update of
// Algorithm 1 (phase 2, model-update step: w <- w - eta * g~), into `params` (may be null).
// More than 64 messages are summed over several launches of 64: every launch but the first
// starts from the running sums a previous one left in `out` (first == 0), and every launch
// but the last leaves its running sums there instead of the mean (last == 0).  The chain of
// multiply-adds is the same as in one pass.  (DecodeSlice below.)
struct DecodeOut {
    float* out;
    float* params;
    float neg_eta;
};
struct DecodeSlice {
    float w_total;      // number of messages of the whole mean (the divisor)
    int first, last;
};
__device__ __forceinline__ void emit1(const DecodeOut& o, uint64_t i, float v) {
    if (o.params) o.params[i] = __fmaf_rn(o.neg_eta, v, o.params[i]);
    if (o.out) o.out[i] = v;
}
__device__ __forceinline__ void emit4(const DecodeOut& o, uint64_t i, float4 v) {
    if (o.params) {
        float4 p = *reinterpret_cast<const float4*>(o.params + i);
        p.x = __fmaf_rn(o.neg_eta, v.x, p.x); p.y = __fmaf_rn(o.neg_eta, v.y, p.y);
        p.z = __fmaf_rn(o.neg_eta, v.z, p.z); p.w = __fmaf_rn(o.neg_eta, v.w, p.w);
        *reinterpret_cast<float4*>(o.params + i) = p;
    }
    if (o.out) *reinterpret_cast<float4*>(o.out + i) = v;
}

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
                   const DecodeOut dst, const uint64_t n_groups, const uint64_t n_words,
                   const float w_recip, const int w_pow2, const DecodeSlice sl) {
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
        for (int j = 0; j < G; ++j) acc[j] = (sl.first || i0 + j >= P.d) ? 0.f : dst.out[i0 + j];
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
        if (!sl.last) {
#pragma unroll
            for (int j = 0; j < G; ++j)
                if (i0 + j < P.d) dst.out[i0 + j] = acc[j];
            continue;
        }
#pragma unroll
        for (int j = 0; j < G; ++j)
            acc[j] = w_pow2 ? __fmul_rn(acc[j], w_recip) : __fdiv_rn(acc[j], sl.w_total);
        if (i0 + G <= P.d) {
#pragma unroll
            for (int j = 0; j < G; j += 4)
                emit4(dst, i0 + j, make_float4(acc[j], acc[j + 1], acc[j + 2], acc[j + 3]));
        } else {
#pragma unroll
            for (int j = 0; j < G; ++j)
                if (i0 + j < P.d) emit1(dst, i0 + j, acc[j]);
        }
    }
}

// Any code width (r up to 16): 32 entries per thread, run-time shifts.
__global__ void __launch_bounds__(256)
decode_mean_generic_kernel(const CodecParams P, const uint32_t W,
                           const __grid_constant__ MessageTable tab, const DecodeOut dst,
                           const uint64_t n_groups, const uint64_t n_words, const float w_recip,
                           const int w_pow2, const DecodeSlice sl) {
    const uint32_t r = P.r, mask = (1u << r) - 1u;
    const float magic = 8388608.f + (float)P.s;
    for (uint64_t gi = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; gi < n_groups;
         gi += (uint64_t)gridDim.x * blockDim.x) {
        const uint64_t i0 = gi * 32;
        const uint64_t b = i0 / P.bucket;
        const uint64_t w0 = gi * r;
        for (int j = 0; j < 32 && i0 + j < P.d; ++j) {
            const uint32_t bit = j * r, wi = bit >> 5, sh = bit & 31;
            float acc = sl.first ? 0.f : dst.out[i0 + j];
            for (uint32_t w = 0; w < W; ++w) {
                const float a = __fdiv_rn(__ldg(tab.scales[w] + b), P.sf);
                const uint32_t lo = __ldg(tab.codes[w] + w0 + wi);
                const uint32_t hi = (sh + r > 32 && w0 + wi + 1 < n_words)
                                        ? __ldg(tab.codes[w] + w0 + wi + 1) : 0u;
                const uint32_t c = __funnelshift_r(lo, hi, sh) & mask;
                const float q = __fsub_rn(__uint_as_float(0x4B000000u | c), magic);
                acc = __fmaf_rn(q, a, acc);
            }
            if (!sl.last) dst.out[i0 + j] = acc;
            else emit1(dst, i0 + j, w_pow2 ? __fmul_rn(acc, w_recip) : __fdiv_rn(acc, sl.w_total));
        }
    }
}


// Ragged end of a vector behind its last whole tile of 1024 outputs: one thread per output,
// the chain of Eq. 4 as in decode_mean_generic_kernel.  The loads of eight messages are issued
// before the first of them is used (one message at a time, each turn of the loop waits for a
// trip to DRAM: 32 messages kept the last CTA 10 us beyond the others), and the outputs go to
// the CTAs from the end of the grid, which are the ones with the fewest tiles.
template <int R>
__device__ __forceinline__ void decode_ragged_end(const CodecParams& P, const uint32_t W,
                                                  const MessageTable& tab, const DecodeOut& dst,
                                                  const uint64_t tail0, const uint64_t n_words,
                                                  const bool first, const bool last, const float w_recip,
                                                  const int w_pow2, const float w_total) {
    constexpr uint32_t mask = (1u << R) - 1u;
    const float magic = 8388608.f + P.sf;
    const uint32_t rev = gridDim.x - 1u - blockIdx.x;
    for (uint64_t i = tail0 + (uint64_t)rev * blockDim.x + threadIdx.x; i < P.d;
         i += (uint64_t)gridDim.x * blockDim.x) {
        const uint64_t b = i / P.bucket, bit = i * R, wi = bit >> 5;
        const uint32_t sh = (uint32_t)(bit & 31);
        const bool two = sh + R > 32 && wi + 1 < n_words;
        float acc1 = first ? 0.f : dst.out[i];
        for (uint32_t w0 = 0; w0 < W; w0 += 8) {
            float sc[8];
            uint32_t lo[8], hi[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const bool in = w0 + k < W;
                sc[k] = in ? __ldg(tab.scales[w0 + k] + b) : 0.f;
                lo[k] = in ? __ldg(tab.codes[w0 + k] + wi) : 0u;
                hi[k] = (in && two) ? __ldg(tab.codes[w0 + k] + wi + 1) : 0u;
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                if (w0 + k < W) {
                    const float a = __fdiv_rn(sc[k], P.sf);
                    const uint32_t c = __funnelshift_r(lo[k], hi[k], sh) & mask;
                    acc1 = __fmaf_rn(__fsub_rn(__uint_as_float(0x4B000000u | c), magic), a, acc1);
                }
            }
        }
        if (!last) dst.out[i] = acc1;
        else emit1(dst, i, w_pow2 ? __fmul_rn(acc1, w_recip) : __fdiv_rn(acc1, w_total));
    }
}

// ===========================================================================
// Tiled path.  Every warp works on its own: a tile is 1024 outputs, one run of
// 32 consecutive entries ("row") per lane, whose codes are R whole words.
//   * the code words of (tile, worker) -- R*128 contiguous bytes -- are copied
//     into a warp-private ring with 16-byte asynchronous copies, kRing-1 units
//     ahead, so that global loads are coalesced and plentiful while each lane
//     reads its own R words from shared memory without bank conflicts;
//   * the level steps a_w = scale_w / s of the lane's bucket are loaded one
//     tile ahead, one worker per lane, and broadcast by shuffles;
//   * each code is turned into a float without a shift or a conversion where
//     its bit field allows it: (word & field) | 0x4B000000 is 2^23 + c*2^p, so
//     one add gives (c - s)*2^p exactly; the power of two is carried through
//     the sum (a_w is pre-scaled by 2^-22, exact) and undone once per output,
//     so the terms are summed in ascending w exactly as Eq. 4 is written out;
//     the subtract and the multiply-add run as packed fp32x2 instructions, two
//     outputs at a time;
//   * the 32x32 block of means goes through a swizzled staging buffer so that
//     the stores to `out` are fully coalesced.
// ===========================================================================
constexpr int kDecTileElems = 1024;
constexpr int kDecWarps = 8;
constexpr int kDecAreg = 8;                 // level steps loaded per lane and tile

template <int R> struct DecodeTiled {
    static constexpr int kRing = (R <= 3) ? 16 : (R <= 8 ? 8 : 6);
    static constexpr int kUnitBytes = R * 128;
    static constexpr int kFit = (23 / R) & ~1;   // whole fields below bit 23 of a word, even
    static constexpr int kATabBytes = kDecAreg * 32 * 8;          // (a_w, a_w) per (lane group, worker)
    static constexpr int kWarpBytes = kRing * kUnitBytes + 4096 + kATabBytes;
    static constexpr int kSmem = kDecWarps * kWarpBytes;
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() {
    asm volatile("cp.async.commit_group;" ::: "memory");
}
template <int N> __device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// CARRY: the launch is one slice of a longer sum (`sl` is honoured); without it the launch
// is the whole sum over W messages.
template <int R, bool CARRY>
__global__ void __launch_bounds__(kDecWarps * 32)
decode_tiled_kernel(const CodecParams P, const uint32_t W, const __grid_constant__ MessageTable tab,
                    const DecodeOut dst, const uint32_t n_tiles, const uint64_t n_words,
                    const float w_recip, const int w_pow2, const uint32_t exp23_bits,
                    const DecodeSlice sl) {
    using L = DecodeTiled<R>;
    const bool first = CARRY ? sl.first != 0 : true, last = CARRY ? sl.last != 0 : true;
    const float w_total = CARRY ? sl.w_total : (float)W;
    constexpr int D = L::kRing;
    constexpr int FIT = L::kFit;
    constexpr uint32_t mask = (1u << R) - 1u;
    extern __shared__ __align__(128) uint8_t dsm[];
    const int lane = threadIdx.x & 31;
    // broadcast from lane 0: the compiler then knows the value is warp-uniform and keeps the
    // per-warp bookkeeping (ring slots, unit counters, pointers) on the uniform datapath
    const int warp = __shfl_sync(0xFFFFFFFFu, (int)(threadIdx.x >> 5), 0);
    uint8_t* const ring = dsm + warp * L::kWarpBytes;
    uint8_t* const stage = ring + D * L::kUnitBytes;
    float2* const a_tab = reinterpret_cast<float2*>(stage + 4096);
    const uint32_t ring_u32 = smem_u32(ring);

    // nothing above touches global memory: the launch may overlap the previous kernel's end
    griddep_launch();
    griddep_wait();
    const uint32_t n_warps = gridDim.x * kDecWarps;
    // Warp k of CTA b is warp number k * gridDim + b of the launch and takes every
    // n_warps-th tile from there.  The warps that get one tile more than the others (n_tiles
    // is seldom a multiple of n_warps) are then spread evenly over the SMs; numbered CTA by
    // CTA they would fill whole CTAs, and the SMs holding those would finish a tile per warp
    // after the rest (3.6 % of a launch over 25 M outputs).
    const uint32_t gw = (uint32_t)warp * gridDim.x + blockIdx.x;
    const uint32_t my_tiles = gw < n_tiles ? (n_tiles - gw + n_warps - 1) / n_warps : 0;
    const uint32_t n_units = my_tiles * W;                          // < 2^32: checked by the host

    // lanes that share a bucket: gsz consecutive lanes (all 32 above 1024 entries);
    // a_tab holds, per group of lanes, a_w for w < W (W <= kDecAreg * gsz)
    const uint32_t gsz = P.bucket >= 1024u ? 32u : (P.bucket >> 5);
    const uint32_t gl = lane & (gsz - 1);
    const uint32_t bucket_shift = 31 - __clz(P.bucket);           // bucket is a power of two
    const uint32_t n_slots = (W + gsz - 1) / gsz;                   // <= kDecAreg
    float2* const a_mine = a_tab + (lane / gsz) * (kDecAreg * gsz);
    // Level steps enter the table as a_w 2^-22 (against the 2^(iR) of the fields) and, when the
    // whole mean is taken here over a power-of-two number of messages, divided by it as well:
    // powers of two, so the chain's roundings are those of Eq. 4 and the stored mean needs one
    // multiply.  With s a power of two the division scale / s is a multiplication too.
    const bool pre_w = !CARRY && w_pow2;
    const bool s_pow2 = (P.s & (P.s - 1u)) == 0u;
    const float k_pre = pre_w ? __fmul_rn(0x1p-22f, w_recip) : 0x1p-22f;
    const float a_mul = s_pow2 ? __fdiv_rn(k_pre, P.sf) : k_pre;

    // 2^23 + s * 2^(iR): subtracting it from (field | 0x4B000000) leaves (c - s) * 2^(iR)
    uint64_t T2[FIT / 2];
#pragma unroll
    for (int i = 0; i < FIT; i += 2)
        T2[i / 2] = pack2(__fmaf_rn(P.sf, (float)(1u << (i * R)), 8388608.f),
                          __fmaf_rn(P.sf, (float)(1u << ((i + 1) * R)), 8388608.f));

    // 2^23 exponent bits for both halves, kept in registers so that mask-and-merge is
    // one logic instruction per field
    // (exp23_bits = 0x4B000000 arrives as a kernel argument so that it lives in a register:
    // a logic instruction takes one immediate, and the field mask is it)
    const uint64_t magic2 = ((uint64_t)exp23_bits << 32) | exp23_bits;

    // ---- asynchronous copy of unit n = (tile index n / W, worker n % W) ----
    uint32_t cp_tile = gw, cp_w = 0, cp_slot = 0;
    uint32_t cp_unit = 0;
    auto issue_unit = [&]() {
        if (cp_unit < n_units) {
            const uint32_t* src = tab.codes[cp_w] + (uint64_t)cp_tile * (R * 32);
            const uint32_t dst = ring_u32 + cp_slot;
#pragma unroll
            for (int p = 0; p < (8 * R + 31) / 32; ++p) {
                const int piece = p * 32 + lane;
                if (piece < 8 * R) cp_async16(dst + piece * 16, src + piece * 4);
            }
            if (++cp_w == W) { cp_w = 0; cp_tile += n_warps; }
            ++cp_unit;
            cp_slot += L::kUnitBytes;
            if (cp_slot == D * L::kUnitBytes) cp_slot = 0;
        }
        cp_async_commit();
    };
    // ---- scales of my bucket for one tile: worker k*gsz + gl in slot k ----
    // (With no more messages than lanes in a group -- the usual case -- a lane has one slot:
    // the unrolled loop over all eight would issue its predicated-off instructions all the
    // same, which shows once the per-tile work is spread over few messages.)
    auto load_scales = [&](uint32_t tile, float (&dst)[kDecAreg]) {
        const uint64_t b = ((uint64_t)tile * kDecTileElems + (uint32_t)lane * 32) >> bucket_shift;
        if (n_slots == 1) {
            dst[0] = (gl < W) ? __ldg(tab.scales[gl] + b) : 0.f;
            return;
        }
#pragma unroll
        for (int k = 0; k < kDecAreg; ++k) {
            if (k < (int)n_slots) {
                const uint32_t w = k * gsz + gl;
                dst[k] = (w < W) ? __ldg(tab.scales[w] + b) : 0.f;
            }
        }
    };

#pragma unroll 1
    for (int i = 0; i < D - 1; ++i) issue_unit();
    float nxt[kDecAreg];
    if (my_tiles) load_scales(gw, nxt);

    uint32_t rd_slot = 0;
    for (uint32_t ti = 0; ti < my_tiles; ++ti) {
        const uint32_t tile = gw + ti * n_warps;
        // a_w = scale_w / s, pre-scaled by 2^-22 (exact; only scales below 2^-104 lose
        // bits, far under the absolute tolerance) against the 2^(iR) of the fields
        if (n_slots == 1) {
            const float a = s_pow2 ? __fmul_rn(nxt[0], a_mul) : __fmul_rn(__fdiv_rn(nxt[0], P.sf), a_mul);
            a_mine[gl] = make_float2(a, a);
        } else {
#pragma unroll
            for (int k = 0; k < kDecAreg; ++k)
                if (k < (int)n_slots) {
                    const float a = s_pow2 ? __fmul_rn(nxt[k], a_mul) : __fmul_rn(__fdiv_rn(nxt[k], P.sf), a_mul);
                    a_mine[k * gsz + gl] = make_float2(a, a);
                }
        }
        __syncwarp();
        if (ti + 1 < my_tiles) load_scales(tile + n_warps, nxt);

        uint64_t acc2[16];                      // outputs (2k, 2k+1) as fp32 pairs
#pragma unroll
        for (int j = 0; j < 16; ++j) acc2[j] = 0ull;
        if (!first) {
            // running sums of the earlier messages: coalesced loads, transposed through the
            // staging buffer to one row per lane, and given the powers of two of their fields
            const float* src = dst.out + (uint64_t)tile * kDecTileElems;
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int idx = k * 32 + lane, row = idx >> 3, ch = idx & 7;
                *reinterpret_cast<float4*>(stage + row * 128 + ((ch ^ (row & 7)) << 4)) =
                    *reinterpret_cast<const float4*>(src + idx * 4);
            }
            __syncwarp();
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const float4 v = *reinterpret_cast<const float4*>(stage + lane * 128 + ((c ^ (lane & 7)) << 4));
                const float in[4] = {v.x, v.y, v.z, v.w};
                float sc[4];
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    sc[q] = __fmul_rn(in[q], __uint_as_float((uint32_t)(127 - 22 + ((4 * c + q) % FIT) * R) << 23));
                acc2[2 * c] = pack2(sc[0], sc[1]);
                acc2[2 * c + 1] = pack2(sc[2], sc[3]);
            }
            __syncwarp();
        }

#pragma unroll 1
        for (uint32_t w = 0; w < W; ++w) {
            cp_async_wait<D - 2>();             // my pieces of this unit have landed
            __syncwarp();                       // everyone's have; the previous unit is read out
            issue_unit();                       // kRing-1 units ahead, into the slot just freed
            const uint64_t a2 = *reinterpret_cast<const uint64_t*>(a_mine + w);   // (a_w, a_w)
            const uint32_t* cwp = reinterpret_cast<const uint32_t*>(ring + rd_slot) + lane * R;
            uint32_t cw[R + 1];
            if constexpr (R % 4 == 0) {
#pragma unroll
                for (int q = 0; q < R / 4; ++q) {
                    const uint4 v = reinterpret_cast<const uint4*>(cwp)[q];
                    cw[4 * q] = v.x; cw[4 * q + 1] = v.y; cw[4 * q + 2] = v.z; cw[4 * q + 3] = v.w;
                }
            } else if constexpr (R % 2 == 0) {
#pragma unroll
                for (int q = 0; q < R / 2; ++q) {
                    const uint2 v = reinterpret_cast<const uint2*>(cwp)[q];
                    cw[2 * q] = v.x; cw[2 * q + 1] = v.y;
                }
            } else {
#pragma unroll
                for (int q = 0; q < R; ++q) cw[q] = cwp[q];
            }
            cw[R] = 0u;
            // groups of FIT consecutive codes: one funnel shift brings the group's first
            // field to bit 0, then every field lies below bit 23
#pragma unroll
            for (int j0 = 0; j0 < 32; j0 += FIT) {
                const int bit = j0 * R, wi = bit >> 5, sh = bit & 31;
                const uint32_t word = (sh == 0) ? cw[wi]
                                    : (sh + FIT * R <= 32 || wi + 1 >= R) ? (cw[wi] >> sh)
                                    : __funnelshift_r(cw[wi], cw[wi + 1], sh);
                // both halves of a 64-bit pair hold the word: one 64-bit and/or then yields
                // the float bits of two fields side by side, ready for the packed arithmetic
                const uint64_t w2 = ((uint64_t)word << 32) | word;
#pragma unroll
                for (int i = 0; i < FIT && j0 + i < 32; i += 2) {
                    const uint64_t m2 = ((uint64_t)(mask << ((i + 1) * R)) << 32) | (uint64_t)(mask << (i * R));
                    // (c - s) 2^(iR) a, two outputs per instruction
                    acc2[(j0 + i) / 2] = fma2(sub2((w2 & m2) | magic2, T2[i / 2]), a2, acc2[(j0 + i) / 2]);
                }
            }
            rd_slot += L::kUnitBytes;
            if (rd_slot == D * L::kUnitBytes) rd_slot = 0;
        }

        // undo the powers of two, divide by W
        float acc[32];
#pragma unroll
        for (int j = 0; j < 16; ++j) unpack2(acc2[j], acc[2 * j], acc[2 * j + 1]);
        if (!last || pre_w) {
#pragma unroll
            for (int j = 0; j < 32; ++j)
                acc[j] = __fmul_rn(acc[j], __uint_as_float((uint32_t)(127 + 22 - (j % FIT) * R) << 23));
        } else if (w_pow2) {
#pragma unroll
            for (int j = 0; j < 32; ++j)
                acc[j] = __fmul_rn(__fmul_rn(acc[j], __uint_as_float((uint32_t)(127 + 22 - (j % FIT) * R) << 23)), w_recip);
        } else {
#pragma unroll
            for (int j = 0; j < 32; ++j)
                acc[j] = __fdiv_rn(__fmul_rn(acc[j], __uint_as_float((uint32_t)(127 + 22 - (j % FIT) * R) << 23)), w_total);
        }
        // transpose through the staging buffer: row-per-lane -> coalesced 16-byte stores
#pragma unroll
        for (int c = 0; c < 8; ++c)
            *reinterpret_cast<float4*>(stage + lane * 128 + ((c ^ (lane & 7)) << 4)) =
                make_float4(acc[4 * c], acc[4 * c + 1], acc[4 * c + 2], acc[4 * c + 3]);
        __syncwarp();
        const uint64_t o = (uint64_t)tile * kDecTileElems;
        if (last && dst.params) {
            // with the fused model update (one branch per tile, not a predicate per store)
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int idx = k * 32 + lane, row = idx >> 3, ch = idx & 7;
                const float4 v = *reinterpret_cast<const float4*>(stage + row * 128 + ((ch ^ (row & 7)) << 4));
                emit4(dst, o + idx * 4, v);
            }
        } else {
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int idx = k * 32 + lane, row = idx >> 3, ch = idx & 7;
                const float4 v = *reinterpret_cast<const float4*>(stage + row * 128 + ((ch ^ (row & 7)) << 4));
                *reinterpret_cast<float4*>(dst.out + o + idx * 4) = v;
            }
        }
        __syncwarp();
    }
    cp_async_wait<0>();

    decode_ragged_end<R>(P, W, tab, dst, (uint64_t)n_tiles * kDecTileElems, n_words, first, last, w_recip,
                         w_pow2, w_total);
}

}  // namespace ecq
