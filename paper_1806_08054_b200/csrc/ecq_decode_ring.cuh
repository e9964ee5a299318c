// Receiver-side kernel for long vectors: unpack -> dequantise -> W-way mean (Eq. 4;
// Algorithm 1, "compute global gradients"), with the code words brought in by bulk copies
// that a whole CTA shares.
//
// A CTA tile is 16 sub-tiles of 1024 outputs.  Warp k owns sub-tiles k and k + 8; a lane
// owns one run of 32 consecutive outputs ("row") in each, whose codes are R whole words.
//   * unit (tile, worker) = the worker's code words of the tile, R * 2048 contiguous
//     bytes: ONE bulk copy into a ring of stages, signalled on the stage's mbarrier.  A warp
//     that has copied its rows to registers counts itself off the stage; the warp that
//     counts last refills the stage at once with the unit `stages` further on, so no warp
//     is the producer and the ring stays full whichever warp runs ahead.  Per unit a warp
//     spends a wait, two shared loads and one atomic on data movement instead of issuing
//     and tracking its own copies;
//   * the two rows of a lane travel as the two halves of packed fp32x2 registers:
//     (word_A & field, word_B & field) | 2^23 exponent bits is (2^23 + c 2^p) for both rows,
//     one packed subtract leaves ((c - s) 2^p), one packed multiply-add with the pair of
//     level steps (a_A, a_B) of the rows' buckets adds the terms; per worker the chain
//     acc <- fma(q_w, a_w, acc) is the one Eq. 4 writes out, in ascending w;
//   * level steps a_w = scale_w / s of the next tile are fetched with 4-byte asynchronous
//     copies while this tile is summed;
//   * means leave through a swizzled staging buffer so that stores to `out` are coalesced.
#pragma once

#include "ecq_decode.cuh"

namespace ecq {

#ifndef ECQ_RING_WARPS
#define ECQ_RING_WARPS 8
#endif
constexpr int kRingWarps = ECQ_RING_WARPS;
constexpr int kRingSubs = 2 * kRingWarps;                       // sub-tiles per CTA tile
constexpr int kRingTileElems = kRingSubs * kDecTileElems;       // 16384 outputs
// shorter vectors leave the CTAs with too uneven a share of these large tiles
constexpr int kRingMinTilesPerCta = 1;

template <int R> struct DecodeRing {
    static constexpr int kUnitBytes = R * 128 * kRingSubs;
    // about 36 KB of copies in flight per CTA, sized so that two CTAs share an SM up to r = 8
    static constexpr int kStagesRaw = 36864 / kUnitBytes + 1;
    static constexpr int kStages = kStagesRaw < 3 ? 3 : (kStagesRaw > 8 ? 8 : kStagesRaw);
    // whole fields below bit 23 of a word; chosen so that the fewest groups need a shift
    static constexpr int kFit = R == 2 ? 8 : R == 3 ? 7 : R == 4 ? 4 : 23 / R;
    static constexpr int kBarBytes = 256;                        // 2 * kStages mbarriers, then the abort flag
    static constexpr int kStageBytes = 4096;                     // per warp: 32 x 32 floats
    static constexpr int kATabBytes = kDecAreg * 32 * 8;         // per warp: (a_A, a_B) pairs
    static constexpr int kRawBytes = kDecAreg * 32 * 8;          // per warp: raw scales, rows A and B
    static constexpr int kWarpBytes = kStageBytes + kATabBytes + kRawBytes;
    static constexpr int kRingOff = kBarBytes;
    static constexpr int kWarpOff = kRingOff + kStages * kUnitBytes;
    static constexpr int kSmem = kWarpOff + kRingWarps * kWarpBytes;
};

__device__ __forceinline__ void cp_async4(uint32_t dst, const void* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}

// Linear bulk load: 16-byte aligned on both sides, size a multiple of 16; completion is
// counted in bytes on the mbarrier.
__device__ __forceinline__ void bulk_load_1d(uint32_t dst, const void* gsrc, uint32_t bytes,
                                             uint32_t bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(dst), "l"(gsrc), "r"(bytes), "r"(bar)
        : "memory");
}

__device__ __forceinline__ uint32_t atom_add_acq_rel_shared(uint32_t a, uint32_t v) {
    uint32_t old;
    asm volatile("atom.acq_rel.cta.shared::cta.add.u32 %0, [%1], %2;" : "=r"(old) : "r"(a), "r"(v) : "memory");
    return old;
}
__device__ __forceinline__ void st_shared_u32(uint32_t a, uint32_t v) {
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(a), "r"(v) : "memory");
}
__device__ __forceinline__ void lds32(uint32_t a, uint32_t& x) {
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(x) : "r"(a));
}
__device__ __forceinline__ void lds64(uint32_t a, uint32_t& x, uint32_t& y) {
    asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(x), "=r"(y) : "r"(a));
}
__device__ __forceinline__ void lds128(uint32_t a, uint32_t& x, uint32_t& y, uint32_t& z, uint32_t& w) {
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(x), "=r"(y), "=r"(z), "=r"(w) : "r"(a));
}

template <int R, bool CARRY>
__global__ void __launch_bounds__(kRingWarps * 32, 2)
decode_ring_kernel(const CodecParams P, const uint32_t W, const __grid_constant__ MessageTable tab,
                   const DecodeOut dst, const uint32_t n_subs, const uint64_t n_words,
                   const float w_recip, const int w_pow2, const uint32_t exp23_bits,
                   const DecodeSlice sl, uint32_t* status) {
    using L = DecodeRing<R>;
    const bool first = CARRY ? sl.first != 0 : true, last = CARRY ? sl.last != 0 : true;
    const float w_total = CARRY ? sl.w_total : (float)W;
    constexpr int S = L::kStages;
    constexpr int FIT = L::kFit;
    constexpr uint32_t mask = (1u << R) - 1u;
    extern __shared__ __align__(128) uint8_t dsm[];
    const uint32_t sm0 = smem_u32(dsm);
    // [0, 64) full mbarriers; [64, 96) warps still to read a stage; [96, 128) copies issued
    // into a stage so far; [128] abort flag
    const uint32_t bar_full = sm0, cnt_u32 = sm0 + 64;
    uint32_t* const s_issued = reinterpret_cast<uint32_t*>(dsm + 96);
    volatile uint32_t* const s_abort = reinterpret_cast<volatile uint32_t*>(dsm + 128);
    static_assert(S <= 8 && L::kBarBytes >= 132, "barriers, counters and flag fit their area");
    const int lane = threadIdx.x & 31;
    // broadcast from lane 0 so that the compiler knows the value is warp-uniform
    const int warp = __shfl_sync(0xFFFFFFFFu, (int)(threadIdx.x >> 5), 0);
    uint8_t* const stage = dsm + L::kWarpOff + warp * L::kWarpBytes;
    float2* const a_tab = reinterpret_cast<float2*>(stage + L::kStageBytes);
    float* const raw = reinterpret_cast<float*>(stage + L::kStageBytes + L::kATabBytes);

    const uint32_t n_tiles = (n_subs + kRingSubs - 1) / kRingSubs;
    const uint32_t my_tiles =
        blockIdx.x < n_tiles ? (n_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    const uint32_t n_units = my_tiles * W;                          // < 2^32: checked by the host

    if (threadIdx.x == 0) {
        for (int i = 0; i < S; ++i) {
            mbar_init(bar_full + 8 * i, 1);
            reinterpret_cast<uint32_t*>(dsm + 64)[i] = 0;
            s_issued[i] = 0;
        }
        *s_abort = 0;
        fence_mbar_init();
    }
    __syncthreads();

    // lanes that share a bucket: gsz consecutive lanes (all 32 from 1024 entries up); a_tab
    // holds, per group of lanes, (a_w of row A, a_w of row B) for w < W (W <= kDecAreg * gsz)
    const uint32_t gsz = P.bucket >= 1024u ? 32u : (P.bucket >> 5);
    const uint32_t gl = lane & (gsz - 1);
    const uint32_t bucket_shift = 31 - __clz(P.bucket);           // bucket is a power of two
    const uint32_t n_slots = (W + gsz - 1) / gsz;                   // <= kDecAreg
    const uint32_t grp = (lane & ~(gsz - 1)) * kDecAreg;            // my group's first entry
    const uint32_t raw_u32 = smem_u32(raw);

    // 2^23 + s 2^(iR) in both halves: subtracting it from (field | 2^23 bits) leaves
    // (c - s) 2^(iR)
    uint64_t T2[FIT];
#pragma unroll
    for (int i = 0; i < FIT; ++i) {
        const float t = __fmaf_rn(P.sf, (float)(1u << (i * R)), 8388608.f);
        T2[i] = pack2(t, t);
    }
    // the exponent bits arrive as a kernel argument so that they live in a register: a
    // logic instruction takes one immediate, and the field mask is it
    const uint64_t magic2 = ((uint64_t)exp23_bits << 32) | exp23_bits;

    // ---- one bulk copy: the code words of (tile, worker w) into stage `slot` ----
    auto issue_unit = [&](uint32_t tile, uint32_t w, uint32_t slot) {
        const uint32_t subs = min((uint32_t)kRingSubs, n_subs - tile * kRingSubs);
        const uint32_t bytes = subs * (R * 128);
        const uint32_t bar = bar_full + 8 * slot;
        s_issued[slot] += 1;
        mbar_arrive_expect_tx(bar, bytes);
        bulk_load_1d(sm0 + L::kRingOff + slot * L::kUnitBytes,
                     tab.codes[w] + (uint64_t)tile * (R * 32 * kRingSubs), bytes, bar);
    };

    // ---- raw scales of a tile's buckets: worker k*gsz + gl of my group, rows A and B ----
    auto fetch_scales = [&](uint32_t tile) {
#pragma unroll
        for (int row = 0; row < 2; ++row) {
            const uint32_t sub = tile * kRingSubs + warp + row * kRingWarps;
            if (sub < n_subs) {
                const uint64_t b = ((uint64_t)sub * kDecTileElems + (uint32_t)lane * 32) >> bucket_shift;
#pragma unroll
                for (int k = 0; k < kDecAreg; ++k) {
                    const uint32_t w = k * gsz + gl;
                    if (k < (int)n_slots && w < W)
                        cp_async4(raw_u32 + ((grp + w) * 2 + row) * 4, tab.scales[w] + b);
                }
            }
        }
        cp_async_commit();
    };

    bool ok = true;
    // (r_tile, r_w): the unit `S` units after the one a warp takes next, i.e. the refill of its stage
    uint32_t r_tile = blockIdx.x, r_w = 0;
    for (uint32_t u = 0; u < (uint32_t)S; ++u) {
        if (threadIdx.x == 0 && u < n_units) issue_unit(r_tile, r_w, u);
        if (++r_w == W) { r_w = 0; r_tile += gridDim.x; }
    }
    if (my_tiles) fetch_scales(blockIdx.x);

    // consumer state: ring offset and phase of the next unit to read, units still to take
    uint32_t c_off = 0, c_par = 0, c_left = n_units;
    const uint32_t my_off = sm0 + L::kRingOff + warp * (R * 128) + lane * (R * 4);
    uint32_t cwa[2][R];
    // waits for the next unit, copies my two rows' words to registers, frees the stage
    auto take_unit = [&](uint32_t (&dstw)[2][R]) -> bool {
        const uint32_t slot = c_off / L::kUnitBytes;
        if (!__all_sync(0xFFFFFFFFu, mbar_wait(bar_full + slot * 8, c_par))) return false;
#pragma unroll
        for (int row = 0; row < 2; ++row) {
            const uint32_t src = my_off + c_off + row * (kRingWarps * R * 128);
            if constexpr (R % 4 == 0) {
#pragma unroll
                for (int q = 0; q < R / 4; ++q)
                    lds128(src + 16 * q, dstw[row][4 * q], dstw[row][4 * q + 1], dstw[row][4 * q + 2],
                           dstw[row][4 * q + 3]);
            } else if constexpr (R % 2 == 0) {
#pragma unroll
                for (int q = 0; q < R / 2; ++q) lds64(src + 8 * q, dstw[row][2 * q], dstw[row][2 * q + 1]);
            } else {
#pragma unroll
                for (int q = 0; q < R; ++q) lds32(src + 4 * q, dstw[row][q]);
            }
        }
        __syncwarp();                               // every lane's loads are ordered before ...
        if (lane == 0) {
            // ... the count (release); the last of the CTA's warps to count has all the others'
            // loads behind it (acquire), resets the counter and refills the stage
            if (atom_add_acq_rel_shared(cnt_u32 + slot * 4, 1u) == (uint32_t)kRingWarps - 1u) {
                st_shared_u32(cnt_u32 + slot * 4, 0u);
                if (c_left > (uint32_t)S) issue_unit(r_tile, r_w, slot);
            }
        }
        if (++r_w == W) { r_w = 0; r_tile += gridDim.x; }
        --c_left;
        c_off += L::kUnitBytes;
        if (c_off == (uint32_t)(S * L::kUnitBytes)) { c_off = 0; c_par ^= 1u; }
        return true;
    };
    // the W terms of one worker for my 64 outputs: groups of FIT consecutive codes, one
    // funnel shift brings a group's first field to bit 0, then every field lies below bit 23
    uint64_t acc2[32];                          // output j of (row A, row B) as an fp32 pair
    auto sum_unit = [&](const uint32_t (&cw)[2][R], const uint64_t a2) {
#pragma unroll
        for (int j0 = 0; j0 < 32; j0 += FIT) {
            const int bit = j0 * R, wi = bit >> 5, sh = bit & 31;
            uint32_t word[2];
#pragma unroll
            for (int row = 0; row < 2; ++row)
                word[row] = (sh == 0) ? cw[row][wi]
                          : (sh + FIT * R <= 32 || wi + 1 >= R) ? (cw[row][wi] >> sh)
                          : __funnelshift_r(cw[row][wi], cw[row][wi + 1], sh);
            const uint64_t w2 = ((uint64_t)word[1] << 32) | word[0];
#pragma unroll
            for (int i = 0; i < FIT && j0 + i < 32; ++i) {
                const uint64_t m2 = ((uint64_t)(mask << (i * R)) << 32) | (uint64_t)(mask << (i * R));
                // (c - s) 2^(iR) a, rows A and B in one instruction
                acc2[j0 + i] = fma2(sub2((w2 & m2) | magic2, T2[i]), a2, acc2[j0 + i]);
            }
        }
    };

    if (ok && n_units) ok = take_unit(cwa);

    for (uint32_t ti = 0; ok && ti < my_tiles; ++ti) {
        const uint32_t tile = blockIdx.x + ti * gridDim.x;
        // a_w = scale_w / s, pre-scaled by 2^-22 (exact; only scales below 2^-104 lose
        // bits, far under the absolute tolerance) against the 2^(iR) of the fields
        cp_async_wait<0>();
        __syncwarp();
#pragma unroll
        for (int k = 0; k < kDecAreg; ++k) {
            const uint32_t w = k * gsz + gl;
            if (k < (int)n_slots && w < W) {
                const float2 sc = *reinterpret_cast<const float2*>(raw + (grp + w) * 2);
                a_tab[grp + w] = make_float2(__fmul_rn(__fdiv_rn(sc.x, P.sf), 0x1p-22f),
                                             __fmul_rn(__fdiv_rn(sc.y, P.sf), 0x1p-22f));
            }
        }
        __syncwarp();
        if (ti + 1 < my_tiles) fetch_scales(tile + gridDim.x);

#pragma unroll
        for (int j = 0; j < 32; ++j) acc2[j] = 0ull;
        if (!first) {
            // running sums of the earlier messages (this path serves more than 64 messages
            // only): every lane reads its own two rows, 128 contiguous bytes each, and gives
            // the sums the powers of two of their fields
            const uint32_t sub_a = tile * kRingSubs + warp, sub_b = sub_a + kRingWarps;
            const float4* src_a = reinterpret_cast<const float4*>(
                dst.out + (uint64_t)sub_a * kDecTileElems + (uint32_t)lane * 32);
            const float4* src_b = reinterpret_cast<const float4*>(
                dst.out + (uint64_t)sub_b * kDecTileElems + (uint32_t)lane * 32);
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const float4 va = src_a[c];                     // sub_a < n_subs for every tile
                const float4 vb = sub_b < n_subs ? src_b[c] : make_float4(0.f, 0.f, 0.f, 0.f);
                const float ia[4] = {va.x, va.y, va.z, va.w}, ib[4] = {vb.x, vb.y, vb.z, vb.w};
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const float e = __uint_as_float((uint32_t)(127 - 22 + ((4 * c + q) % FIT) * R) << 23);
                    acc2[4 * c + q] = pack2(__fmul_rn(ia[q], e), __fmul_rn(ib[q], e));
                }
            }
        }

        const float2* const a_mine = a_tab + grp;
#pragma unroll 1
        for (uint32_t w = 0; w < W; ++w) {
            const uint64_t a2 = *reinterpret_cast<const uint64_t*>(a_mine + w);       // (a_A, a_B)
            sum_unit(cwa, a2);
            if (c_left) { if (!take_unit(cwa)) { ok = false; break; } }
        }
        if (!ok) break;

        // undo the powers of two, divide by W; one row at a time through the staging buffer:
        // row-per-lane -> coalesced 16-byte stores
#pragma unroll
        for (int row = 0; row < 2; ++row) {
            const uint32_t sub = tile * kRingSubs + warp + row * kRingWarps;
            if (sub >= n_subs) break;
            float acc[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                float lo, hi;
                unpack2(acc2[j], lo, hi);
                acc[j] = row ? hi : lo;
            }
            if (!last) {
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
#pragma unroll
            for (int c = 0; c < 8; ++c)
                *reinterpret_cast<float4*>(stage + lane * 128 + ((c ^ (lane & 7)) << 4)) =
                    make_float4(acc[4 * c], acc[4 * c + 1], acc[4 * c + 2], acc[4 * c + 3]);
            __syncwarp();
            const uint64_t o = (uint64_t)sub * kDecTileElems;
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int idx = k * 32 + lane, rw = idx >> 3, ch = idx & 7;
                const float4 v = *reinterpret_cast<const float4*>(stage + rw * 128 + ((ch ^ (rw & 7)) << 4));
                if (last) emit4(dst, o + idx * 4, v);
                else *reinterpret_cast<float4*>(dst.out + o + idx * 4) = v;
            }
            __syncwarp();
        }
    }
    cp_async_wait<0>();

    // A wait ran out (a copy that never completed): flag it, and let the copies that were
    // issued land before the CTA gives its shared memory back.
    if (!ok) { *s_abort = 1; if (lane == 0) atomicOr(status, kStatusTimeout); }
    __syncthreads();
    if (*s_abort) {
        if (threadIdx.x == 0)
            for (int i = 0; i < S; ++i)
                if (s_issued[i]) mbar_wait(bar_full + 8 * i, (s_issued[i] - 1u) & 1u);
        return;
    }

    // ragged end (fewer than 1024 outputs): one thread per output
    const uint64_t tail0 = (uint64_t)n_subs * kDecTileElems;
    const float magic = 8388608.f + P.sf;
    for (uint64_t i = tail0 + (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < P.d;
         i += (uint64_t)gridDim.x * blockDim.x) {
        const uint64_t b = i / P.bucket, bit = i * R, wi = bit >> 5;
        const uint32_t sh = (uint32_t)(bit & 31);
        float acc1 = first ? 0.f : dst.out[i];
        for (uint32_t w = 0; w < W; ++w) {
            const float a = __fdiv_rn(__ldg(tab.scales[w] + b), P.sf);
            const uint32_t lo = __ldg(tab.codes[w] + wi);
            const uint32_t hi1 = (sh + R > 32 && wi + 1 < n_words) ? __ldg(tab.codes[w] + wi + 1) : 0u;
            const uint32_t c = __funnelshift_r(lo, hi1, sh) & mask;
            acc1 = __fmaf_rn(__fsub_rn(__uint_as_float(0x4B000000u | c), magic), a, acc1);
        }
        if (!last) dst.out[i] = acc1;
        else emit1(dst, i, w_pow2 ? __fmul_rn(acc1, w_recip) : __fdiv_rn(acc1, w_total));
    }
}

}  // namespace ecq
