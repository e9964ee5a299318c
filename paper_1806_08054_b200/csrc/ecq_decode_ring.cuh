// Receiver-side kernel for long vectors: unpack -> dequantise -> W-way mean (Eq. 4;
// Algorithm 1, phase 2, global-gradient step), with the code words brought in by bulk copies
// that a whole CTA shares.
//
// One CTA per SM: 15 consumer warps and one producer warp.  A CTA tile is 30 sub-tiles of
// 1024 outputs.  Consumer warp k owns sub-tiles k and k + 15; a lane owns one run of 32
// consecutive outputs ("row") in each, whose codes are R whole words.
//   * a ring stage holds the code words of (tile, kGroup consecutive workers): one bulk copy
//     of R * 3840 contiguous bytes per worker, all counted on the stage's "full" mbarrier.
//     Lane 0 of the producer warp issues them in order, each stage as soon as the 15 consumer
//     warps have handed it back on its "empty" mbarrier.  A consumer warp waits once per
//     stage, reads the stage's words of its two rows into registers (all loads first, so the
//     shared-memory latency is met once), sums, and arrives once;
//   * the two rows of a lane travel as the two halves of packed fp32x2 registers: one packed
//     multiply-add with the pair of level steps (a_A, a_B) of the rows' buckets adds the
//     terms; per worker the chain acc <- fma(q_w, a_w, acc) is the one Eq. 4 writes out, in
//     ascending w;
//   * turning a bit field into the float q = c - s is what the kernel is bound by: issue
//     slots (a packed fp32x2 instruction takes two, so packing saves none) and the 16-lane
//     logic pipe.  For code widths that divide 16 the fields are merged two at a time into
//     an fp16 pair: (word & field-in-both-halves) | 0x64006400 is (1024 + c 2^p) twice, and
//     one mixed-precision add per code (f16 + f32 -> f32) takes 1024 + s 2^p off and widens,
//     exactly: half a logic instruction and one add per code.  Other widths merge the field
//     into the mantissa of 2^23, (word_A & field, word_B & field) | 2^23 bits, and one packed
//     subtract leaves ((c - s) 2^p) for both rows: one logic instruction and half a packed
//     subtract (one slot) per code;
//   * level steps a_w = scale_w / s of the next tile are fetched with 4-byte asynchronous
//     copies while this tile is summed;
//   * a lane stores its rows with 32-byte stores (whole sectors), so the means need no
//     transposition; `out` and `params` must be 32-byte aligned for this kernel.
#pragma once

#include "ecq_decode.cuh"

namespace ecq {

// 15 consumer warps and the producer warp make 512 threads, which leaves a thread 128 registers
constexpr int kRingWarps = 15;
constexpr int kRingThreads = (kRingWarps + 1) * 32;
constexpr int kRingSubs = 2 * kRingWarps;                       // sub-tiles per CTA tile
constexpr int kRingTileElems = kRingSubs * kDecTileElems;       // 30720 outputs
// What the automatic choice asks for: shorter vectors leave the CTAs with too uneven a share
// of these large tiles (a CTA's time goes by whole tiles), and at r = 9 the receiver is bound
// by HBM, not by instruction issue, where the warp-tiled kernel's deeper private rings do
// better.  With few messages of wide codes the vector has to be long:
constexpr int kRingMinTilesPerCta = 12;
// The more messages and the narrower the codes, the smaller the per-tile work (level steps,
// stores) is beside the per-code work, and the sooner this kernel is ahead.  Measured on
// vectors of 3.3 / 5.6 / 8.8 tiles per CTA, time of this kernel over the warp-tiled one:
// 16 messages of 2 bits 0.84 / 0.77 / 0.74, of 4 bits 0.94 / 0.88 / 0.86, of 5 bits 1.04 / 0.97 /
// 0.97; 12 messages the same within 0.03; 8 messages of 2 bits 1.00 / 0.93 / 0.89, of 4 bits
// 1.14 / 1.07 / 1.00, of 5 bits 1.19 / 1.10 / 1.02; 32 messages of 4 bits 0.81 / 0.77 and 0.96
// at 2.1 tiles; 4 messages always above 1.
__host__ __device__ constexpr int ring_min_tiles_per_cta(int r, uint32_t W) {
    return (r <= 4 && W >= 12) ? 3 : ((r <= 2 && W >= 8) || W >= 12) ? 5 : kRingMinTilesPerCta;
}
constexpr int kRingMaxAutoBits = 8;

template <int R> struct DecodeRing {
    // fp16 pair merge where two fields sit 16 bits apart in a word
    static constexpr bool kHalf = (R == 2 || R == 4 || R == 8);
    static constexpr int kHalfFields = 16 / R;                   // fields of a 16-bit half
    static constexpr int kViewFields = 10 / R;                   // of which lie below bit 10 at a time
    // fp32 merge: whole fields below bit 23 of a word; chosen so that the fewest groups need a shift
    static constexpr int kFit = R == 2 ? 8 : R == 3 ? 7 : R == 4 ? 4 : 23 / R;
    // bit position of code j's field in the register it is merged from
    __host__ __device__ static constexpr int field_shift(int j) {
        return kHalf ? (((j % (32 / R)) % kHalfFields) % kViewFields) * R : (j % kFit) * R;
    }
    static constexpr int kGroup = R <= 4 ? 2 : 1;                // workers per ring stage
    static constexpr int kUnitBytes = R * 128 * kRingSubs;       // one worker's words of a tile
    static constexpr int kStageBytes = kGroup * kUnitBytes;
    // full mbarriers at 0, empty ones at 128, abort flag at 256, stages filled at 260, zero at 264
    static constexpr int kBarBytes = 512;
    static constexpr int kRingOff = kBarBytes;
    static constexpr int kMaxSmem = 232448 - 1024;               // what one CTA per SM can have
    static constexpr int kMaxStages = 12;                        // 16 barriers fit each barrier area
    // at two bits the kernel is shortest of registers: ring depth and table strides stay
    // compile-time constants there (worst-case tables of 4 KB a warp; measured 2 % faster)
    static constexpr bool kFixedLayout = R == 2;
    static constexpr int kFixedStages = (kMaxSmem - kRingOff - kRingWarps * kDecAreg * 32 * 16) / kStageBytes > kMaxStages
        ? kMaxStages : (kMaxSmem - kRingOff - kRingWarps * kDecAreg * 32 * 16) / kStageBytes;
};

// Shared memory of one launch: the ring takes what the level-step tables leave.  A consumer
// warp keeps, per group of lanes that share a bucket, `wstride` entries of (a_A, a_B) and as
// many raw scale pairs: 16 bytes per entry, (32 / gsz) groups.  (With every table at its
// largest, 4 KB a warp, the ring would lose 46 KB; its depth is worth 3-4 % a stage.)
struct RingLayout {
    uint32_t wstride;        // table entries per lane group: the workers of the launch, even
    uint32_t warp_bytes;     // tables of one consumer warp
    uint32_t stages;         // ring depth
    uint32_t smem;           // dynamic shared memory of the launch
};
template <int R>
inline RingLayout ring_layout(uint32_t W, uint32_t bucket) {
    using L = DecodeRing<R>;
    const uint32_t gsz = bucket >= 1024u ? 32u : (bucket >> 5);
    RingLayout y;
    y.wstride = (W + 1u) & ~1u;
    if (L::kFixedLayout) y.wstride = (uint32_t)kDecAreg * gsz;       // 4 KB a warp whatever the launch
    y.warp_bytes = (32u / gsz) * y.wstride * 16u;
    const uint32_t room = (uint32_t)L::kMaxSmem - (uint32_t)L::kRingOff - (uint32_t)kRingWarps * y.warp_bytes;
    y.stages = room / (uint32_t)L::kStageBytes;
    if (y.stages > (uint32_t)L::kMaxStages) y.stages = (uint32_t)L::kMaxStages;
    y.smem = (uint32_t)L::kRingOff + y.stages * (uint32_t)L::kStageBytes + (uint32_t)kRingWarps * y.warp_bytes;
    return y;
}

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

__device__ __forceinline__ void stg256(float* p, const float (&v)[8]) {
    asm volatile("st.global.v8.f32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"l"(p), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7])
                 : "memory");
}
__device__ __forceinline__ void ldg256(const float* p, float (&v)[8]) {
    asm volatile("ld.global.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7])
                 : "l"(p)
                 : "memory");
}
// eight consecutive means: to `out` (may be null) and, for the fused model update, into `params`
__device__ __forceinline__ void emit8(const DecodeOut& o, uint64_t i, const float (&v)[8]) {
    if (o.params) {
        float p[8];
        ldg256(o.params + i, p);
#pragma unroll
        for (int k = 0; k < 8; ++k) p[k] = __fmaf_rn(o.neg_eta, v[k], p[k]);
        stg256(o.params + i, p);
    }
    if (o.out) stg256(o.out + i, v);
}
__device__ __forceinline__ void lds32(uint32_t a, uint32_t& x) {
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(x) : "r"(a) : "memory");
}
__device__ __forceinline__ void lds64(uint32_t a, uint32_t& x, uint32_t& y) {
    asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(x), "=r"(y) : "r"(a) : "memory");
}
__device__ __forceinline__ void lds128(uint32_t a, uint32_t& x, uint32_t& y, uint32_t& z, uint32_t& w) {
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(x), "=r"(y), "=r"(z), "=r"(w) : "r"(a) : "memory");
}

// Both halves of `m` read as fp16, each plus the fp32 `c`, as fp32: one instruction per half,
// one rounding (none here: the sums are small integers times a power of two).
__device__ __forceinline__ void add_f32_f16x2(uint32_t m, float c, float& lo, float& hi) {
    asm("{\n\t.reg .b16 h0, h1;\n\t"
        "mov.b32 {h0, h1}, %2;\n\t"
        "add.rn.f32.f16 %0, h0, %3;\n\t"
        "add.rn.f32.f16 %1, h1, %3;\n\t}"
        : "=f"(lo), "=f"(hi) : "r"(m), "f"(c));
}

// The 64 terms of one worker for the two rows of a lane:
// acc2[j] <- fma((c_j - s) 2^p_j, (a_A, a_B), acc2[j]), rows A and B in the two halves.
// subh[i] = -(1024 + s 2^(iR)) (fp16 pair merge); T2[i] = (t, t), t = 2^23 + s 2^(iR)
// (fp32 merge).  exp_bits: 0x64006400 or 0x4B000000, in a register because a logic
// instruction takes one immediate, and the field mask is it.
template <int R, int NH, int NT>
__device__ __forceinline__ void ring_pair_terms(const uint32_t (&cwa)[R], const uint32_t (&cwb)[R],
                                                const uint64_t a2, uint64_t (&acc2)[32],
                                                const uint32_t exp_bits, const float (&subh)[NH],
                                                const uint64_t (&T2)[NT]) {
    using L = DecodeRing<R>;
    constexpr uint32_t mask = (1u << R) - 1u;
    if constexpr (L::kHalf) {
        constexpr int CW = 32 / R, NF = L::kHalfFields, FV = L::kViewFields;
#pragma unroll
        for (int wi = 0; wi < R; ++wi) {
#pragma unroll
            for (int v0 = 0; v0 < NF; v0 += FV) {
                // fields v0 .. v0 + FV - 1 of both halves, brought below bit 10 of each half
                const uint32_t xa = v0 == 0 ? cwa[wi] : (cwa[wi] >> (v0 * R));
                const uint32_t xb = v0 == 0 ? cwb[wi] : (cwb[wi] >> (v0 * R));
#pragma unroll
                for (int i = 0; i < FV && v0 + i < NF; ++i) {
                    const uint32_t ma = (xa & ((mask << (i * R)) * 0x00010001u)) | exp_bits;
                    const uint32_t mb = (xb & ((mask << (i * R)) * 0x00010001u)) | exp_bits;
                    float la, ha, lb, hb;
                    add_f32_f16x2(ma, subh[i], la, ha);
                    add_f32_f16x2(mb, subh[i], lb, hb);
                    const int jl = wi * CW + v0 + i, jh = jl + NF;
                    acc2[jl] = fma2(pack2(la, lb), a2, acc2[jl]);
                    acc2[jh] = fma2(pack2(ha, hb), a2, acc2[jh]);
                }
            }
            // the sums of this word are due here: keeps the compiler from widening every code
            // of a worker first and holding 64 of them in registers (no instruction is emitted)
#pragma unroll
            for (int j = wi * CW; j < wi * CW + CW; ++j) asm volatile("" : "+l"(acc2[j]));
        }
    } else {
        constexpr int FIT = L::kFit;
        const uint64_t magic2 = ((uint64_t)exp_bits << 32) | exp_bits;
        // groups of FIT consecutive codes: one funnel shift brings a group's first field to
        // bit 0, then every field lies below bit 23
#pragma unroll
        for (int j0 = 0; j0 < 32; j0 += FIT) {
            const int bit = j0 * R, wi = bit >> 5, sh = bit & 31;
            const uint32_t wa = (sh == 0) ? cwa[wi]
                              : (sh + FIT * R <= 32 || wi + 1 >= R) ? (cwa[wi] >> sh)
                              : __funnelshift_r(cwa[wi], cwa[wi + 1 < R ? wi + 1 : wi], sh);
            const uint32_t wb = (sh == 0) ? cwb[wi]
                              : (sh + FIT * R <= 32 || wi + 1 >= R) ? (cwb[wi] >> sh)
                              : __funnelshift_r(cwb[wi], cwb[wi + 1 < R ? wi + 1 : wi], sh);
            const uint64_t w2 = ((uint64_t)wb << 32) | wa;
#pragma unroll
            for (int i = 0; i < FIT && j0 + i < 32; ++i) {
                const uint64_t m2 = ((uint64_t)(mask << (i * R)) << 32) | (uint64_t)(mask << (i * R));
                // (c - s) 2^(iR) a, rows A and B in one instruction
                acc2[j0 + i] = fma2(sub2((w2 & m2) | magic2, T2[i]), a2, acc2[j0 + i]);
            }
#pragma unroll
            for (int i = 0; i < FIT && j0 + i < 32; ++i) asm volatile("" : "+l"(acc2[j0 + i]));
        }
    }
}

// What one consumer warp does: its two rows of every tile of the CTA.
template <int R, bool CARRY>
__device__ __forceinline__ void decode_ring_consumer(
        const CodecParams& P, const uint32_t W, const MessageTable& tab, const DecodeOut& dst,
        const uint32_t n_subs, const float w_recip, const int w_pow2, const uint32_t exp_bits,
        const bool first, const bool last, const float w_total, const uint32_t my_tiles,
        const uint32_t wait_limit, const RingLayout lay, const int warp, const int lane, uint8_t* dsm,
        uint32_t* status) {
    using L = DecodeRing<R>;
    const uint32_t S = L::kFixedLayout ? (uint32_t)L::kFixedStages : lay.stages;
    constexpr int FIT = L::kFit;
    constexpr int G = L::kGroup;
    const uint32_t sm0 = smem_u32(dsm);
    const uint32_t bar_full = sm0, bar_empty = sm0 + 128;
    volatile uint32_t* const s_abort = reinterpret_cast<volatile uint32_t*>(dsm + 256);
    const uint32_t warp_bytes = L::kFixedLayout ? (uint32_t)kDecAreg * 32 * 16 : lay.warp_bytes;
    uint8_t* const my_tabs = dsm + L::kRingOff + S * L::kStageBytes + warp * warp_bytes;
    float2* const a_tab = reinterpret_cast<float2*>(my_tabs);
    float* const raw = reinterpret_cast<float*>(my_tabs + warp_bytes / 2);

    // lanes that share a bucket: gsz consecutive lanes (all 32 from 1024 entries up); a_tab
    // holds, per group of lanes, (a_w of row A, a_w of row B) for w < W (W <= kDecAreg * gsz),
    // lay.wstride entries a group
    const uint32_t gsz = P.bucket >= 1024u ? 32u : (P.bucket >> 5);
    const uint32_t gl = lane & (gsz - 1);
    const uint32_t bucket_shift = 31 - __clz(P.bucket);           // bucket is a power of two
    // Level steps enter the tables as a_w 2^-22 (against the 2^p of the fields) and, when the
    // whole mean is taken here over a power-of-two number of messages, divided by it as well:
    // powers of two, so the chain's roundings are those of Eq. 4 and the stored mean needs one
    // multiply.  With s a power of two the division scale / s is a multiplication too.
    const bool pre_w = !CARRY && w_pow2;
    const bool s_pow2 = (P.s & (P.s - 1u)) == 0u;
    const float k_pre = pre_w ? __fmul_rn(0x1p-22f, w_recip) : 0x1p-22f;
    const float a_mul = s_pow2 ? __fdiv_rn(k_pre, P.sf) : k_pre;
    const uint32_t grp = L::kFixedLayout ? (lane & ~(gsz - 1)) * kDecAreg : ((uint32_t)lane / gsz) * lay.wstride;   // my group's first entry
    const uint32_t raw_u32 = smem_u32(raw);

    // what turns a merged field into (c - s) 2^p, per field position (see ring_pair_terms)
    uint64_t T2[FIT];
#pragma unroll
    for (int i = 0; i < FIT; ++i) {
        const float t = __fmaf_rn(P.sf, (float)(1u << (i * R)), 8388608.f);
        T2[i] = pack2(t, t);
    }
    float subh[L::kViewFields > 0 ? L::kViewFields : 1];
#pragma unroll
    for (int i = 0; i < L::kViewFields; ++i) subh[i] = -__fmaf_rn(P.sf, (float)(1u << (i * R)), 1024.f);

    // ---- raw scales of a tile's buckets: worker k*gsz + gl of my group, rows A and B ----
    auto fetch_scales = [&](uint32_t tile) {
#pragma unroll
        for (int row = 0; row < 2; ++row) {
            const uint32_t sub = tile * kRingSubs + warp + row * kRingWarps;
            if (sub < n_subs) {
                const uint64_t b = ((uint64_t)sub * kDecTileElems + (uint32_t)lane * 32) >> bucket_shift;
#pragma unroll 1
                for (uint32_t w = gl; w < W; w += gsz)
                    cp_async4(raw_u32 + ((grp + w) * 2 + row) * 4, tab.scales[w] + b);
            }
        }
        cp_async_commit();
    };
    if (my_tiles) fetch_scales(blockIdx.x);

    // ring position of the next stage: byte offset, its barriers' offset, phase
    uint32_t c_off = 0, c_bar = 0, c_par = 0;
    const uint32_t my_off = sm0 + L::kRingOff + warp * (R * 128) + lane * (R * 4);
    uint32_t cw[G][2][R];
    uint32_t dep = 0;
    // Waits for the next stage and copies the words of my two rows, for all its workers, to
    // registers: all loads first, so their latency is met once per stage.  (Loading at the top
    // of a stage keeps the words out of the loop-carried state: carrying them over from the
    // previous turn, or fetching a stage ahead into a second register set, costs more in
    // register moves and control flow than the latency it hides.)
    auto take_stage = [&]() -> bool {
        // With two workers a stage the first poll usually finds the stage complete, and going
        // straight on without the warp vote pays (alexnet-shaped launch 6 % faster, r = 4 1 %);
        // with one worker a stage (twice as many stages) the same form measured 2 % slower.
        if constexpr (G == 2) {
            if (!mbar_try_wait(bar_full + c_bar, c_par) &&
                !__all_sync(0xFFFFFFFFu, mbar_wait_n(bar_full + c_bar, c_par, wait_limit))) return false;
        } else {
            if (!__all_sync(0xFFFFFFFFu, mbar_wait_n(bar_full + c_bar, c_par, wait_limit))) return false;
        }
        constexpr int kStep = (R % 4 == 0) ? 4 : (R % 2 == 0) ? 2 : 1;    // words per load
#pragma unroll
        for (int k = 0; k < G; ++k) {
#pragma unroll
            for (int row = 0; row < 2; ++row) {
                const uint32_t src = my_off + c_off + k * L::kUnitBytes + row * (kRingWarps * R * 128);
                if constexpr (R % 4 == 0) {
#pragma unroll
                    for (int q = 0; q < R / 4; ++q)
                        lds128(src + 16 * q, cw[k][row][4 * q], cw[k][row][4 * q + 1], cw[k][row][4 * q + 2], cw[k][row][4 * q + 3]);
                } else if constexpr (R % 2 == 0) {
#pragma unroll
                    for (int q = 0; q < R / 2; ++q) lds64(src + 8 * q, cw[k][row][2 * q], cw[k][row][2 * q + 1]);
                } else {
#pragma unroll
                    for (int q = 0; q < R; ++q) lds32(src + 4 * q, cw[k][row][q]);
                }
#pragma unroll
                for (int q = 0; q < R; q += kStep) dep ^= cw[k][row][q];
            }
        }
        return true;
    };
    // The stage is handed back only after its words have been used: the loads have then
    // certainly completed, which an arrive issued right behind them does not wait for.  `zero`
    // is 0, but only at run time: (dep & zero) makes the arrive depend on one word of every
    // shared load of the stage (a shared load is one instruction for the whole warp, so lane
    // 0's dependence covers every lane).
    const uint32_t zero = *reinterpret_cast<volatile uint32_t*>(dsm + 264);
    auto release_stage = [&]() {
        if (lane == 0 && (dep & zero) == 0u) mbar_arrive(bar_empty + c_bar);
        c_off += L::kStageBytes;
        c_bar += 8;
        if (c_bar == 8u * S) { c_off = 0; c_bar = 0; c_par ^= 1u; }
    };

    bool ok = true;
    const float2* const a_mine = a_tab + grp;

    for (uint32_t ti = 0; ok && ti < my_tiles; ++ti) {
        const uint32_t tile = blockIdx.x + ti * gridDim.x;
        // a_w = scale_w / s, pre-scaled by 2^-22 (exact; only scales below 2^-104 lose
        // bits, far under the absolute tolerance) against the 2^(iR) of the fields
        cp_async_wait<0>();
        __syncwarp();
#pragma unroll 1
        for (uint32_t w = gl; w < W; w += gsz) {
            const float2 sc = *reinterpret_cast<const float2*>(raw + (grp + w) * 2);
            a_tab[grp + w] = s_pow2 ? make_float2(__fmul_rn(sc.x, a_mul), __fmul_rn(sc.y, a_mul))
                                    : make_float2(__fmul_rn(__fdiv_rn(sc.x, P.sf), a_mul),
                                                  __fmul_rn(__fdiv_rn(sc.y, P.sf), a_mul));
        }
        __syncwarp();
        if (ti + 1 < my_tiles) fetch_scales(tile + gridDim.x);

        const uint32_t sub_a = tile * kRingSubs + warp, sub_b = sub_a + kRingWarps;
        uint64_t acc2[32];                      // output j of (row A, row B) as an fp32 pair
#pragma unroll
        for (int j = 0; j < 32; ++j) acc2[j] = 0ull;
        if (!first) {
            // running sums of the earlier messages (this path serves more than 64 messages
            // only): every lane reads its own two rows, 128 contiguous bytes each, and gives
            // the sums the powers of two of their fields
            const float4* src_a = reinterpret_cast<const float4*>(
                dst.out + (uint64_t)sub_a * kDecTileElems + (uint32_t)lane * 32);
            const float4* src_b = reinterpret_cast<const float4*>(
                dst.out + (uint64_t)sub_b * kDecTileElems + (uint32_t)lane * 32);
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const float4 va = sub_a < n_subs ? src_a[c] : make_float4(0.f, 0.f, 0.f, 0.f);
                const float4 vb = sub_b < n_subs ? src_b[c] : make_float4(0.f, 0.f, 0.f, 0.f);
                const float ia[4] = {va.x, va.y, va.z, va.w}, ib[4] = {vb.x, vb.y, vb.z, vb.w};
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const float e = __uint_as_float((uint32_t)(127 - 22 + L::field_shift(4 * c + q)) << 23);
                    acc2[4 * c + q] = pack2(__fmul_rn(ia[q], e), __fmul_rn(ib[q], e));
                }
            }
        }

        // the workers in ascending order, a stage (G of them) per turn
#pragma unroll 2
        for (uint32_t w0 = 0; w0 < W; w0 += G) {
            if (!take_stage()) { ok = false; break; }
#pragma unroll
            for (int k = 0; k < G; ++k) {
                if (k > 0 && w0 + k >= W) break;                     // a last, partly filled stage
                const uint64_t a2 = *reinterpret_cast<const uint64_t*>(a_mine + w0 + k);   // (a_A, a_B)
                ring_pair_terms<R>(cw[k][0], cw[k][1], a2, acc2, exp_bits, subh, T2);
            }
            release_stage();
        }
        if (!ok) break;

        // undo the powers of two, divide by W, store: 32 bytes (one sector) per store
#pragma unroll
        for (int row = 0; row < 2; ++row) {
            const uint32_t sub = row ? sub_b : sub_a;
            if (sub >= n_subs) continue;
            const uint64_t o = (uint64_t)sub * kDecTileElems + (uint32_t)lane * 32;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                float v[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const int j = 8 * c + k;
                    float lo, hi;
                    unpack2(acc2[j], lo, hi);
                    const float x = __fmul_rn(row ? hi : lo, __uint_as_float((uint32_t)(127 + 22 - L::field_shift(j)) << 23));
                    v[k] = (!last || pre_w) ? x : w_pow2 ? __fmul_rn(x, w_recip) : __fdiv_rn(x, w_total);
                }
                if (last) emit8(dst, o + 8 * c, v);
                else stg256(dst.out + o + 8 * c, v);
            }
        }
    }
    cp_async_wait<0>();
    if (!ok) { *s_abort = 1; if (lane == 0) atomicOr(status, kStatusTimeout); }
}

template <int R, bool CARRY>
__global__ void __launch_bounds__(kRingThreads, 1)
decode_ring_kernel(const CodecParams P, const uint32_t W, const __grid_constant__ MessageTable tab,
                   const DecodeOut dst, const uint32_t n_subs, const uint64_t n_words,
                   const float w_recip, const int w_pow2, const uint32_t exp_bits,
                   const uint32_t wait_limit, const RingLayout lay, const DecodeSlice sl, uint32_t* status) {
    using L = DecodeRing<R>;
    const bool first = CARRY ? sl.first != 0 : true, last = CARRY ? sl.last != 0 : true;
    const float w_total = CARRY ? sl.w_total : (float)W;
    const uint32_t S = L::kFixedLayout ? (uint32_t)L::kFixedStages : lay.stages;
    extern __shared__ __align__(128) uint8_t dsm[];
    const uint32_t sm0 = smem_u32(dsm);
    const uint32_t bar_full = sm0, bar_empty = sm0 + 128;
    volatile uint32_t* const s_abort = reinterpret_cast<volatile uint32_t*>(dsm + 256);
    volatile uint32_t* const s_issued = reinterpret_cast<volatile uint32_t*>(dsm + 260);   // stages the producer filled
    const int lane = threadIdx.x & 31;
    // broadcast from lane 0 so that the compiler knows the value is warp-uniform
    const int warp = __shfl_sync(0xFFFFFFFFu, (int)(threadIdx.x >> 5), 0);

    const uint32_t n_tiles = (n_subs + kRingSubs - 1) / kRingSubs;
    const uint32_t my_tiles =
        blockIdx.x < n_tiles ? (n_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;

    if (threadIdx.x == 0) {
        for (uint32_t i = 0; i < S; ++i) {
            mbar_init(bar_full + 8 * i, 1);
            mbar_init(bar_empty + 8 * i, kRingWarps);
        }
        *s_abort = 0;
        *s_issued = 0;
        *reinterpret_cast<volatile uint32_t*>(dsm + 264) = 0;
        fence_mbar_init();
    }
    griddep_launch();
    __syncthreads();
    griddep_wait();

    if (warp == kRingWarps) {
        // ---- producer: fill n = my n / n_groups-th tile, workers G (n % n_groups) and up, in
        // order, into stage n % S ----
        if (lane == 0) {
            bool ok = true;
            uint32_t tile = blockIdx.x, w = 0, slot = 0, par = 0, u = 0;
            constexpr int G = L::kGroup;
            const uint32_t n_fills = my_tiles * ((W + G - 1) / G);
            for (; u < n_fills; ++u) {
                // stages are free the first time round; later the consumers hand them back
                if (u >= S && !mbar_wait_n(bar_empty + 8 * slot, par ^ 1u, wait_limit)) { ok = false; break; }
                if (*s_abort) break;                        // a consumer's wait ran out
                const uint32_t subs = min((uint32_t)kRingSubs, n_subs - tile * kRingSubs);
                const uint32_t bytes = subs * (R * 128);
                const uint32_t n = min((uint32_t)G, W - w);
                const uint32_t bar = bar_full + 8 * slot;
                mbar_arrive_expect_tx(bar, n * bytes);
                for (uint32_t k = 0; k < n; ++k)
                    bulk_load_1d(sm0 + L::kRingOff + slot * L::kStageBytes + k * L::kUnitBytes,
                                 tab.codes[w + k] + (uint64_t)tile * (R * 32 * kRingSubs), bytes, bar);
                w += n;
                if (w == W) { w = 0; tile += gridDim.x; }
                if (++slot == S) { slot = 0; par ^= 1u; }
            }
            *s_issued = u;
            if (!ok) { *s_abort = 1; atomicOr(status, kStatusTimeout); }    // a stage never came back
        }
        __syncwarp();
    } else {
        decode_ring_consumer<R, CARRY>(P, W, tab, dst, n_subs, w_recip, w_pow2, exp_bits, first, last,
                                       w_total, my_tiles, wait_limit, lay, warp, lane, dsm, status);
    }
    __syncthreads();
    if (*s_abort) {
        // a wait ran out: let the copies in flight land before the CTA gives its shared memory
        // back (fill v went into stage v % S; the last S fills may still be on their way).
        // This wait keeps the full limit whatever the context's.
        if (threadIdx.x == 0) {
            const uint32_t u = *s_issued;
            for (uint32_t v = (u > S ? u - S : 0); v < u; ++v)
                mbar_wait(bar_full + 8 * (v % S), (v / S) & 1u);
        }
        return;
    }

    decode_ragged_end<R>(P, W, tab, dst, (uint64_t)n_subs * kDecTileElems, n_words, first, last, w_recip,
                         w_pow2, w_total);
}

}  // namespace ecq
