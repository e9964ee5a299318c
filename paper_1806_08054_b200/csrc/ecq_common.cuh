// Shared device helpers of the ECQ-SGD codec kernels (sm_100a).
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

namespace ecq {

// Programmatic dependent launch: a kernel launched with the stream-serialisation attribute may
// start while its predecessor in the stream still runs; it must not touch global memory
// before griddep_wait() (which returns once the predecessor has completed and its writes are
// visible).  griddep_launch() lets the successor's CTAs be scheduled as this grid's leave.
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }


constexpr uint32_t kStatusNonFinite = 1u;   // device status word bits
constexpr uint32_t kStatusTimeout = 2u;

// Constants of one context, passed by value to every kernel.
struct CodecParams {
    uint64_t d;          // entries
    uint32_t bucket;     // entries per bucket (multiple of 32)
    uint32_t s;          // non-zero levels of Eq. 9
    uint32_t r;          // ceil(log2(2s+1))
    int32_t mode;        // 0: Eq. 6 books g - g~; 1: books (g + alpha h) - g~
    int32_t norm;        // scale of Eq. 8: 0 l-infinity, 1 l2 (fixed summation order)
    float alpha, beta, sf;
    uint32_t key0[10];   // Philox round keys: the 64-bit seed advanced by the
    uint32_t key1[10];   // Weyl constants, one pair per round
};

// ---------------------------------------------------------------------------
// Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11).  One round maps
// (c0,c1,c2,c3) -> (hi(M1 c2)^c1^k0, lo(M1 c2), hi(M0 c0)^c3^k1, lo(M0 c0)).
// The round keys do not depend on the counter, so the host advances them once.
// ---------------------------------------------------------------------------
__device__ __forceinline__ void philox4x32_10(const CodecParams& P, uint32_t c0, uint32_t c1,
                                              uint32_t c2, uint32_t c3, uint32_t out[4]) {
#pragma unroll
    for (int i = 0; i < 10; ++i) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ P.key0[i];
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ P.key1[i];
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
        c0 = n0;
        c2 = n2;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Per-bucket constants derived from the l-infinity scale (Eq. 8).
struct BucketScale {
    float inv;      // s / scale
    float a;        // scale / s, the level step
    float scale;    // value written to scales[b]
    int kind;       // 0 regular, 1 all levels zero, 2 non-finite (accumulator kept)
};

// sbits: sign-cleared bit pattern of the bucket's max |v| (l-infinity) or of its sum of
// squares (l2).
__device__ __forceinline__ BucketScale bucket_scale(uint32_t sbits, float sf, int norm = 0) {
    BucketScale b;
    b.inv = 0.f; b.a = 0.f; b.scale = 0.f; b.kind = 0;
    if (sbits >= 0x7F800000u) { b.kind = 2; return b; }
    if (sbits == 0u) { b.kind = 1; return b; }
    const float scale = norm ? __fsqrt_rn(__uint_as_float(sbits)) : __uint_as_float(sbits);
    b.inv = __fdiv_rn(sf, scale);
    if (__float_as_uint(b.inv) >= 0x7F800000u) { b.kind = 1; b.inv = 0.f; return b; }
    b.a = __fdiv_rn(scale, sf);
    b.scale = scale;
    return b;
}

// Eq. 9 + Eq. 8 + Eq. 6 for one entry of a regular bucket.  Every operation is
// a single IEEE round-to-nearest fp32 operation (no contraction), except the
// floor, which is taken with a round-toward-zero add of 2^23 (exact for
// 0 <= x < 2^22).  Returns the non-negative code q + s and the new accumulator.
__device__ __forceinline__ uint32_t quantise_entry(float g, float h, float v, uint32_t R,
                                                   const BucketScale& b, const CodecParams& P,
                                                   float& h_new) {
    float x = __fmul_rn(fabsf(v), b.inv);
    x = fminf(x, P.sf);
    const float lf = __fsub_rn(__fadd_rz(x, 8388608.f), 8388608.f);   // floor(x)
    const float f = __fsub_rn(x, lf);                                  // exact
    const float u = __fmul_rn(__uint2float_rn(R >> 8), 0x1p-24f);      // exact, [0, 1)
    const float m = __fadd_rn(lf, (u < f) ? 1.f : 0.f);
    const float q = (__float_as_uint(v) >> 31) ? __fsub_rn(0.f, m) : m;   // -0 never arises
    const float gq = __fmul_rn(q, b.a);                                // dequantised entry
    const float e = __fsub_rn(P.mode ? v : g, gq);
    h_new = __fmaf_rn(P.beta, h, e);
    // (int)q + s without a conversion: q + 1.5*2^23 has q in its low mantissa bits
    return __float_as_uint(__fadd_rn(q, 12582912.f)) - (0x4B400000u - P.s);
}

// ---------------------------------------------------------------------------
// mbarrier / bulk-copy (TMA) wrappers.  Every wait is bounded.
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Non-blocking test of a phase (try_wait may suspend the thread for a while when the phase
// is not complete; this one returns at once).
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Bounded wait: false when the limit is reached (a copy that never completed).
constexpr uint32_t kWaitLimit = 1u << 22;
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t it = 0; it < kWaitLimit; ++it)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// The same with the context's limit (ecq_set_wait_limit; kWaitLimit unless a caller changed
// it).  Only the waits of the steady state take it: the waits that let copies in flight land
// after a wait has run out keep kWaitLimit, so that no copy lands in shared memory its CTA
// has already given back.
__device__ __forceinline__ bool mbar_wait_n(uint32_t bar, uint32_t parity, uint32_t limit) {
    for (uint32_t it = 0; it < limit; ++it)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}

__device__ __forceinline__ void fence_proxy_async_smem() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void fence_mbar_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

// 2-D tiled TMA load into this CTA's own shared memory.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const void* tmap, int x, int y,
                                            uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(tmap), "r"(x), "r"(y), "r"(bar)
        : "memory");
}

// 2-D tiled TMA store from shared memory.
__device__ __forceinline__ void tma_store_2d(const void* tmap, int x, int y, uint32_t src) {
    asm volatile(
        "cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];"
        ::"l"(tmap), "r"(x), "r"(y), "r"(src)
        : "memory");
}

// Linear bulk store: 16-byte aligned on both sides, size a multiple of 16.
__device__ __forceinline__ void bulk_store_1d(void* gdst, uint32_t src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(gdst), "r"(src), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ void bulk_commit() {
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void bulk_wait_read0() {
    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}
__device__ __forceinline__ void bulk_wait_all() {
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

// ---------------------------------------------------------------------------
// Packed fp32x2 arithmetic (sm_100): two independent IEEE round-to-nearest
// operations per instruction on a 64-bit register pair.
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t add2_rz(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("add.rz.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

__device__ __forceinline__ void named_bar_sync(uint32_t id, uint32_t nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

}  // namespace ecq
