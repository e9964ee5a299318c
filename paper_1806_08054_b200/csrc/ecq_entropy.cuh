// Entropy-coded message (paragraph after Eq. 9: the r-bit codes may be compressed further by
// an entropy code, Huffman coding being the one named; the linear-model experiments count
// bits that way).
//
// Format: canonical prefix code over the 2s+1 level indices with words of at most 12 bits;
// a word's bits enter the stream in tree order, first bit in the lowest free bit of the
// current 32-bit word; the entries are cut into chunks of 1024, every chunk starts on a
// word boundary, offsets[c] is its first word and offsets[n_chunks] the stream length;
// quarters[3c + j] is the bit, counted from the chunk's first word, at which entry
// 256 (j + 1) of chunk c starts (the chunk's end if it has fewer entries), so that four
// threads can decode one chunk.
//
// Sender: three launches -- words needed per chunk, their running sum, the stream itself
// (a single pass cannot place a chunk before all earlier chunk sizes are known, and no
// kernel here waits on another).  Receiver: one launch, one thread per quarter chunk.
#pragma once

#include "ecq_common.cuh"

namespace ecq {

constexpr uint32_t kHuffMaxLen = 12;
constexpr uint32_t kHuffChunk = 1024;
constexpr uint32_t kHuffQuarter = 256;
constexpr uint32_t kHuffMaxSymbols = 1u << kHuffMaxLen;
constexpr uint32_t kHuffChunkWords = kHuffChunk * kHuffMaxLen / 32;     // longest chunk
constexpr int kHuffWarps = 8;
constexpr uint32_t kStatusCapacity = 4u;    // device status word bits (after 1 and 2)
constexpr uint32_t kStatusSymbol = 8u;

// Device tables of one code, built on the host:
//   enc[c]  = length << 16 | the word with its first bit in bit 0      (c < 4096)
//   dec[p]  for every 12-bit pattern p: the words that lie wholly inside it, decoded
//           greedily from bit 0 (at most kHuffDecMaxSyms, and as many as fit 16 bits of
//           r-bit codes):
//             bits  0..15  their symbols, r bits each, first one lowest
//             bits 16..19  how many (0: p starts with no word)
//             bits 20..23  bits used by all of them
//             bits 24..27  bits used by the first alone
//   group_syms  k: the sender looks up k codes at a time (k*r <= 12 table index bits,
//           k * longest word <= 24 bits)
struct HuffTables {
    uint32_t enc[kHuffMaxSymbols];
    uint32_t dec[1u << kHuffMaxLen];
    uint32_t group_syms;
    uint32_t reserved[3];
};
constexpr uint32_t kHuffDecMaxSyms = 4;

// Group table entry (shared memory, built per CTA): bits 0..23 the k words back to back
// (first symbol lowest), bits 24..28 their total length, bit 31 set when one of the
// symbols has no word.
constexpr uint32_t kGroupInvalid = 1u << 31;

__device__ __forceinline__ uint32_t enc_or_zero(const HuffTables* t, uint32_t sym, uint32_t n_sym) {
    return sym < n_sym ? __ldg(t->enc + sym) : 0u;
}

__device__ __forceinline__ void build_group_table(uint32_t* s_group, const HuffTables* t,
                                                  uint32_t n_sym, uint32_t r, uint32_t k) {
    const uint32_t mask = (1u << r) - 1u;
    for (uint32_t v = threadIdx.x; v < (1u << (k * r)); v += blockDim.x) {
        uint32_t bits = 0, total = 0, bad = 0;
        for (uint32_t i = 0; i < k; ++i) {
            const uint32_t e = enc_or_zero(t, (v >> (i * r)) & mask, n_sym);
            bits |= (e & 0xFFFFu) << total;
            total += e >> 16;
            bad |= (e >> 16) == 0;
        }
        s_group[v] = bits | (total << 24) | (bad ? kGroupInvalid : 0u);
    }
    __syncthreads();
}

// The codes of one row (32 entries = r whole words, nv of them valid), as groups of k:
// fn(entry) for every whole group's table entry, then for each left-over code of a
// ragged row (the end of the vector only).
template <typename F>
__device__ __forceinline__ void for_each_group(const uint32_t* __restrict__ codes, uint64_t row,
                                               uint32_t r, uint32_t k, uint32_t nv,
                                               const uint32_t* s_group, const HuffTables* t,
                                               uint32_t n_sym, F fn) {
    const uint32_t gbits = k * r;
    const uint32_t* w = codes + row * r;
    const uint32_t nw = (nv * r + 31) >> 5;
    const uint32_t gmask = (1u << gbits) - 1u, mask = (1u << r) - 1u;
    const uint32_t n_groups = nv / k;
    uint64_t acc = 0;
    uint32_t have = 0, kw = 0;
    for (uint32_t g = 0; g < n_groups; ++g) {
        if (have < gbits) { acc |= (uint64_t)(kw < nw ? __ldg(w + kw) : 0u) << have; ++kw; have += 32; }
        fn(s_group[(uint32_t)acc & gmask]);
        acc >>= gbits; have -= gbits;
    }
    for (uint32_t j = n_groups * k; j < nv; ++j) {
        if (have < r) { acc |= (uint64_t)(kw < nw ? __ldg(w + kw) : 0u) << have; ++kw; have += 32; }
        const uint32_t e = enc_or_zero(t, (uint32_t)acc & mask, n_sym);
        fn((e & 0xFFFFu) | ((e >> 16) << 24) | ((e >> 16) ? 0u : kGroupInvalid));
        acc >>= r; have -= r;
    }
}

// Saturating 32-bit store of a 64-bit running sum (0xFFFFFFFF = does not fit).
__device__ __forceinline__ uint32_t sat32(unsigned long long v) {
    return v > 0xFFFFFFFEull ? 0xFFFFFFFFu : (uint32_t)v;
}

// Inclusive running sum, in place, of a[0..n) by one CTA of NT threads (a multiple of 32),
// continuing from *s_carry (shared); saturating.  Ends with a barrier; *s_carry holds the
// total.
template <int NT, int PER>
__device__ __forceinline__ void cta_scan_in_place(uint32_t* a, uint64_t n, unsigned long long* s_warp,
                                                  unsigned long long* s_carry) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (uint64_t base = 0; base < n; base += (uint64_t)NT * PER) {
        const uint64_t i0 = base + (uint64_t)tid * PER;
        uint32_t v[PER];
        unsigned long long mine = 0;
#pragma unroll
        for (int k = 0; k < PER; ++k) {
            v[k] = (i0 + k < n) ? a[i0 + k] : 0u;
            mine += v[k];
        }
        unsigned long long incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += up;
        }
        if (lane == 31) s_warp[warp] = incl;
        __syncthreads();
        unsigned long long before = *s_carry + (incl - mine);
        for (int w = 0; w < warp; ++w) before += s_warp[w];
#pragma unroll
        for (int k = 0; k < PER; ++k) {
            before += v[k];
            if (i0 + k < n) a[i0 + k] = sat32(before);
        }
        __syncthreads();
        if (tid == NT - 1) *s_carry = before;
        __syncthreads();
    }
}

// Launch 1: CTA b owns the chunks [b*seg, (b+1)*seg): offsets[c + 1] = words chunk c needs
// (one warp per chunk, one row per lane), then their running sum within the segment.
__global__ void __launch_bounds__(kHuffWarps * 32)
huff_count_kernel(const CodecParams P, const HuffTables* __restrict__ tables,
                  const uint32_t* __restrict__ codes, uint32_t* __restrict__ offsets,
                  uint32_t* status, const uint64_t n_chunks, const uint64_t seg) {
    extern __shared__ uint32_t s_group[];
    __shared__ unsigned long long s_warp[kHuffWarps];
    __shared__ unsigned long long s_carry;
    const uint32_t n_sym = 2 * P.s + 1, k = tables->group_syms;
    build_group_table(s_group, tables, n_sym, P.r, k);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint64_t c0 = (uint64_t)blockIdx.x * seg;
    const uint64_t c1 = c0 + seg < n_chunks ? c0 + seg : n_chunks;
    for (uint64_t c = c0 + warp; c < c1; c += kHuffWarps) {
        const uint64_t e0 = c * kHuffChunk + (uint32_t)lane * 32;
        const uint32_t nv = e0 >= P.d ? 0u : (uint32_t)((P.d - e0 < 32) ? (P.d - e0) : 32);
        uint32_t bits = 0, bad = 0;
        for_each_group(codes, e0 >> 5, P.r, k, nv, s_group, tables, n_sym, [&](uint32_t e) {
            bits += (e >> 24) & 31u;
            bad |= e >> 31;
        });
        bits = __reduce_add_sync(0xFFFFFFFFu, bits);
        bad = __reduce_or_sync(0xFFFFFFFFu, bad);
        if (lane == 0) {
            offsets[c + 1] = (bits + 31) >> 5;
            if (bad) atomicOr(status, kStatusSymbol);
        }
    }
    if (threadIdx.x == 0) s_carry = 0;
    __syncthreads();                        // the segment's counts are written (same CTA)
    cta_scan_in_place<kHuffWarps * 32, 4>(offsets + 1 + c0, c1 - c0, s_warp, &s_carry);
}

// Launch 2: one CTA turns the segment totals (the last entry of every segment) into their
// running sum, which makes those entries final.  A stream beyond `capacity` words (or
// 2^32 - 2) leaves offsets[n_chunks] = 0xFFFFFFFF and raises the capacity flag.
constexpr int kScanThreads = 1024;
__global__ void __launch_bounds__(kScanThreads)
huff_scan_kernel(uint32_t* __restrict__ offsets, const uint64_t n_chunks, const uint64_t seg,
                 const uint64_t capacity, uint32_t* status) {
    __shared__ unsigned long long s_warp[kScanThreads / 32];
    __shared__ unsigned long long s_carry;
    __shared__ uint32_t s_over;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint64_t n_seg = (n_chunks + seg - 1) / seg;
    if (tid == 0) { s_carry = 0; s_over = 0; offsets[0] = 0; }
    __syncthreads();
    for (uint64_t base = 0; base < n_seg; base += kScanThreads) {
        const uint64_t sgm = base + tid;
        const uint64_t at = (sgm + 1) * seg < n_chunks ? (sgm + 1) * seg : n_chunks;   // its last entry
        const uint32_t v = sgm < n_seg ? offsets[at] : 0u;
        if (v == 0xFFFFFFFFu) s_over = 1;
        unsigned long long incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += up;
        }
        if (lane == 31) s_warp[warp] = incl;
        __syncthreads();
        unsigned long long total = s_carry + incl;
        for (int w = 0; w < warp; ++w) total += s_warp[w];
        if (sgm < n_seg) offsets[at] = sat32(total);
        __syncthreads();
        if (tid == kScanThreads - 1) s_carry = total;
        __syncthreads();
    }
    if (tid == 0 && (s_over || s_carry > capacity || s_carry > 0xFFFFFFFEull)) {
        offsets[n_chunks] = 0xFFFFFFFFu;
        atomicOr(status, kStatusCapacity);
    }
}

// Launch 3: the stream.  CTA b first makes the offsets of its segment final (adds the
// words of all earlier segments, which launch 2 left in the entry before the segment).
// Then one warp per chunk: every lane encodes its row into a private strip of shared
// memory, a shuffle scan gives the bit position the rows before it leave, the strip is
// shifted into place in the chunk's zeroed staging area (neighbouring rows share a 32-bit
// word, hence the shared-memory atomics), and the warp copies the chunk out with
// coalesced stores.  Nothing is written when the stream does not fit.
constexpr uint32_t kHuffRowWords = 32 * kHuffMaxLen / 32 + 1;       // longest row, odd stride
__global__ void __launch_bounds__(kHuffWarps * 32)
huff_write_kernel(const CodecParams P, const HuffTables* __restrict__ tables,
                  const uint32_t* __restrict__ codes, uint32_t* __restrict__ offsets,
                  uint16_t* __restrict__ quarters, uint32_t* __restrict__ stream,
                  const uint64_t n_chunks, const uint64_t seg) {
    extern __shared__ uint32_t s_group[];
    const uint32_t n_sym = 2 * P.s + 1, k = tables->group_syms;
    build_group_table(s_group, tables, n_sym, P.r, k);
    if (offsets[n_chunks] == 0xFFFFFFFFu) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint64_t c0 = (uint64_t)blockIdx.x * seg;
    const uint64_t c1 = c0 + seg < n_chunks ? c0 + seg : n_chunks;
    const uint32_t base = offsets[c0];
    for (uint64_t c = c0 + threadIdx.x; c + 1 < c1; c += blockDim.x) offsets[c + 1] += base;
    __syncthreads();
    uint32_t* stage = s_group + (1u << (k * P.r)) + warp * (kHuffChunkWords + 32 + 32 * kHuffRowWords);
    uint32_t* strip = stage + kHuffChunkWords + 32 + lane * kHuffRowWords;
    for (uint64_t c = c0 + warp; c < c1; c += kHuffWarps) {
        const uint32_t first = offsets[c], n_words = offsets[c + 1] - first;
        for (uint32_t i = lane; i < n_words; i += 32) stage[i] = 0;
        const uint64_t e0 = c * kHuffChunk + (uint32_t)lane * 32;
        const uint32_t nv = e0 >= P.d ? 0u : (uint32_t)((P.d - e0 < 32) ? (P.d - e0) : 32);
        // my row, from bit 0 of my strip (a group adds at most 24 bits to at most 31)
        uint64_t win = 0;
        uint32_t fill = 0, sw = 0;
        for_each_group(codes, e0 >> 5, P.r, k, nv, s_group, tables, n_sym, [&](uint32_t e) {
            win |= (uint64_t)(e & 0xFFFFFFu) << fill;
            fill += (e >> 24) & 31u;
            if (fill >= 32) { strip[sw++] = (uint32_t)win; win >>= 32; fill -= 32; }
        });
        strip[sw] = (uint32_t)win;                           // the rest (or zero)
        const uint32_t bits = sw * 32 + fill;
        uint32_t at = bits;                                  // inclusive scan over the lanes
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, at, o);
            if (lane >= o) at += up;
        }
        at -= bits;                                          // my first bit in the chunk
        if (lane && (lane & 7) == 0) quarters[3 * c + (lane >> 3) - 1] = (uint16_t)at;
        __syncwarp();                                        // the staging area is zeroed
        const uint32_t sh = at & 31, w0 = at >> 5;
        const uint32_t n_out = (sh + bits + 31) >> 5;        // staging words my row touches
        uint32_t prev = 0;
        for (uint32_t j = 0; j < n_out; ++j) {
            const uint32_t cur = j <= sw ? strip[j] : 0u;
            const uint32_t v = __funnelshift_l(prev, cur, sh);   // (cur << sh) | (prev >> (32 - sh))
            if (v) atomicOr(stage + w0 + j, v);
            prev = cur;
        }
        __syncwarp();
        for (uint32_t i = lane; i < n_words; i += 32) stream[first + i] = stage[i];
        __syncwarp();
    }
}

// Receiver: one thread per quarter of a chunk walks the stream from the quarter's mark;
// every look-up of the next 12 stream bits yields all the words that lie wholly inside them
// (up to four codes at once for short words), whose r-bit codes are appended to the
// output.  A pattern that is no word raises the symbol flag and ends the quarter (its
// remaining codes are written as zeros).
constexpr int kHuffDecThreads = 128;
__global__ void __launch_bounds__(kHuffDecThreads)
huff_decode_kernel(const CodecParams P, const HuffTables* __restrict__ tables,
                   const uint32_t* __restrict__ stream, const uint32_t* __restrict__ offsets,
                   const uint16_t* __restrict__ quarters, uint32_t* __restrict__ codes,
                   uint32_t* status, const uint64_t n_chunks, const uint64_t n_code_words,
                   const uint64_t stream_len) {
    __shared__ uint32_t s_dec[1u << kHuffMaxLen];
    for (uint32_t k = threadIdx.x; k < (1u << kHuffMaxLen); k += blockDim.x) s_dec[k] = tables->dec[k];
    __syncthreads();
    const uint32_t r = P.r, mask = (1u << r) - 1u;
    // never read beyond the caller's buffer, whatever the offsets say
    const uint64_t end = offsets[n_chunks] < stream_len ? offsets[n_chunks] : stream_len;
    const uint4* stream4 = reinterpret_cast<const uint4*>(stream);       // 16-byte aligned (host check)
    auto load4 = [&](uint64_t b) -> uint4 {
        const uint64_t w = b * 4;
        if (w + 4 <= end) return __ldg(stream4 + b);
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (w < end) v.x = __ldg(stream + w);
        if (w + 1 < end) v.y = __ldg(stream + w + 1);
        if (w + 2 < end) v.z = __ldg(stream + w + 2);
        return v;
    };
    for (uint64_t q = (uint64_t)blockIdx.x * kHuffDecThreads + threadIdx.x; q < 4 * n_chunks;
         q += (uint64_t)gridDim.x * kHuffDecThreads) {
        const uint64_t c = q >> 2;
        const uint32_t part = (uint32_t)q & 3u;
        const uint64_t e0 = c * kHuffChunk + part * kHuffQuarter;
        if (e0 >= P.d) continue;
        uint32_t left = (uint32_t)((P.d - e0 < kHuffQuarter) ? (P.d - e0) : kHuffQuarter);
        const uint32_t bit0 = part ? quarters[3 * c + part - 1] : 0u;
        const uint64_t word0 = (uint64_t)offsets[c] + (bit0 >> 5);
        // the stream is read 16 bytes at a time, one load ahead of its use
        uint64_t blk = word0 >> 2;
        uint32_t sub = (uint32_t)word0 & 3u;
        uint4 cur = load4(blk), nxt = load4(blk + 1);
        uint64_t buf = 0;
        uint32_t have = 0;
        if (bit0 & 31u) {                                   // enter in the middle of a word
            const uint32_t word = sub == 0 ? cur.x : sub == 1 ? cur.y : sub == 2 ? cur.z : cur.w;
            buf = word >> (bit0 & 31u);
            have = 32 - (bit0 & 31u);
            if (++sub == 4) { sub = 0; cur = nxt; ++blk; nxt = load4(blk + 1); }
        }
        uint64_t out = 0;
        uint32_t out_bits = 0;
        uint64_t wr = e0 / 32 * r;                          // first code word of the chunk
        uint4 ow = make_uint4(0u, 0u, 0u, 0u);              // four output words at a time
        uint32_t oi = 0;
        bool ok = true;
        while (left) {
            if (have <= 32) {
                const uint32_t word = sub == 0 ? cur.x : sub == 1 ? cur.y : sub == 2 ? cur.z : cur.w;
                buf |= (uint64_t)word << have;
                have += 32;
                if (++sub == 4) { sub = 0; cur = nxt; ++blk; nxt = load4(blk + 1); }
            }
            const uint32_t e = ok ? s_dec[(uint32_t)buf & ((1u << kHuffMaxLen) - 1u)] : 0u;
            uint32_t n = (e >> 16) & 15u, used = (e >> 20) & 15u, syms = e & 0xFFFFu;
            if (n == 0) { ok = false; n = 1; used = 0; syms = 0; }
            else if (n > left) { n = 1; used = (e >> 24) & 15u; syms &= mask; }
            buf >>= used; have -= used;
            out |= (uint64_t)syms << out_bits;
            out_bits += n * r;
            left -= n;
            if (out_bits >= 32) {
                const uint32_t v = (uint32_t)out;
                out >>= 32; out_bits -= 32;
                if (oi == 0) ow.x = v; else if (oi == 1) ow.y = v; else if (oi == 2) ow.z = v; else ow.w = v;
                if (++oi == 4) {
                    if (wr + 4 <= n_code_words) {
                        *reinterpret_cast<uint4*>(codes + wr) = ow;
                    } else {
                        if (wr < n_code_words) codes[wr] = ow.x;
                        if (wr + 1 < n_code_words) codes[wr + 1] = ow.y;
                        if (wr + 2 < n_code_words) codes[wr + 2] = ow.z;
                    }
                    wr += 4; oi = 0;
                }
            }
        }
        // what is left: up to three whole words and one partial
        if (out_bits) {
            const uint32_t v = (uint32_t)out;
            if (oi == 0) ow.x = v; else if (oi == 1) ow.y = v; else if (oi == 2) ow.z = v; else ow.w = v;
            ++oi;
        }
        if (oi > 0 && wr < n_code_words) codes[wr] = ow.x;
        if (oi > 1 && wr + 1 < n_code_words) codes[wr + 1] = ow.y;
        if (oi > 2 && wr + 2 < n_code_words) codes[wr + 2] = ow.z;
        if (oi > 3 && wr + 3 < n_code_words) codes[wr + 3] = ow.w;
        if (!ok) atomicOr(status, kStatusSymbol);
    }
}

}  // namespace ecq
