// Entropy-coded message (paragraph after Eq. 9: the r-bit codes "can be further compressed
// by entropy coding, e.g. Huffman"; the linear-model experiments count bits that way).
//
// Format: canonical prefix code over the 2s+1 level indices with words of at most 12 bits;
// a word's bits enter the stream in tree order, first bit in the lowest free bit of the
// current 32-bit word; the entries are cut into chunks of 1024, every chunk starts on a
// word boundary, offsets[c] is its first word and offsets[n_chunks] the stream length.
//
// Sender: three launches -- words needed per chunk, their running sum, the stream itself
// (a single pass cannot place a chunk before all earlier chunk sizes are known, and no
// kernel here waits on another).  Receiver: one launch, one thread per chunk.
#pragma once

#include "ecq_common.cuh"

namespace ecq {

constexpr uint32_t kHuffMaxLen = 12;
constexpr uint32_t kHuffChunk = 1024;
constexpr uint32_t kHuffMaxSymbols = 1u << kHuffMaxLen;
constexpr uint32_t kHuffChunkWords = kHuffChunk * kHuffMaxLen / 32;     // longest chunk
constexpr int kHuffWarps = 8;
constexpr uint32_t kStatusCapacity = 4u;    // device status word bits (after 1 and 2)
constexpr uint32_t kStatusSymbol = 8u;

// Device tables of one code, built on the host:
//   enc[c]  = length << 16 | the word with its first bit in bit 0      (c < 4096)
//   dec[p]  = symbol << 4 | length for every 12-bit pattern p whose low bits spell
//             a word; 0 where no word matches
struct HuffTables {
    uint32_t enc[kHuffMaxSymbols];
    uint16_t dec[1u << kHuffMaxLen];
};

// The 32 codes of row `row` (r whole words) -> `fn(j, c)` for the nv valid ones.
template <typename F>
__device__ __forceinline__ void for_each_code(const uint32_t* __restrict__ codes, uint64_t row,
                                              uint32_t r, uint32_t nv, F fn) {
    const uint32_t* w = codes + row * r;
    const uint32_t nw = (nv * r + 31) >> 5;
    const uint32_t mask = (1u << r) - 1u;
    uint64_t acc = 0;
    uint32_t have = 0, kw = 0;
    for (uint32_t j = 0; j < nv; ++j) {
        if (have < r) { acc |= (uint64_t)(kw < nw ? __ldg(w + kw) : 0u) << have; ++kw; have += 32; }
        fn(j, (uint32_t)acc & mask);
        acc >>= r; have -= r;
    }
}

__device__ __forceinline__ void load_enc_table(uint32_t* s_enc, const HuffTables* t, uint32_t n_sym) {
    for (uint32_t k = threadIdx.x; k < n_sym; k += blockDim.x) s_enc[k] = t->enc[k];
    __syncthreads();
}

// Launch 1: offsets[c + 1] = words chunk c needs.  One warp per chunk, one row per lane.
__global__ void __launch_bounds__(kHuffWarps * 32)
huff_count_kernel(const CodecParams P, const HuffTables* __restrict__ tables,
                  const uint32_t* __restrict__ codes, uint32_t* __restrict__ offsets,
                  uint32_t* status, const uint64_t n_chunks) {
    extern __shared__ uint32_t s_enc[];
    const uint32_t n_sym = 2 * P.s + 1;
    load_enc_table(s_enc, tables, n_sym);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (uint64_t c = (uint64_t)blockIdx.x * kHuffWarps + warp; c < n_chunks;
         c += (uint64_t)gridDim.x * kHuffWarps) {
        const uint64_t e0 = c * kHuffChunk + (uint32_t)lane * 32;
        const uint32_t nv = e0 >= P.d ? 0u : (uint32_t)((P.d - e0 < 32) ? (P.d - e0) : 32);
        uint32_t bits = 0, bad = 0;
        for_each_code(codes, e0 >> 5, P.r, nv, [&](uint32_t, uint32_t sym) {
            const uint32_t e = sym < n_sym ? s_enc[sym] : 0u;
            bits += e >> 16;
            bad |= (e >> 16) == 0;
        });
        bits = __reduce_add_sync(0xFFFFFFFFu, bits);
        bad = __reduce_or_sync(0xFFFFFFFFu, bad);
        if (lane == 0) {
            offsets[c + 1] = (bits + 31) >> 5;
            if (bad) atomicOr(status, kStatusSymbol);
        }
    }
}

// Launch 2: running sum in place, offsets[0] = 0.  One CTA; every thread owns 16
// consecutive entries per sweep.  A stream beyond `capacity` words (or 2^32 - 2) leaves
// offsets[n_chunks] = 0xFFFFFFFF and raises the capacity flag.
constexpr int kScanThreads = 1024, kScanPer = 16;
__global__ void __launch_bounds__(kScanThreads)
huff_scan_kernel(uint32_t* __restrict__ offsets, const uint64_t n_chunks, const uint64_t capacity,
                 uint32_t* status) {
    __shared__ unsigned long long s_warp[kScanThreads / 32];
    __shared__ unsigned long long s_carry;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) { s_carry = 0; offsets[0] = 0; }
    __syncthreads();
    for (uint64_t base = 0; base < n_chunks; base += (uint64_t)kScanThreads * kScanPer) {
        const uint64_t i0 = base + (uint64_t)tid * kScanPer;
        uint32_t v[kScanPer];
        unsigned long long mine = 0;
#pragma unroll
        for (int k = 0; k < kScanPer; ++k) {
            v[k] = (i0 + k < n_chunks) ? offsets[1 + i0 + k] : 0u;
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
        unsigned long long before = s_carry + (incl - mine);
        for (int w = 0; w < warp; ++w) before += s_warp[w];
#pragma unroll
        for (int k = 0; k < kScanPer; ++k) {
            before += v[k];
            if (i0 + k < n_chunks)
                offsets[1 + i0 + k] = before > 0xFFFFFFFEull ? 0xFFFFFFFFu : (uint32_t)before;
        }
        __syncthreads();
        if (tid == kScanThreads - 1) s_carry = before;
        __syncthreads();
    }
    if (tid == 0 && (s_carry > capacity || s_carry > 0xFFFFFFFEull)) {
        offsets[n_chunks] = 0xFFFFFFFFu;
        atomicOr(status, kStatusCapacity);
    }
}

// Launch 3: the stream.  One warp per chunk: every lane lays the words of its row into a
// zeroed staging area at the bit position the rows before it leave (neighbouring rows
// share a 32-bit word, hence the shared-memory atomics), then the warp copies the chunk
// out with coalesced stores.  Nothing is written when the stream does not fit.
__global__ void __launch_bounds__(kHuffWarps * 32)
huff_write_kernel(const CodecParams P, const HuffTables* __restrict__ tables,
                  const uint32_t* __restrict__ codes, const uint32_t* __restrict__ offsets,
                  uint32_t* __restrict__ stream, const uint64_t n_chunks) {
    extern __shared__ uint32_t s_enc[];
    const uint32_t n_sym = 2 * P.s + 1;
    load_enc_table(s_enc, tables, n_sym);
    if (offsets[n_chunks] == 0xFFFFFFFFu) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t* stage = s_enc + ((n_sym + 31) & ~31u) + warp * (kHuffChunkWords + 32);
    for (uint64_t c = (uint64_t)blockIdx.x * kHuffWarps + warp; c < n_chunks;
         c += (uint64_t)gridDim.x * kHuffWarps) {
        const uint32_t first = offsets[c], n_words = offsets[c + 1] - first;
        for (uint32_t k = lane; k < n_words; k += 32) stage[k] = 0;
        __syncwarp();
        const uint64_t e0 = c * kHuffChunk + (uint32_t)lane * 32;
        const uint32_t nv = e0 >= P.d ? 0u : (uint32_t)((P.d - e0 < 32) ? (P.d - e0) : 32);
        uint32_t bits = 0;
        for_each_code(codes, e0 >> 5, P.r, nv, [&](uint32_t, uint32_t sym) {
            bits += (sym < n_sym ? s_enc[sym] : 0u) >> 16;
        });
        uint32_t at = bits;                                  // inclusive scan over the lanes
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, at, o);
            if (lane >= o) at += up;
        }
        at -= bits;                                          // my first bit in the chunk
        uint64_t acc = 0;
        uint32_t fill = at & 31, wi = at >> 5;
        for_each_code(codes, e0 >> 5, P.r, nv, [&](uint32_t, uint32_t sym) {
            const uint32_t e = sym < n_sym ? s_enc[sym] : 0u;
            acc |= (uint64_t)(e & 0xFFFFu) << fill;
            fill += e >> 16;
            if (fill >= 32) {
                atomicOr(stage + wi, (uint32_t)acc);
                acc >>= 32; fill -= 32; ++wi;
            }
        });
        if (fill) atomicOr(stage + wi, (uint32_t)acc);
        __syncwarp();
        for (uint32_t k = lane; k < n_words; k += 32) stream[first + k] = stage[k];
        __syncwarp();
    }
}

// Receiver: one thread per chunk walks its words with a 12-bit look-up per symbol and
// writes the r-bit codes of its 1024 entries.  A pattern that is no word raises the
// symbol flag and ends the chunk (its remaining codes are written as zero words).
constexpr int kHuffDecThreads = 128;
__global__ void __launch_bounds__(kHuffDecThreads)
huff_decode_kernel(const CodecParams P, const HuffTables* __restrict__ tables,
                   const uint32_t* __restrict__ stream, const uint32_t* __restrict__ offsets,
                   uint32_t* __restrict__ codes, uint32_t* status, const uint64_t n_chunks,
                   const uint64_t n_code_words, const uint64_t stream_len) {
    __shared__ uint16_t s_dec[1u << kHuffMaxLen];
    for (uint32_t k = threadIdx.x; k < (1u << kHuffMaxLen); k += blockDim.x) s_dec[k] = tables->dec[k];
    __syncthreads();
    const uint32_t r = P.r;
    // never read beyond the caller's buffer, whatever the offsets say
    const uint64_t end = offsets[n_chunks] < stream_len ? offsets[n_chunks] : stream_len;
    for (uint64_t c = (uint64_t)blockIdx.x * kHuffDecThreads + threadIdx.x; c < n_chunks;
         c += (uint64_t)gridDim.x * kHuffDecThreads) {
        const uint64_t e0 = c * kHuffChunk;
        const uint32_t nv = (uint32_t)((P.d - e0 < kHuffChunk) ? (P.d - e0) : kHuffChunk);
        uint64_t rd = offsets[c];
        uint64_t buf = 0;
        uint32_t have = 0;
        uint64_t out = 0;
        uint32_t out_bits = 0;
        uint64_t wr = e0 / 32 * r;                          // first code word of the chunk
        bool ok = true;
        for (uint32_t j = 0; j < nv; ++j) {
            if (have <= 32) {
                buf |= (uint64_t)(rd < end ? __ldg(stream + rd) : 0u) << have;
                ++rd; have += 32;
            }
            const uint32_t e = ok ? s_dec[(uint32_t)buf & ((1u << kHuffMaxLen) - 1u)] : 0u;
            const uint32_t len = e & 15u;
            if (len == 0) ok = false;
            buf >>= len; have -= len;
            out |= (uint64_t)(e >> 4) << out_bits;
            out_bits += r;
            if (out_bits >= 32) {
                codes[wr++] = (uint32_t)out;
                out >>= 32; out_bits -= 32;
            }
        }
        if (out_bits && wr < n_code_words) codes[wr] = (uint32_t)out;
        if (!ok) atomicOr(status, kStatusSymbol);
    }
}

}  // namespace ecq
