// ECQ-SGD gradient codec -- CPU oracle.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, single-threaded, obviously
// correct restatement of the codec of "Error Compensated Quantized SGD"
// (Wu et al., ICML 2018) that the CUDA library is checked against.  It shares no
// source, header, table or helper with the CUDA path and the product never
// calls it.
//
// What it computes, per worker p and iteration t, on a flat fp32 vector that is
// cut into contiguous buckets of B entries (the last one may be shorter):
//
//   encode       Section 4: Eq. 7 (compensation), Eq. 8 with the l-infinity (or l2)
//                scale taken per bucket, Eq. 9 (two-point stochastic rounding),
//                Eq. 6 (incremental error accumulator), and the fixed-width
//                r = ceil(log2(2s+1)) bit code of the paragraph after Eq. 9.
//   decode_mean  Eq. 4 / Algorithm 1, phase 2, global-gradient step: the mean of
//                the P dequantised messages.
//
// The paper works over the reals.  Every fp32 rounding decision below is a
// convention of this codec (one IEEE operation per line, round to nearest even,
// no contraction: build with -ffp-contract=off).  The random draw that turns
// the probability of Eq. 9 into a decision is Philox4x32-10 (Salmon, Moraes,
// Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3", SC'11), written
// here from its published round function.
//
//   decode_mean_update  the same followed by Algorithm 1's model-update step.
//
// Parity pins (tests/test_oracle_*.py): Philox known answers; closed forms for
// r and the message length; hand-worked level-boundary inputs; exact-rational
// threshold checks of the rounding law; brute-force expectation on d = 8;
// unbiasedness (Lemma 1); Eq. 5 == Eq. 6; the recursion used in the proof of
// Lemma 2; conservation at beta = 1; library max-abs; independent unpacking.
// No function here is "parity unpinned".

#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

namespace {

inline uint32_t f2u(float x) { uint32_t u; std::memcpy(&u, &x, 4); return u; }
inline float u2f(uint32_t u) { float x; std::memcpy(&x, &u, 4); return x; }

// ---- Philox4x32-10 (SC'11, Section 3.3 and the reference constants) --------
// One round maps (c0,c1,c2,c3) to
//   (hi(M1*c2) ^ c1 ^ k0, lo(M1*c2), hi(M0*c0) ^ c3 ^ k1, lo(M0*c0))
// and the key is advanced by the Weyl constants between rounds.
const uint32_t kM0 = 0xD2511F53u, kM1 = 0xCD9E8D57u;
const uint32_t kW0 = 0x9E3779B9u, kW1 = 0xBB67AE85u;

void philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        const uint64_t p0 = (uint64_t)kM0 * c0;
        const uint64_t p1 = (uint64_t)kM1 * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        const uint32_t n1 = (uint32_t)p1;
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        const uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += kW0; k1 += kW1;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// The 32-bit word that element i of worker p draws at iteration t:
// counter = (lo32(i/4), hi32(i/4), p, t), key = (lo32(seed), hi32(seed)),
// lane i mod 4 of the four output words.
uint32_t draw_word(uint64_t seed, uint32_t worker, uint32_t step, uint64_t i) {
    const uint64_t blk = i >> 2;
    const uint32_t ctr[4] = {(uint32_t)blk, (uint32_t)(blk >> 32), worker, step};
    const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    uint32_t out[4];
    philox4x32_10(ctr, key, out);
    return out[i & 3];
}

// r = ceil(log2(2s+1)): the smallest width that holds the 2s+1 signed levels
// (paragraph after Eq. 9).
uint32_t code_bits(uint32_t s) {
    uint32_t r = 0;
    while ((1ull << r) < 2ull * s + 1ull) ++r;
    return r;
}

// Write the r-bit value c at stream position `bitpos` (LSB first; stream bit k
// is bit k mod 32 of word k div 32).  The words were zeroed beforehand.
void put_code(uint32_t* words, uint64_t bitpos, uint32_t r, uint32_t c) {
    for (uint32_t j = 0; j < r; ++j) {
        const uint64_t k = bitpos + j;
        if ((c >> j) & 1u) words[k >> 5] |= (1u << (k & 31));
    }
}

uint32_t get_code(const uint32_t* words, uint64_t bitpos, uint32_t r) {
    uint32_t c = 0;
    for (uint32_t j = 0; j < r; ++j) {
        const uint64_t k = bitpos + j;
        c |= ((words[k >> 5] >> (k & 31)) & 1u) << j;
    }
    return c;
}

enum { STATUS_NONFINITE = 1u };

// Encode one slice.  `first_index` is the global index of g[0] (a multiple of
// B) so that a sampled run of whole buckets can be checked at any position of
// a large vector; `random_words`, when not null, replaces the Philox draw
// (one word per element) so that tests can choose the draws.
int encode_core(uint64_t n, uint32_t B, uint32_t s, float alpha, float beta,
                uint64_t seed, int mode, int norm, uint32_t worker, uint32_t step,
                uint64_t first_index, const uint32_t* random_words,
                const float* g, float* h, uint32_t* codes, float* scales,
                uint32_t* status) {
    if (B == 0 || B % 32 != 0 || s == 0 || s > 32767 || first_index % B != 0) return 1;
    const uint32_t r = code_bits(s);
    const uint64_t nb = (n + B - 1) / B;
    const uint64_t nwords = (n * r + 31) / 32;
    for (uint64_t k = 0; k < nwords; ++k) codes[k] = 0;
    const float sf = (float)s;
    std::vector<float> v(B);

    for (uint64_t b = 0; b < nb; ++b) {
        const uint64_t lo = b * B;
        const uint64_t hi = (lo + B < n) ? lo + B : n;

        // Eq. 7: compensated gradient v = g + alpha*h (one fused multiply-add).
        uint32_t sbits = 0;
        for (uint64_t i = lo; i < hi; ++i) {
            v[i - lo] = std::fmaf(alpha, h[i], g[i]);
            // Eq. 8 scale, l-infinity over the bucket: for non-negative IEEE
            // values the integer order of the bit patterns is the numeric
            // order, and NaN/Inf patterns sort above every finite value.
            const uint32_t a = f2u(v[i - lo]) & 0x7FFFFFFFu;
            if (a > sbits) sbits = a;
        }
        float scale = u2f(sbits);
        if (norm == 1) {
            // Eq. 8 with the l2 norm.  The fp32 sum of squares needs a stated order:
            // each run of 32 consecutive entries is summed front to back with one fused
            // multiply-add per entry, and the run sums are combined pairwise in index
            // order, level by level (an odd one out is carried up unchanged).
            std::vector<float> runs;
            for (uint64_t i = lo; i < hi; i += 32) {
                float acc = 0.0f;
                for (uint64_t j = i; j < hi && j < i + 32; ++j) acc = std::fmaf(v[j - lo], v[j - lo], acc);
                runs.push_back(acc);
            }
            while (runs.size() > 1) {
                std::vector<float> up;
                for (size_t k = 0; k < runs.size(); k += 2)
                    up.push_back(k + 1 < runs.size() ? runs[k] + runs[k + 1] : runs[k]);
                runs.swap(up);
            }
            sbits = f2u(runs[0]) & 0x7FFFFFFFu;       // NaN/Inf (also an overflowed sum) sort on top
            scale = std::sqrt(runs[0]);
        }

        bool zero_bucket = false;
        float inv = 0.0f, a_step = 0.0f;
        if (sbits >= 0x7F800000u) {
            // Non-finite input: the bucket is sent as all-zero levels with
            // scale 0, its accumulator is left untouched, and the condition is
            // reported.
            if (status) *status |= STATUS_NONFINITE;
            for (uint64_t i = lo; i < hi; ++i)
                put_code(codes, i * r, r, s);
            scales[b] = 0.0f;
            continue;
        }
        if (scale == 0.0f) {
            zero_bucket = true;
        } else {
            inv = sf / scale;                       // s / ||v||, once per bucket
            if (std::isinf(inv)) zero_bucket = true;
            a_step = scale / sf;                    // level step ||v|| / s
        }
        if (zero_bucket) {
            // Every level is 0; Eq. 6 with g~ = 0.
            for (uint64_t i = lo; i < hi; ++i) {
                put_code(codes, i * r, r, s);
                const float vi = v[i - lo];
                const float e = (mode == 0) ? g[i] : vi;
                h[i] = std::fmaf(beta, h[i], e);
            }
            scales[b] = 0.0f;
            continue;
        }

        for (uint64_t i = lo; i < hi; ++i) {
            const float vi = v[i - lo];
            // Eq. 9: s*|v_i|/||v|| lies in [l, l+1); go up with probability
            // equal to the fractional part.  The clamp keeps the ratio at s
            // when the rounded reciprocal overshoots by an ulp.
            float x = std::fabs(vi) * inv;
            if (x > sf) x = sf;
            const int32_t l = (int32_t)x;           // floor, x >= 0
            const float f = x - (float)l;           // exact
            const uint32_t R = random_words ? random_words[i]
                                            : draw_word(seed, worker, step, first_index + i);
            const float u = (float)(R >> 8) * 0x1p-24f;   // uniform on {0..2^24-1}/2^24
            const int32_t m = l + ((u < f) ? 1 : 0);
            // Eq. 8: sign of v_i times the level; the code is the level index
            // shifted to be non-negative.
            const int32_t q = (f2u(vi) >> 31) ? -m : m;
            put_code(codes, i * r, r, (uint32_t)(q + (int32_t)s));
            const float gq = (float)q * a_step;     // dequantised value g~_i
            // Eq. 6: h <- beta*h + (g - g~).  Mode 1 books the compensated
            // value instead of the raw gradient.
            const float e = ((mode == 0) ? g[i] : vi) - gq;
            h[i] = std::fmaf(beta, h[i], e);
        }
        scales[b] = scale;
    }
    return 0;
}

}  // namespace

extern "C" {

void ecqo_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) {
    philox4x32_10(ctr, key, out);
}

uint32_t ecqo_draw_word(uint64_t seed, uint32_t worker, uint32_t step, uint64_t i) {
    return draw_word(seed, worker, step, i);
}

uint32_t ecqo_code_bits(uint32_t s) { return code_bits(s); }

uint64_t ecqo_num_buckets(uint64_t d, uint32_t B) { return (d + B - 1) / B; }

uint64_t ecqo_codes_words(uint64_t d, uint32_t s) { return (d * code_bits(s) + 31) / 32; }

int ecqo_encode(uint64_t n, uint32_t B, uint32_t s, float alpha, float beta,
                uint64_t seed, int mode, int norm, uint32_t worker, uint32_t step,
                uint64_t first_index, const float* g, float* h,
                uint32_t* codes, float* scales, uint32_t* status) {
    return encode_core(n, B, s, alpha, beta, seed, mode, norm, worker, step, first_index,
                       nullptr, g, h, codes, scales, status);
}

int ecqo_encode_given_draws(uint64_t n, uint32_t B, uint32_t s, float alpha, float beta,
                            int mode, int norm, const uint32_t* random_words, const float* g,
                            float* h, uint32_t* codes, float* scales, uint32_t* status) {
    return encode_core(n, B, s, alpha, beta, 0, mode, norm, 0, 0, 0, random_words, g, h,
                       codes, scales, status);
}

// Eq. 4 / Algorithm 1, phase 2, global-gradient step: out_i = (1/W) sum_w q_{w,i} a_{w,b},
// a_{w,b} = scale_{w,b}/s, summed in ascending w, then one division by W.
int ecqo_decode_mean(uint64_t n, uint32_t B, uint32_t s, uint32_t W,
                     const uint32_t* const* codes, const float* const* scales,
                     float* out) {
    if (B == 0 || B % 32 != 0 || s == 0 || s > 32767 || W == 0) return 1;
    const uint32_t r = code_bits(s);
    const float sf = (float)s;
    for (uint64_t i = 0; i < n; ++i) {
        const uint64_t b = i / B;
        float acc = 0.0f;
        for (uint32_t w = 0; w < W; ++w) {
            const float a = scales[w][b] / sf;
            const int32_t q = (int32_t)get_code(codes[w], i * r, r) - (int32_t)s;
            acc = std::fmaf((float)q, a, acc);
        }
        out[i] = acc / (float)W;
    }
    return 0;
}

// Algorithm 1, phase 2, model-update step: w <- w - eta * g~, with g~ the mean above,
// as one fused multiply-add per entry.
int ecqo_decode_mean_update(uint64_t n, uint32_t B, uint32_t s, uint32_t W,
                            const uint32_t* const* codes, const float* const* scales,
                            float eta, float* params, float* out) {
    std::vector<float> mean(n);
    const int rc = ecqo_decode_mean(n, B, s, W, codes, scales, mean.data());
    if (rc != 0) return rc;
    for (uint64_t i = 0; i < n; ++i) {
        params[i] = std::fmaf(-eta, mean[i], params[i]);
        if (out) out[i] = mean[i];
    }
    return 0;
}

// Level counts d_k of one message and the entropy-coding bound of the paragraph after
// Eq. 9: at most sum_k d_k log2(d / d_k) bits.
void ecqo_code_histogram(uint64_t n, uint32_t s, const uint32_t* codes, uint64_t* counts) {
    const uint32_t r = code_bits(s);
    for (uint32_t k = 0; k < 2 * s + 1; ++k) counts[k] = 0;
    for (uint64_t i = 0; i < n; ++i) {
        const uint32_t c = get_code(codes, i * r, r);
        if (c < 2 * s + 1) counts[c] += 1;
    }
}

double ecqo_entropy_bound_bits(const uint64_t* counts, uint32_t n_bins) {
    double d = 0.0, bits = 0.0;
    for (uint32_t k = 0; k < n_bins; ++k) d += (double)counts[k];
    for (uint32_t k = 0; k < n_bins; ++k)
        if (counts[k]) bits += (double)counts[k] * std::log2(d / (double)counts[k]);
    return bits;
}

// Unpack one message into signed levels q_i (test helper for round trips).
void ecqo_unpack_levels(uint64_t n, uint32_t s, const uint32_t* codes, int32_t* q) {
    const uint32_t r = code_bits(s);
    for (uint64_t i = 0; i < n; ++i) q[i] = (int32_t)get_code(codes, i * r, r) - (int32_t)s;
}

}  // extern "C"
