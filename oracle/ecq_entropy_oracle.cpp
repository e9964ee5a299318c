// ECQ-SGD gradient codec -- CPU oracle of the entropy-coded message.
//
// TEST INFRASTRUCTURE ONLY (see ecq_oracle.cpp): shares nothing with the CUDA
// path and is never called by the product.
//
// The paragraph after Eq. 9 notes that the fixed r-bit codes can be compressed
// further by an entropy code "e.g. Huffman", and the linear-model experiments
// count their communication cost with such a code.  The paper fixes nothing
// beyond that, so the format below is this codec's convention:
//
//   * symbols are the level indices c = q + s in [0, 2s], with d_k occurrences;
//   * code lengths come from an optimal prefix code whose longest word has at
//     most `max_len` bits (length-limited Huffman; with max_len large enough
//     it is Huffman's code).  Construction: the package-merge procedure of
//     Larmore and Hirschberg (JACM 1990), stated on explicit trees of packages;
//   * code words are canonical: symbols ordered by (length, index), first word
//     all zeros, each next word = (previous + 1) shifted left by the growth in
//     length;
//   * the bits of a word enter the stream in tree order (the word's most
//     significant bit first); the stream is a sequence of 32-bit words whose
//     bit k is bit (k mod 32) of word k / 32;
//   * the entries are cut into chunks of 1024; every chunk starts on a word
//     boundary, offsets[c] is its first word and offsets[n_chunks] the length
//     of the stream in words (unused bits of a chunk's last word are zero);
//   * so that a chunk can be decoded by four independent readers, quarters[3c + j]
//     (j = 0, 1, 2) is the bit position, counted from the chunk's first word, at
//     which entry 256 (j + 1) of the chunk starts (the chunk's end if it has fewer
//     entries).
//
// Pins (tests/test_oracle_entropy.py): exhaustive search over all admissible
// length vectors on tiny alphabets; a textbook six-symbol example; Huffman's
// cost via a heap on random histograms when the limit is slack; a
// dynamic-programme optimum when it binds; Kraft equality; prefix-freeness by
// pairwise comparison; a hand-packed stream; round trips.

#include <algorithm>
#include <cstdint>
#include <vector>

namespace {

const uint32_t kChunk = 1024;
const uint32_t kQuarter = 256;

uint32_t get_bits(const uint32_t* words, uint64_t bit, uint32_t n) {
    uint32_t v = 0;
    for (uint32_t k = 0; k < n; ++k) {
        const uint64_t b = bit + k;
        v |= ((words[b >> 5] >> (b & 31)) & 1u) << k;
    }
    return v;
}

// A node of the package-merge forest: a leaf (one symbol) or a package of two nodes.
struct Node {
    uint64_t weight;
    int32_t left, right;    // -1 for a leaf
    uint32_t symbol;
};

void count_leaves(const std::vector<Node>& nodes, int32_t at, std::vector<uint32_t>& len) {
    if (nodes[at].left < 0) { len[nodes[at].symbol] += 1; return; }
    count_leaves(nodes, nodes[at].left, len);
    count_leaves(nodes, nodes[at].right, len);
}

// Canonical code words from lengths (0 = symbol absent).  Returns false when the
// lengths are not those of a prefix code (Kraft sum above 1) or exceed 32 bits.
bool canonical_words(const uint8_t* lengths, uint32_t n_sym, std::vector<uint32_t>& word) {
    word.assign(n_sym, 0);
    std::vector<uint32_t> order;
    for (uint32_t k = 0; k < n_sym; ++k) {
        if (lengths[k] > 32) return false;
        if (lengths[k]) order.push_back(k);
    }
    std::stable_sort(order.begin(), order.end(),
                     [&](uint32_t a, uint32_t b) { return lengths[a] < lengths[b]; });
    uint64_t next = 0;
    uint32_t prev_len = 0;
    for (size_t i = 0; i < order.size(); ++i) {
        const uint32_t L = lengths[order[i]];
        if (i > 0) next = (next + 1) << (L - prev_len);
        if (next >> L) return false;              // ran out of words of this length
        word[order[i]] = (uint32_t)next;
        prev_len = L;
    }
    return true;
}

}  // namespace

extern "C" {

// Lengths of an optimal prefix code with no word longer than max_len, for the symbols
// with counts[k] > 0 (the others get length 0).  A lone symbol gets a 1-bit word.
// Returns 0, or 1 if the limit cannot hold the alphabet (more than 2^max_len symbols).
int ecqo_huffman_lengths(const uint64_t* counts, uint32_t n_sym, uint32_t max_len,
                         uint8_t* lengths) {
    std::vector<uint32_t> present;
    for (uint32_t k = 0; k < n_sym; ++k) {
        lengths[k] = 0;
        if (counts[k]) present.push_back(k);
    }
    const size_t n = present.size();
    if (n == 0) return 0;
    if (n == 1) { lengths[present[0]] = 1; return 0; }
    if (max_len == 0 || max_len > 32 || (max_len < 32 && n > ((size_t)1 << max_len))) return 1;

    // leaves in order of weight (ties: by symbol index)
    std::stable_sort(present.begin(), present.end(),
                     [&](uint32_t a, uint32_t b) { return counts[a] < counts[b]; });
    std::vector<Node> nodes;
    auto new_leaves = [&]() {
        std::vector<int32_t> ids;
        for (uint32_t sym : present) {
            nodes.push_back(Node{counts[sym], -1, -1, sym});
            ids.push_back((int32_t)nodes.size() - 1);
        }
        return ids;
    };
    // The list of the deepest level holds the leaves alone.  Going up one level: pair the
    // list's nodes from the front into packages (an odd one out is dropped) and merge the
    // packages with a fresh copy of the leaves by weight (a leaf before a package of
    // equal weight).
    std::vector<int32_t> list = new_leaves();
    for (uint32_t level = 1; level < max_len; ++level) {
        std::vector<int32_t> packages;
        for (size_t i = 0; i + 1 < list.size(); i += 2) {
            nodes.push_back(Node{nodes[list[i]].weight + nodes[list[i + 1]].weight,
                                 list[i], list[i + 1], 0});
            packages.push_back((int32_t)nodes.size() - 1);
        }
        const std::vector<int32_t> leaves = new_leaves();
        std::vector<int32_t> merged;
        size_t a = 0, b = 0;
        while (a < leaves.size() || b < packages.size()) {
            const bool take_leaf = b == packages.size() ||
                (a < leaves.size() && nodes[leaves[a]].weight <= nodes[packages[b]].weight);
            merged.push_back(take_leaf ? leaves[a++] : packages[b++]);
        }
        list.swap(merged);
    }
    // The 2n - 2 lightest nodes of the top list: a symbol's length is the number of times
    // its leaf occurs in them.
    std::vector<uint32_t> len(n_sym, 0);
    for (size_t i = 0; i < 2 * n - 2; ++i) count_leaves(nodes, list[i], len);
    for (uint32_t k = 0; k < n_sym; ++k) lengths[k] = (uint8_t)len[k];
    return 0;
}

// Canonical code words (as integers whose bit L-1 is the first bit sent).
int ecqo_huffman_words(const uint8_t* lengths, uint32_t n_sym, uint32_t* words) {
    std::vector<uint32_t> w;
    if (!canonical_words(lengths, n_sym, w)) return 1;
    for (uint32_t k = 0; k < n_sym; ++k) words[k] = w[k];
    return 0;
}

uint64_t ecqo_huffman_chunks(uint64_t n) { return (n + kChunk - 1) / kChunk; }

// Entropy-code the n r-bit codes of `codes`.  stream must hold `capacity` words;
// offsets n_chunks + 1 entries, quarters 3 n_chunks.  Returns 0; 1 for lengths that are no
// prefix code or a symbol without a word; 2 if the stream does not fit (nothing useful is
// written).
int ecqo_huffman_encode(uint64_t n, uint32_t r, const uint8_t* lengths, uint32_t n_sym,
                        const uint32_t* codes, uint32_t* stream, uint64_t capacity,
                        uint32_t* offsets, uint16_t* quarters) {
    std::vector<uint32_t> word;
    if (!canonical_words(lengths, n_sym, word)) return 1;
    const uint64_t n_chunks = ecqo_huffman_chunks(n);
    uint64_t at = 0;                                   // next free word
    for (uint64_t c = 0; c < n_chunks; ++c) {
        offsets[c] = (uint32_t)at;
        const uint64_t lo = c * kChunk, hi = std::min<uint64_t>(n, lo + kChunk);
        uint64_t bit = at * 32;
        for (uint32_t j = 0; j < 3; ++j) quarters[3 * c + j] = 0;
        for (uint64_t i = lo; i < hi; ++i) {
            if (i > lo && (i - lo) % kQuarter == 0)
                quarters[3 * c + (i - lo) / kQuarter - 1] = (uint16_t)(bit - at * 32);
            const uint32_t sym = get_bits(codes, i * r, r);
            if (sym >= n_sym || lengths[sym] == 0) return 1;
            const uint32_t L = lengths[sym];
            if ((bit + L + 31) / 32 > capacity) return 2;
            for (uint32_t k = 0; k < L; ++k) {         // first bit sent = top bit of the word
                const uint32_t b = (word[sym] >> (L - 1 - k)) & 1u;
                if ((bit & 31) == 0) stream[bit >> 5] = 0;
                stream[bit >> 5] |= b << (bit & 31);
                ++bit;
            }
        }
        for (uint64_t q = (hi - lo + kQuarter - 1) / kQuarter; q < 4; ++q)   // quarters that do not exist
            if (q > 0) quarters[3 * c + q - 1] = (uint16_t)(bit - at * 32);
        at = (bit + 31) / 32;
    }
    if (at > 0xFFFFFFFFull) return 2;
    offsets[n_chunks] = (uint32_t)at;
    return 0;
}

// Inverse: walks the stream bit by bit, extending the current word until it equals a
// code word of that length; every quarter of a chunk is entered at its recorded bit
// position.  Writes the n symbols as r-bit codes (unused bits of the last word zero).
// Returns 0, or 1 on a bit pattern that is no code word.
int ecqo_huffman_decode(uint64_t n, uint32_t r, const uint8_t* lengths, uint32_t n_sym,
                        const uint32_t* stream, const uint32_t* offsets,
                        const uint16_t* quarters, uint32_t* codes) {
    std::vector<uint32_t> word;
    if (!canonical_words(lengths, n_sym, word)) return 1;
    std::vector<std::vector<uint32_t>> of_length(33);      // the symbols of every word length
    for (uint32_t k = 0; k < n_sym; ++k)
        if (lengths[k]) of_length[lengths[k]].push_back(k);
    const uint64_t n_words = (n * r + 31) / 32;
    for (uint64_t k = 0; k < n_words; ++k) codes[k] = 0;
    const uint64_t n_chunks = ecqo_huffman_chunks(n);
    for (uint64_t c = 0; c < n_chunks; ++c) {
        const uint64_t lo = c * kChunk, hi = std::min<uint64_t>(n, lo + kChunk);
        uint64_t bit = (uint64_t)offsets[c] * 32;
        for (uint64_t i = lo; i < hi; ++i) {
            if (i > lo && (i - lo) % kQuarter == 0)
                bit = (uint64_t)offsets[c] * 32 + quarters[3 * c + (i - lo) / kQuarter - 1];
            uint32_t acc = 0, L = 0, sym = n_sym;
            while (sym == n_sym) {
                if (L == 32) return 1;
                acc = (acc << 1) | ((stream[bit >> 5] >> (bit & 31)) & 1u);
                ++bit; ++L;
                for (uint32_t k : of_length[L])
                    if (word[k] == acc) { sym = k; break; }
            }
            for (uint32_t k = 0; k < r; ++k) {
                const uint64_t b = i * r + k;
                codes[b >> 5] |= ((sym >> k) & 1u) << (b & 31);
            }
        }
    }
    return 0;
}

}  // extern "C"
