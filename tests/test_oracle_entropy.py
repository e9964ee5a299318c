"""Pins of the oracle's entropy-coded message (paragraph after Eq. 9: the r-bit codes "can be
further compressed by entropy coding, e.g. Huffman").  The oracle's length-limited Huffman
construction, canonical words, chunked stream and its inverse are checked against things
that are not the oracle: exhaustive search, a heap, a dynamic programme, hand-packed bits."""
import heapq
import itertools
import math

import numpy as np
import pytest

import oracle


def cost(counts, lengths):
    return int(sum(int(c) * int(l) for c, l in zip(counts, lengths)))


def kraft(lengths, max_len):
    """Kraft sum in units of 2^-max_len (exact integer)."""
    return sum(1 << (max_len - int(l)) for l in lengths if l)


# ------------------------------------------------------------- the lengths ---
def test_exhaustive_optimum_on_tiny_alphabets():
    # every length vector with all words <= max_len and Kraft sum <= 1 is a prefix code;
    # the oracle's must be one of the cheapest
    rng = np.random.default_rng(1)
    for n in (2, 3, 4, 5):
        for max_len in range(max(1, math.ceil(math.log2(n))), 5):
            for trial in range(12):
                counts = rng.integers(1, 9 if trial % 2 else 200, size=n)
                best = min(cost(counts, ls) for ls in itertools.product(range(1, max_len + 1), repeat=n)
                           if kraft(ls, max_len) <= (1 << max_len))
                L = oracle.huffman_lengths(counts, max_len=max_len)
                assert L.max() <= max_len and L.min() >= 1
                assert kraft(L, max_len) <= (1 << max_len)
                assert cost(counts, L) == best, (counts, max_len, L)


def test_textbook_six_symbol_example():
    # frequencies 45, 13, 12, 16, 9, 5 (in thousands) -- the classic worked example whose
    # optimal code spends 224 (thousand) bits with words of 1, 3, 3, 3, 4, 4 bits
    counts = np.array([45, 13, 12, 16, 9, 5])
    L = oracle.huffman_lengths(counts, max_len=12)
    assert cost(counts, L) == 224
    assert sorted(L.tolist()) == [1, 3, 3, 3, 4, 4]
    assert L[0] == 1 and set(L[[4, 5]].tolist()) == {4}


def heap_huffman_cost(counts):
    h = [int(c) for c in counts if c]
    heapq.heapify(h)
    total = 0
    while len(h) > 1:
        a, b = heapq.heappop(h), heapq.heappop(h)
        total += a + b
        heapq.heappush(h, a + b)
    return total


def test_slack_limit_gives_huffman_cost():
    rng = np.random.default_rng(2)
    for trial in range(60):
        n = int(rng.integers(2, 70))
        counts = rng.integers(0, 5, size=n) * rng.integers(1, 10 ** int(rng.integers(1, 7)), size=n)
        if np.count_nonzero(counts) < 2:
            counts[:2] = (3, 4)
        L = oracle.huffman_lengths(counts, max_len=32)
        assert cost(counts, L) == heap_huffman_cost(counts)
        assert np.all((L == 0) == (counts == 0))


def dp_limited_cost(counts, max_len):
    """Cheapest sum(count * length) over all length vectors with Kraft sum <= 1, by a
    dynamic programme over the remaining Kraft budget (units of 2^-max_len)."""
    w = [int(c) for c in counts if c]
    full = 1 << max_len
    INF = float("inf")
    best = [0] * (full + 1)                    # no symbols left: cost 0 whatever remains
    for wi in reversed(w):
        nxt = [INF] * (full + 1)
        for budget in range(full + 1):
            for l in range(1, max_len + 1):
                use = 1 << (max_len - l)
                if use <= budget and best[budget - use] + wi * l < nxt[budget]:
                    nxt[budget] = best[budget - use] + wi * l
        best = nxt
    return best[full]


def test_binding_limit_matches_the_dynamic_programme():
    fib = [1, 1, 2, 3, 5, 8, 13, 21, 34, 55, 89, 144, 233, 377]
    rng = np.random.default_rng(3)
    cases = [(fib, 5), (fib, 6), (fib, 8), (fib[:9], 4), ([1, 1, 1, 1, 100, 1000, 10000], 3),
             ([1] * 16, 4), ([7] * 11, 4), ([7] * 11, 5)]
    for _ in range(10):
        n = int(rng.integers(5, 17))
        cases.append(((2.0 ** rng.uniform(0, 18, size=n)).astype(np.int64) + 1, int(rng.integers(4, 8))))
    for counts, max_len in cases:
        counts = np.asarray(counts)
        if len(counts) > (1 << max_len):
            continue
        L = oracle.huffman_lengths(counts, max_len=max_len)
        assert L.max() <= max_len
        assert cost(counts, L) == dp_limited_cost(counts, max_len), (counts, max_len, L)
        # the limit really binds in the Fibonacci cases
    assert oracle.huffman_lengths(np.asarray(fib), max_len=32).max() == len(fib) - 1
    assert cost(fib, oracle.huffman_lengths(np.asarray(fib), max_len=5)) > heap_huffman_cost(fib)


def test_optimal_codes_are_complete_and_monotone():
    rng = np.random.default_rng(4)
    for trial in range(40):
        n = int(rng.integers(2, 300))
        counts = rng.integers(1, 10 ** 6, size=n)
        L = oracle.huffman_lengths(counts, max_len=12)
        assert kraft(L, 12) == 1 << 12                       # no unused word
        # a heavier symbol never has the longer word: the cost equals the cheapest pairing
        # of these lengths with these counts
        assert cost(counts, L) == cost(np.sort(counts)[::-1], np.sort(L))


def test_degenerate_alphabets():
    assert oracle.huffman_lengths(np.array([0, 0, 0])).tolist() == [0, 0, 0]
    assert oracle.huffman_lengths(np.array([0, 17, 0])).tolist() == [0, 1, 0]
    assert oracle.huffman_lengths(np.array([5, 0, 5])).tolist() == [1, 0, 1]
    with pytest.raises(ValueError):
        oracle.huffman_lengths(np.ones(9, dtype=np.int64), max_len=3)
    assert oracle.huffman_lengths(np.ones(8, dtype=np.int64), max_len=3).tolist() == [3] * 8
    big = np.array([2 ** 40, 1, 2 ** 39, 3], dtype=np.uint64)   # counts beyond 32 bits
    assert oracle.huffman_lengths(big).tolist() == [1, 3, 2, 3]


# --------------------------------------------------------------- the words ---
def test_canonical_words_are_prefix_free_and_ordered():
    rng = np.random.default_rng(5)
    for trial in range(30):
        n = int(rng.integers(2, 40))
        counts = rng.integers(0, 3, size=n) * rng.integers(1, 1000, size=n)
        if np.count_nonzero(counts) < 2:
            counts[-2:] = (1, 2)
        L = oracle.huffman_lengths(counts, max_len=10)
        W = oracle.huffman_words(L)
        present = [k for k in range(n) if L[k]]
        bits = {k: format(int(W[k]), "0%db" % L[k]) for k in present}
        for a in present:
            for b in present:
                if a != b:
                    assert not bits[b].startswith(bits[a])
        order = sorted(present, key=lambda k: (L[k], k))
        assert int(W[order[0]]) == 0
        vals = [bits[k].ljust(10, "0") for k in order]      # left-aligned words increase
        assert vals == sorted(vals) and len(set(vals)) == len(vals)
    # lengths 1, 2, 3, 3 -> 0, 10, 110, 111
    assert oracle.huffman_words(np.array([2, 1, 3, 3])).tolist() == [0b10, 0b0, 0b110, 0b111]
    with pytest.raises(ValueError):                          # Kraft sum above one
        oracle.huffman_words(np.array([1, 1, 2]))


# -------------------------------------------------------------- the stream ---
def pack(symbols, r):
    words = np.zeros((len(symbols) * r + 31) // 32, dtype=np.uint32)
    for i, c in enumerate(symbols):
        for k in range(r):
            if (int(c) >> k) & 1:
                words[(i * r + k) >> 5] |= np.uint32(1 << ((i * r + k) & 31))
    return words


def test_hand_packed_stream():
    # s = 1: symbols 0, 1, 2 (levels -1, 0, +1), r = 2.  Lengths (2, 1, 2) give the words
    # 1 -> "0", 0 -> "10", 2 -> "11".  The message 1 0 2 1 1 2 0 is sent as
    # 0 10 11 0 0 11 10, first bit in bit 0 of the word:
    # bits 1, 3, 4, 7, 8, 9 are set -> 2 + 8 + 16 + 128 + 256 + 512 = 922.
    L = np.array([2, 1, 2], dtype=np.uint8)
    stream, offsets, quarters = oracle.huffman_encode(pack([1, 0, 2, 1, 1, 2, 0], 2), L, n=7, s=1)
    assert stream.tolist() == [922] and offsets.tolist() == [0, 1]
    assert quarters.tolist() == [11, 11, 11]          # no entry 256, 512, 768: the chunk's end


def test_chunks_start_on_word_boundaries():
    # 1024 one-bit words fill exactly 32 stream words; the next chunk starts at word 32
    # even when the first does not end on a boundary
    L = np.array([2, 1, 2], dtype=np.uint8)
    msg = [1] * 1024 + [2]
    stream, offsets, quarters = oracle.huffman_encode(pack(msg, 2), L, n=1025, s=1)
    assert offsets.tolist() == [0, 32, 33] and stream[:32].tolist() == [0] * 32 and stream[32] == 3
    # one bit per entry in chunk 0: its quarters start at bits 256, 512, 768; chunk 1 has
    # one entry of two bits and no further quarter
    assert quarters.tolist() == [256, 512, 768, 2, 2, 2]
    msg = [1] * 1023 + [0] + [2, 1, 0]
    stream, offsets, quarters = oracle.huffman_encode(pack(msg, 2), L, n=1027, s=1)
    # chunk 0: 1023 zeros then "10" = 1025 bits -> 33 words, bit 1023 set; chunk 1: 11 0 10
    assert offsets.tolist() == [0, 33, 34]
    assert stream[31] == 1 << 31 and stream[32] == 0 and stream[33] == 0b01011
    assert quarters.tolist() == [256, 512, 768, 5, 5, 5]
    # two-bit words in the second quarter shift the later marks
    msg = [1] * 256 + [0] * 256 + [1] * 300
    _, _, quarters = oracle.huffman_encode(pack(msg, 2), L, n=812, s=1)
    assert quarters.tolist() == [256, 768, 1024]


@pytest.mark.parametrize("s", [1, 2, 4, 8, 128, 300, 2047])
def test_round_trip_and_length(s):
    rng = np.random.default_rng(s)
    r = oracle.code_bits(s)
    for n in (1, 31, 1024, 1025, 5000, 3 * 1024 + 77):
        # levels concentrated around zero like a quantised gradient
        q = np.clip(np.rint(rng.standard_normal(n) * max(s / 3.0, 0.6)), -s, s).astype(np.int64)
        sym = (q + s).astype(np.uint32)
        codes = pack(sym, r) if n <= 5000 and r <= 5 else None
        if codes is None:
            bits = ((sym[:, None] >> np.arange(r)) & 1).astype(np.uint8).reshape(-1)
            bits = np.concatenate([bits, np.zeros(-bits.size % 32, np.uint8)])
            codes = (bits.reshape(-1, 32).astype(np.uint64) << np.arange(32, dtype=np.uint64)).sum(axis=1).astype(np.uint32)
        counts = oracle.code_histogram(codes, n=n, s=s)
        assert counts.sum() == n and np.array_equal(counts, np.bincount(sym, minlength=2 * s + 1))
        L = oracle.huffman_lengths(counts, max_len=12)
        stream, offsets, quarters = oracle.huffman_encode(codes, L, n=n, s=s)
        n_chunks = -(-n // 1024)
        # a quarter mark is the number of bits the entries before it take
        for c in range(n_chunks):
            lens = L[sym[c * 1024:(c + 1) * 1024]].astype(np.int64)
            cum = np.concatenate([[0], np.cumsum(lens)])
            want = [int(cum[min(256 * (j + 1), lens.size)]) for j in range(3)]
            assert quarters[3 * c:3 * c + 3].tolist() == want
        assert offsets.size == n_chunks + 1 and offsets[0] == 0 and offsets[-1] == stream.size
        # every chunk takes exactly the words its symbols need
        for c in range(n_chunks):
            bits_c = int(L[sym[c * 1024:(c + 1) * 1024]].astype(np.int64).sum())
            assert offsets[c + 1] - offsets[c] == -(-bits_c // 32)
        back = oracle.huffman_decode(stream, offsets, quarters, L, n=n, s=s)
        assert np.array_equal(back, codes)
        if n > 256 and np.count_nonzero(counts) > 1:
            # the quarters are really entered at their marks: a wrong mark breaks the decode
            wrong = quarters.copy()
            wrong[0] += 1
            try:
                assert not np.array_equal(oracle.huffman_decode(stream, offsets, wrong, L, n=n, s=s), codes)
            except ValueError:
                pass
        # Huffman: within one bit per symbol of the entropy bound, never below it
        payload = cost(counts, L)
        H = oracle.entropy_bound_bits(counts)
        if np.count_nonzero(counts) > 1:
            assert H - 1e-6 <= payload < H + n


def test_encode_refusals():
    L = np.array([2, 1, 2], dtype=np.uint8)
    codes = pack([1, 0, 2, 1], 2)
    with pytest.raises(OverflowError):
        oracle.huffman_encode(pack([0] * 40, 2), L, n=40, s=1, capacity=2)
    with pytest.raises(ValueError):          # symbol 2 has no word
        oracle.huffman_encode(codes, np.array([1, 1, 0], dtype=np.uint8), n=4, s=1)
    with pytest.raises(ValueError):          # r = 2 can spell 3, which is no level
        oracle.huffman_encode(pack([3], 2), L, n=1, s=1)
