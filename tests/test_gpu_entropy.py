"""GPU parity of the entropy-coded message (paragraph after Eq. 9): the CUDA Huffman coder,
called through the C ABI, against the CPU oracle -- stream words, chunk offsets and the
decoded codes bit for bit; the library's own code lengths by their cost."""
import numpy as np
import pytest
import torch

import oracle
import paper_1806_08054_b200 as ecq
from paper_1806_08054_b200 import workloads as wl

pytestmark = pytest.mark.gpu
SEED = wl.CODEC_SEED
GUARD = 0x5A5A5A5A


def u32(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint32)


def kraft(lengths, max_len=12):
    return sum(1 << (max_len - int(l)) for l in lengths if l)


def cost(counts, lengths):
    return int(sum(int(c) * int(l) for c, l in zip(counts, lengths)))


class Message:
    """One worker's codes on the device (made by the encode kernel) plus their host copy."""

    def __init__(self, d, bucket, s, scale=0.01, seed=0, grad=None):
        self.d, self.s = d, s
        self.ctx = ecq.ecq_create(d, bucket, s, 1.0, 0.9, SEED)
        nw, nb = ecq.ecq_codes_words(self.ctx), ecq.ecq_num_buckets(self.ctx)
        if grad is None:
            gen = torch.Generator(device="cuda")
            gen.manual_seed(seed)
            grad = scale * torch.randn(d, generator=gen, device="cuda")
        self.codes = torch.zeros(nw, dtype=torch.int32, device="cuda")
        self.scales = torch.zeros(nb, device="cuda")
        err = torch.zeros(d, device="cuda")
        ecq.ecq_encode(self.ctx, 0, 0, grad, err, self.codes, self.scales)
        assert ecq.ecq_status(self.ctx) == ecq.ECQ_OK
        self.codes_np = u32(self.codes)
        self.counts = oracle.code_histogram(self.codes_np, n=d, s=s)
        self.n_chunks = ecq.ecq_huffman_chunks(self.ctx)
        self.tables = torch.zeros(ecq.ECQ_HUFFMAN_TABLE_BYTES, dtype=torch.uint8, device="cuda")

    def gpu_encode(self, lengths, capacity=None):
        ecq.ecq_huffman_tables(self.ctx, lengths, self.tables)
        cap = capacity if capacity is not None else ecq.ecq_huffman_stream_bound(self.ctx, self.counts, lengths)
        pad = 8
        buf = torch.full((cap + 2 * pad,), GUARD, dtype=torch.int32, device="cuda")
        offs = torch.full((self.n_chunks + 1 + 2 * pad,), GUARD, dtype=torch.int32, device="cuda")
        qts = torch.full((3 * self.n_chunks + 2 * pad,), 0x5A5A, dtype=torch.int16, device="cuda")
        ecq.ecq_huffman_encode(self.ctx, self.tables, self.codes, buf[pad:pad + cap],
                               offs[pad:pad + self.n_chunks + 1], qts[pad:pad + 3 * self.n_chunks])
        st = ecq.ecq_status(self.ctx)
        b, o, q = u32(buf), u32(offs), qts.cpu().numpy()
        assert np.all(b[:pad] == GUARD) and np.all(b[pad + cap:] == GUARD), "write outside the stream"
        assert np.all(o[:pad] == GUARD) and np.all(o[pad + self.n_chunks + 1:] == GUARD)
        assert np.all(q[:pad] == 0x5A5A) and np.all(q[pad + 3 * self.n_chunks:] == 0x5A5A)
        self.quarters = qts[pad:pad + 3 * self.n_chunks]
        return st, buf[pad:pad + cap], offs[pad:pad + self.n_chunks + 1]

    def gpu_decode(self, stream, offsets, quarters=None):
        nw = self.codes.numel()
        pad = 8
        out = torch.full((nw + 2 * pad,), GUARD, dtype=torch.int32, device="cuda")
        # 16-byte aligned view: pad is 8 words
        ecq.ecq_huffman_decode(self.ctx, self.tables, stream, offsets,
                               self.quarters if quarters is None else quarters, out[pad:pad + nw])
        st = ecq.ecq_status(self.ctx)
        o = u32(out)
        assert np.all(o[:pad] == GUARD) and np.all(o[pad + nw:] == GUARD), "write outside the codes"
        return st, o[pad:pad + nw]

    def close(self):
        ecq.ecq_destroy(self.ctx)


def check_against_oracle(m: Message):
    # the library's lengths: a prefix code within the limit and as cheap as the oracle's
    L_or = oracle.huffman_lengths(m.counts, max_len=12)
    L_lib = np.array(ecq.ecq_huffman_lengths(m.ctx, m.counts), dtype=np.uint8)
    assert L_lib.max() <= 12 and np.all((L_lib == 0) == (m.counts == 0))
    assert kraft(L_lib) <= 1 << 12
    assert cost(m.counts, L_lib) == cost(m.counts, L_or)
    for L in (L_or, L_lib):
        s_or, o_or, q_or = oracle.huffman_encode(m.codes_np, L, n=m.d, s=m.s)
        st, stream, offs = m.gpu_encode(L)
        assert st == ecq.ECQ_OK
        assert np.array_equal(u32(offs), o_or), "chunk offsets differ"
        assert np.array_equal(m.quarters.cpu().numpy().view(np.uint16), q_or), "quarter marks differ"
        assert np.array_equal(u32(stream)[:s_or.size], s_or), "stream differs"
        assert s_or.size <= stream.numel()
        st, back = m.gpu_decode(stream, offs)
        assert st == ecq.ECQ_OK
        assert np.array_equal(back, m.codes_np), "decoded codes differ"
        # and the oracle's decoder reads the GPU's stream
        assert np.array_equal(oracle.huffman_decode(u32(stream)[:s_or.size], u32(offs),
                                                    m.quarters.cpu().numpy().view(np.uint16), L, n=m.d, s=m.s),
                              m.codes_np)


@pytest.mark.parametrize("s", [1, 2, 4, 8, 128, 300, 2047])
@pytest.mark.parametrize("d", [1, 31, 1000, 1024, 1025, 4096 * 3 + 5 * 32 + 7, 300000])
def test_streams_offsets_and_round_trip(s, d):
    if d == 300000 and s not in (1, 4, 128):
        pytest.skip("one large case per width class")
    m = Message(d, 512, s, seed=d + s)
    try:
        check_against_oracle(m)
    finally:
        m.close()


def test_skewed_and_flat_level_distributions():
    d = 4096 * 5 + 100
    gen = torch.Generator(device="cuda")
    gen.manual_seed(9)
    # one huge entry per bucket: almost every level is 0 (long words for the rest)
    g = 1e-4 * torch.randn(d, generator=gen, device="cuda")
    g[::512] = 1.0
    # uniform values: all levels about equally likely
    u = torch.rand(d, generator=gen, device="cuda") * 2 - 1
    for grad, s in ((g, 128), (g, 4), (u, 8), (u, 300)):
        m = Message(d, 512, s, grad=grad)
        try:
            check_against_oracle(m)
        finally:
            m.close()


def test_single_level_message():
    # an all-zero gradient: every code is s, one 1-bit word
    d = 3000
    m = Message(d, 512, 4, grad=torch.zeros(d, device="cuda"))
    try:
        assert np.count_nonzero(m.counts) == 1
        check_against_oracle(m)
        L = ecq.ecq_huffman_lengths(m.ctx, m.counts)
        assert L[4] == 1 and sum(L) == 1
    finally:
        m.close()


def test_stream_that_does_not_fit_is_refused_and_nothing_written():
    m = Message(4096 * 4 + 40, 512, 4, seed=3)
    try:
        L = oracle.huffman_lengths(m.counts, max_len=12)
        need = oracle.huffman_encode(m.codes_np, L, n=m.d, s=m.s)[0].size
        st, stream, offs = m.gpu_encode(L, capacity=need - 1)
        assert st == ecq.ECQ_ERR_CAPACITY
        assert np.all(u32(stream) == GUARD), "stream touched although it does not fit"
        assert u32(offs)[-1] == 0xFFFFFFFF
        st, stream, offs = m.gpu_encode(L, capacity=need)          # exactly enough
        assert st == ecq.ECQ_OK and u32(offs)[-1] == need
    finally:
        m.close()


def test_level_without_a_word_is_flagged():
    m = Message(4096 + 77, 512, 4, seed=4)
    try:
        L = oracle.huffman_lengths(m.counts, max_len=12).copy()
        k = int(np.argmax(m.counts))
        # a code that lacks the most frequent level (still a prefix code)
        L[k] = 0
        st, _, _ = m.gpu_encode(L, capacity=m.d)
        assert st == ecq.ECQ_ERR_SYMBOL
    finally:
        m.close()


def test_pattern_that_is_no_word_is_flagged_by_the_decoder():
    m = Message(2048, 512, 1, seed=5)
    try:
        # an incomplete code: lengths 2, 2, 2 leave the pattern "11" unused
        L = [2, 2, 2]
        st, stream, offs = m.gpu_encode(L)
        assert st == ecq.ECQ_OK
        st, back = m.gpu_decode(stream, offs)
        assert st == ecq.ECQ_OK and np.array_equal(back, m.codes_np)
        bad = stream.clone()
        bad[0] = -1                                   # all ones: "11" comes first
        st, _ = m.gpu_decode(bad, offs)
        assert st == ecq.ECQ_ERR_SYMBOL
    finally:
        m.close()


def test_argument_errors():
    m = Message(1024, 512, 4)
    try:
        with pytest.raises(ecq.EcqError):             # Kraft sum above one
            ecq.ecq_huffman_tables(m.ctx, [1, 1, 1, 0, 0, 0, 0, 0, 0], m.tables)
        with pytest.raises(ecq.EcqError):             # a word longer than the limit
            ecq.ecq_huffman_tables(m.ctx, [13, 1, 0, 0, 0, 0, 0, 0, 0], m.tables)
        L = ecq.binding.lib()
        assert L.ecq_huffman_encode(m.ctx, None, None, None, 0, None, None, None) == ecq.ECQ_ERR_ARG
        assert L.ecq_huffman_decode(m.ctx, None, None, 0, None, None, None, None) == ecq.ECQ_ERR_ARG
    finally:
        m.close()
    big = ecq.ecq_create(1024, 512, 2048, 1.0, 0.9, 1)      # 4097 levels: beyond the coder
    try:
        with pytest.raises(ecq.EcqError):
            ecq.ecq_huffman_lengths(big, [1] * 4097)
    finally:
        ecq.ecq_destroy(big)


def test_resnet50_sized_message_bits_per_entry():
    w = wl.WORKLOADS["resnet50"]
    grad = wl.gradient(w, 0, 0, "cuda")
    m = Message(w.d, w.bucket, w.s, grad=grad)
    try:
        check_against_oracle(m)
        L = ecq.ecq_huffman_lengths(m.ctx, m.counts)
        payload = cost(m.counts, L)
        H = oracle.entropy_bound_bits(m.counts)
        # Huffman's guarantee, and far below the fixed-width r bits per entry
        assert H <= payload < H + w.d
        assert payload < 0.8 * w.d * ecq.ecq_code_bits(m.ctx)
    finally:
        m.close()


def test_lm_350m_sized_message_on_sampled_chunks():
    # full benchmark size: the oracle codes sampled runs of chunks (a chunk's stream depends
    # only on its own entries); offsets and quarter marks are checked there, the round trip
    # over the whole message on the device
    w = wl.WORKLOADS["lm_350m"]
    free, _ = torch.cuda.mem_get_info()
    if free < 12 * w.d:
        pytest.skip("needs %.0f GB of free device memory" % (12 * w.d / 1e9))
    ctx = ecq.ecq_create(w.d, w.bucket, w.s, 1.0, 0.9, SEED)
    try:
        r = ecq.ecq_code_bits(ctx)
        grad = wl.gradient(w, 0, 0, "cuda")
        err = torch.zeros(w.d, device="cuda")
        codes = torch.zeros(ecq.ecq_codes_words(ctx), dtype=torch.int32, device="cuda")
        scales = torch.zeros(ecq.ecq_num_buckets(ctx), device="cuda")
        ecq.ecq_encode(ctx, 0, 0, grad, err, codes, scales)
        del grad, err
        counts_dev = torch.zeros(2 * w.s + 1, dtype=torch.int64, device="cuda")
        ecq.ecq_code_histogram(ctx, codes, counts_dev)
        counts = counts_dev.cpu().numpy().astype(np.uint64)
        assert int(counts.sum()) == w.d
        L = oracle.huffman_lengths(counts, max_len=12)
        n_chunks = ecq.ecq_huffman_chunks(ctx)
        cap = ecq.ecq_huffman_stream_bound(ctx, counts, L)
        tables = torch.zeros(ecq.ECQ_HUFFMAN_TABLE_BYTES, dtype=torch.uint8, device="cuda")
        stream = torch.zeros(cap, dtype=torch.int32, device="cuda")
        offsets = torch.zeros(n_chunks + 1, dtype=torch.int32, device="cuda")
        quarters = torch.zeros(3 * n_chunks, dtype=torch.int16, device="cuda")
        ecq.ecq_huffman_tables(ctx, L, tables)
        ecq.ecq_huffman_encode(ctx, tables, codes, stream, offsets, quarters)
        assert ecq.ecq_status(ctx) == ecq.ECQ_OK
        off = u32(offsets).astype(np.int64)
        assert off[0] == 0 and np.all(np.diff(off) >= 0) and off[-1] <= cap
        # the whole stream is as long as the counts say, up to the padding of each chunk
        payload = cost(counts, L)
        assert payload <= 32 * off[-1] < payload + 32 * n_chunks
        rng = np.random.default_rng(7)
        starts = [0, n_chunks - 40] + [int(x) for x in rng.integers(0, n_chunks - 40, size=4)]
        for c0 in starts:
            c1 = min(c0 + 40, n_chunks)
            lo, hi = c0 * 1024, min(c1 * 1024, w.d)
            piece = u32(codes[c0 * 32 * r: -(-hi * r // 32)])
            s_or, o_or, q_or = oracle.huffman_encode(piece, L, n=hi - lo, s=w.s)
            assert np.array_equal(off[c0:c1 + 1] - off[c0], o_or.astype(np.int64))
            assert np.array_equal(u32(stream[off[c0]:off[c1]]), s_or)
            assert np.array_equal(quarters[3 * c0:3 * c1].cpu().numpy().view(np.uint16), q_or)
        back = torch.zeros_like(codes)
        ecq.ecq_huffman_decode(ctx, tables, stream, offsets, quarters, back)
        assert ecq.ecq_status(ctx) == ecq.ECQ_OK
        assert torch.equal(back, codes)
    finally:
        ecq.ecq_destroy(ctx)
        wl.clear_cache()
        torch.cuda.empty_cache()
