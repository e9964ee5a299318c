"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests re-types the oracle's formulas: they use published
known-answer vectors, hand-worked encodings, exact rational arithmetic, brute
force over all rounding patterns, statistical laws (Lemma 1), identities
between the paper's equations (Eq. 5 vs Eq. 6, the recursion in the proof of
Lemma 2), and library routines for the pieces that have one.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return [ln.strip() for ln in f if ln.strip() and not ln.startswith("#")]


def np_unpack(codes, n, r):
    """Independent unpacking: little-endian bit stream, r bits per entry."""
    bits = np.unpackbits(np.ascontiguousarray(codes).view(np.uint8), bitorder="little")
    bits = bits[: n * r].reshape(n, r).astype(np.int64)
    return (bits << np.arange(r)).sum(axis=1)


def enc(g, h, **kw):
    kw.setdefault("seed", 1234)
    kw.setdefault("worker", 0)
    kw.setdefault("step", 0)
    kw.setdefault("alpha", 1.0)
    kw.setdefault("beta", 0.9)
    return oracle.encode(g, h, **kw)


# ---------------------------------------------------------------- Philox -----
def test_philox_known_answers():
    for row in _rows("philox4x32_10_kat.txt"):
        w = [int(x, 16) for x in row.split()]
        out = oracle.philox4x32_10(w[0:4], w[4:6])
        assert [int(x) for x in out] == w[6:10]


def test_draw_word_counter_layout():
    # counter = (lo32(i/4), hi32(i/4), worker, step), key = (lo32 seed, hi32 seed)
    seed = 0x0123456789ABCDEF
    for i in (0, 1, 2, 3, 4, 7, 1 << 20, (1 << 34) + 5, (1 << 40) + 2):
        blk = i >> 2
        ref = oracle.philox4x32_10([blk & 0xFFFFFFFF, blk >> 32, 7, 11],
                                   [seed & 0xFFFFFFFF, seed >> 32])
        assert oracle.draw_word(seed, 7, 11, i) == int(ref[i & 3])


# ----------------------------------------------------------- closed forms ----
def test_code_width_closed_form():
    # r = ceil(log2(2s+1)), evaluated in exact integer arithmetic
    for s in list(range(1, 300)) + [511, 512, 16383, 16384, 32767]:
        r = (2 * s).bit_length()  # smallest r with 2^r >= 2s+1
        assert 2 ** r >= 2 * s + 1 > 2 ** (r - 1)
        assert oracle.code_bits(s) == r
    assert [oracle.code_bits(s) for s in (1, 2, 4, 8, 128)] == [2, 3, 4, 5, 9]


def test_message_length_closed_form():
    # 32 + d*r bits per scaled vector, applied per bucket (whole words per bucket)
    for d, B, s in ((1 << 20, 512, 4), (25_557_032, 512, 8), (61_100_840, 2048, 1),
                    (1000, 128, 2), (33, 32, 128)):
        r = oracle.code_bits(s)
        nb = -(-d // B)
        assert oracle.num_buckets(d, B) == nb
        assert oracle.codes_words(d, s) == -(-d * r // 32)
        bits = 32 * nb + 32 * oracle.codes_words(d, s)
        assert 0 <= bits - (32 * nb + d * r) < 32


# ------------------------------------------------ hand-worked level cases ----
def test_level_boundary_golden():
    for row in _rows("level_boundary_cases.txt"):
        s, B, vals, scale, levels, word = [x.strip() for x in row.split("|")]
        s, B = int(s), int(B)
        g = np.zeros(B, np.float32)
        vv = [float(x) for x in vals.split(",")]
        g[: len(vv)] = vv
        h = np.zeros(B, np.float32)
        for seed in (0, 1, 99):      # deterministic whatever the draws
            hh = h.copy()
            codes, scales, st = enc(g, hh, bucket=B, s=s, seed=seed)
            assert st == 0 and scales[0] == np.float32(scale)
            q = oracle.unpack_levels(codes, n=B, s=s)
            assert list(q[: len(vv)]) == [int(x) for x in levels.split(",")]
            assert np.all(q[len(vv):] == 0)
            assert int(codes[0]) == int(word, 16)
            # exact dequantisation => the accumulator stays 0 (Eq. 6)
            assert np.all(hh == 0)


# ---------------------------------------------- the two-point rounding law ---
def test_round_up_threshold_exact():
    # Eq. 9: up with probability f = s|v|/||v|| - l.  With a 24-bit uniform
    # U/2^24 and the strict test U/2^24 < f, exactly ceil(f*2^24) of the 2^24
    # draws go up.  f is evaluated in exact rational arithmetic here.
    rng = np.random.default_rng(5)
    for s in (1, 4, 8, 128):
        B = 32
        g = np.zeros(B, np.float32)
        g[0] = 1.0                                  # the scale
        g[1:9] = rng.uniform(0.01, 0.99, 8).astype(np.float32)
        g[9] = np.float32(3e-9)                     # f below 2^-24 resolution
        inv = np.float32(s) / np.float32(1.0)
        for i in range(1, 10):
            x = Fraction(float(np.float32(abs(g[i])) * inv))   # fp32 product, as specified
            assert float(x) == float(np.float32(g[i]) * inv)
            l = math.floor(x)
            f = x - l
            thr = math.ceil(f * (1 << 24))          # number of U values that go up
            for U in {0, max(thr - 1, 0), thr, min(thr + 1, (1 << 24) - 1), (1 << 24) - 1}:
                draws = np.zeros(B, np.uint32)
                draws[i] = (U << 8) | 0xA5          # low 8 bits must not matter
                codes, scales, _ = enc(g, np.zeros(B, np.float32), bucket=B, s=s, draws=draws)
                q = oracle.unpack_levels(codes, n=B, s=s)
                assert q[i] == l + (1 if U < thr else 0), (s, i, U, thr)


def test_bruteforce_expectation_d8():
    # All 2^8 up/down patterns of 8 entries, each forced through chosen draws;
    # their probabilities come from exact fractional parts.  The expectation of
    # the dequantised vector must be the input (Lemma 1, unbiasedness), and each
    # entry takes exactly the two neighbouring levels of Eq. 9.
    rng = np.random.default_rng(11)
    for s in (1, 2, 4):
        B = 32
        g = np.zeros(B, np.float32)
        g[:8] = (rng.uniform(0.05, 0.95, 8) * rng.choice([-1, 1], 8)).astype(np.float32)
        g[8] = 1.0
        fr = []
        for i in range(8):
            x = Fraction(float(np.float32(abs(g[i])) * np.float32(s)))
            fr.append((math.floor(x), x - math.floor(x)))
        expect = [Fraction(0)] * 8
        total = Fraction(0)
        for pat in range(256):
            draws = np.full(B, 0xFFFFFFFF, np.uint32)
            p = Fraction(1)
            for i in range(8):
                up = (pat >> i) & 1
                draws[i] = 0 if up else 0xFFFFFFFF
                p *= fr[i][1] if up else 1 - fr[i][1]
            codes, scales, _ = enc(g, np.zeros(B, np.float32), bucket=B, s=s, draws=draws)
            q = oracle.unpack_levels(codes, n=B, s=s)
            for i in range(8):
                up = (pat >> i) & 1
                assert abs(int(q[i])) == fr[i][0] + up
                assert q[i] * g[i] > 0 or q[i] == 0
                expect[i] += p * Fraction(int(q[i]), s) * Fraction(float(scales[0]))
            total += p
        assert total == 1
        for i in range(8):
            assert abs(float(expect[i]) - float(g[i])) < 1e-12


def test_philox_driven_frequencies_follow_eq9():
    # Chi-square of observed up-counts over many (seed, step) against f.
    s, B, n = 4, 32, 32
    rng = np.random.default_rng(3)
    g = rng.uniform(-1, 1, n).astype(np.float32)
    g[0] = 1.0
    N = 4000
    ups = np.zeros(n)
    x = np.abs(g.astype(np.float64)) * s
    l = np.floor(x)
    f = x - l
    for k in range(N):
        codes, _, _ = enc(g, np.zeros(n, np.float32), bucket=B, s=s, seed=1000 + k // 40, step=k % 40)
        q = np.abs(oracle.unpack_levels(codes, n=n, s=s))
        assert np.all((q == l) | (q == l + 1))
        ups += (q == l + 1)
    var = N * f * (1 - f)
    ok = var > 0
    chi2 = (((ups - N * f) ** 2)[ok] / var[ok]).sum()
    dof = ok.sum()
    assert chi2 < dof + 5 * math.sqrt(2 * dof)
    assert np.all(ups[~ok] == 0) or np.all(f[~ok] == 0)


# ------------------------------------------------------------ invariants -----
@pytest.mark.parametrize("s,B", [(1, 128), (4, 512), (8, 512), (128, 4096), (3, 96), (127, 32)])
def test_range_step_sign_and_max(s, B):
    rng = np.random.default_rng(s * 1000 + B)
    n = 5 * B + 40
    g = (rng.standard_normal(n) * 0.01).astype(np.float32)
    h = (rng.standard_normal(n) * 0.003).astype(np.float32)
    alpha = 0.7
    v = np.float32(alpha) * h.astype(np.float64) + g            # exact product+sum in fp64
    hh = h.copy()
    codes, scales, st = enc(g, hh, bucket=B, s=s, alpha=alpha)
    r = oracle.code_bits(s)
    c = np_unpack(codes, n, r)
    assert st == 0 and c.min() >= 0 and c.max() <= 2 * s         # code range
    q = c - s
    assert np.array_equal(q, oracle.unpack_levels(codes, n=n, s=s))   # independent unpack
    nb = -(-n // B)
    for b in range(nb):
        sl = slice(b * B, min((b + 1) * B, n))
        vb = np.float32(v[sl])                                    # fma rounds once
        # library max-abs
        assert scales[b] == torch.amax(torch.abs(torch.from_numpy(vb))).item()
        a = float(scales[b]) / s
        gq = q[sl] * a
        assert np.all(np.abs(gq - vb) <= a * (1 + 2.0 ** -20))    # within one level step
        assert np.all(q[sl] * vb >= 0)                             # sign
        top = np.abs(vb) == scales[b]
        assert np.all(np.abs(q[sl][top]) == s)                     # the max gets level s


def test_alpha_beta_zero_is_plain_quantisation():
    # alpha = 0 is QSGD-style quantisation of g itself (Section 5.2 remark):
    # codes do not depend on h, and with beta = 0 the accumulator is g - g~.
    rng = np.random.default_rng(2)
    n, B, s = 1000, 128, 4
    g = rng.standard_normal(n).astype(np.float32)
    h1 = np.zeros(n, np.float32)
    h2 = rng.standard_normal(n).astype(np.float32)
    c1, s1, _ = enc(g, h1, bucket=B, s=s, alpha=0.0, beta=0.0)
    c2, s2, _ = enc(g, h2, bucket=B, s=s, alpha=0.0, beta=0.0)
    assert np.array_equal(c1, c2) and np.array_equal(s1, s2)
    q = oracle.unpack_levels(c1, n=n, s=s)
    gq = q * np.repeat(s1.astype(np.float64) / s, B)[:n]
    assert np.allclose(h1, g - gq, rtol=0, atol=1e-6)
    assert np.array_equal(h1, h2)


def test_unbiasedness_lemma1():
    s, B, n, N = 4, 64, 64, 3000
    rng = np.random.default_rng(8)
    g = (rng.standard_normal(n) * 0.01).astype(np.float32)
    acc = np.zeros(n)
    acc2 = np.zeros(n)
    for k in range(N):
        codes, scales, _ = enc(g, np.zeros(n, np.float32), bucket=B, s=s, seed=k, step=k % 7, worker=k % 3)
        gq = oracle.unpack_levels(codes, n=n, s=s) * (float(scales[0]) / s)
        acc += gq
        acc2 += gq * gq
    a = float(scales[0]) / s
    mean = acc / N
    assert np.all(np.abs(mean - g) <= 5 * a / (2 * math.sqrt(N)))
    x = np.abs(g.astype(np.float64)) / a
    f = x - np.floor(x)
    var_exact = (a * a * f * (1 - f)).sum()
    var_emp = (acc2 / N - mean ** 2).sum()
    assert abs(var_emp - var_exact) < 0.1 * var_exact


def _run_steps(T, n, B, s, alpha, beta, mode, seed=4):
    rng = np.random.default_rng(seed)
    gs = [(rng.standard_normal(n) * 0.01).astype(np.float32) for _ in range(T)]
    h = np.zeros(n, np.float32)
    hs, gqs, vs = [h.copy()], [], []
    for t in range(T):
        vs.append(np.float32(alpha) * hs[-1].astype(np.float64) + gs[t])
        codes, scales, _ = enc(gs[t], h, bucket=B, s=s, alpha=alpha, beta=beta, step=t, mode=mode)
        q = oracle.unpack_levels(codes, n=n, s=s)
        gqs.append(q * np.repeat(scales.astype(np.float64) / s, B)[:n])
        hs.append(h.copy())
    return gs, hs, gqs, vs


def test_eq5_equals_eq6():
    # closed form h(T) = sum_t beta^(T-1-t) (g(t) - g~(t)) vs the incremental update
    T, n, B, s, alpha, beta = 12, 700, 128, 4, 0.5, 0.9
    gs, hs, gqs, _ = _run_steps(T, n, B, s, alpha, beta, mode=0)
    direct = sum(beta_pow * (gs[t] - gqs[t]) for t, beta_pow in
                 ((t, float(np.float32(beta)) ** (T - 1 - t)) for t in range(T)))
    assert np.allclose(hs[T], direct, rtol=1e-5, atol=1e-7)
    assert np.all(hs[0] == 0)


def test_recursion_of_lemma2_proof_selects_the_raw_gradient_form():
    # h(t+1) = (beta - alpha) h(t) - eps(t), eps = g~ - (g + alpha h): holds for
    # the paper's Eq. 6 (mode 0); the variant that books the compensated value
    # (mode 1) satisfies h(t+1) = beta h(t) - eps(t) instead.
    T, n, B, s, alpha, beta = 6, 500, 128, 8, 0.3, 0.9
    b32, a32 = float(np.float32(beta)), float(np.float32(alpha))
    for mode, coef in ((0, b32 - a32), (1, b32)):
        gs, hs, gqs, vs = _run_steps(T, n, B, s, alpha, beta, mode=mode)
        for t in range(T):
            eps = gqs[t] - vs[t]
            assert np.allclose(hs[t + 1], coef * hs[t] - eps, rtol=1e-5, atol=2e-8)
        if mode == 0:   # and the other form must NOT hold
            eps = gqs[T - 1] - vs[T - 1]
            assert not np.allclose(hs[T], b32 * hs[T - 1] - eps, rtol=1e-5, atol=2e-8)


def test_conservation_beta_one():
    # beta = 1 in Eq. 5: sum_t g~(t) + h(T) = sum_t g(t): nothing is lost, only delayed
    T, n, B, s = 10, 600, 128, 2
    gs, hs, gqs, _ = _run_steps(T, n, B, s, alpha=1.0, beta=1.0, mode=0)
    assert np.allclose(sum(gqs) + hs[T], sum(g.astype(np.float64) for g in gs), rtol=0, atol=1e-6)


# ------------------------------------------------------------- edge cases ----
def test_zero_tiny_nonfinite_and_negative_zero():
    B, s = 32, 4
    n = 4 * B
    g = np.zeros(n, np.float32)
    h = np.zeros(n, np.float32)
    g[B:2 * B] = np.float32(1e-39)          # denormal bucket: s/scale overflows
    g[2 * B] = np.nan                         # non-finite bucket
    g[2 * B + 1] = 5.0
    g[3 * B] = -0.0
    g[3 * B + 1] = 1.0
    h[:] = 0.5
    h[3 * B:] = 0
    h0 = h.copy()
    codes, scales, st = enc(g, h, bucket=B, s=s, alpha=0.0, beta=0.5)
    q = oracle.unpack_levels(codes, n=n, s=s)
    assert st == oracle.STATUS_NONFINITE
    assert np.all(q[:3 * B] == 0) and np.all(scales[:3] == 0)
    assert np.array_equal(h[:B], np.float32(0.25) + g[:B])             # beta*h + g, g~ = 0
    assert np.allclose(h[B:2 * B], 0.25 + 1e-39)
    assert np.array_equal(h[2 * B:3 * B], h0[2 * B:3 * B])             # untouched
    assert q[3 * B] == 0 and q[3 * B + 1] == s and scales[3] == 1.0     # -0.0 -> level 0


def test_tail_bucket_and_slices():
    # a ragged tail forms its own bucket; encoding whole buckets of a slice with
    # first_index gives the same result as the matching part of the full vector
    rng = np.random.default_rng(21)
    n, B, s = 3 * 96 + 40, 96, 8
    r = oracle.code_bits(s)
    g = rng.standard_normal(n).astype(np.float32)
    h = (rng.standard_normal(n) * 0.1).astype(np.float32)
    hf = h.copy()
    codes, scales, _ = enc(g, hf, bucket=B, s=s, worker=3, step=9)
    assert scales.size == 4 and codes.size == -(-n * r // 32)
    v_tail = np.float32(np.float32(1.0) * h[3 * B:].astype(np.float64) + g[3 * B:])
    assert scales[3] == np.abs(v_tail).max()
    hs = h[2 * B:].copy()
    c2, s2, _ = enc(g[2 * B:].copy(), hs, bucket=B, s=s, worker=3, step=9, first_index=2 * B)
    assert np.array_equal(s2, scales[2:]) and np.array_equal(hs, hf[2 * B:])
    assert np.array_equal(np_unpack(c2, n - 2 * B, r), np_unpack(codes, n, r)[2 * B:])


# ---------------------------------------------------------------- decode -----
def test_decode_special_cases():
    rng = np.random.default_rng(17)
    n, B, s = 1000, 128, 4
    g = rng.standard_normal(n).astype(np.float32)
    codes, scales, _ = enc(g, np.zeros(n, np.float32), bucket=B, s=s)
    q = oracle.unpack_levels(codes, n=n, s=s)
    a = np.repeat(scales / np.float32(s), B)[:n]
    gq = (q.astype(np.float32) * a).astype(np.float32)
    # W = 1, and W identical messages, return the dequantised vector itself
    assert np.array_equal(oracle.decode_mean([codes], [scales], n=n, bucket=B, s=s), gq)
    out4 = oracle.decode_mean([codes] * 4, [scales] * 4, n=n, bucket=B, s=s)
    assert np.allclose(out4, gq, rtol=1e-6, atol=0)


def test_decode_exact_integer_case_and_fp64():
    # power-of-two scales and s make every operation exact: compare with integers
    rng = np.random.default_rng(23)
    n, B, s, W = 640, 64, 4, 8
    msgs, scl, qs = [], [], []
    for w in range(W):
        g = rng.integers(-s, s + 1, n).astype(np.float32)
        g[::B] = s * rng.choice([-1, 1], n // B)           # scale = s exactly -> a = 1
        g *= 2.0 ** (w % 3)                                   # a in {1,2,4}
        codes, scales, _ = enc(g, np.zeros(n, np.float32), bucket=B, s=s, worker=w)
        msgs.append(codes); scl.append(scales)
        qs.append(g.astype(np.int64))
    out = oracle.decode_mean(msgs, scl, n=n, bucket=B, s=s)
    assert np.array_equal(out * W, sum(qs).astype(np.float32))
    # generic case against an independent fp64 evaluation of Eq. 4
    msgs, scl, acc = [], [], np.zeros(n)
    for w in range(W):
        g = (rng.standard_normal(n) * 10.0 ** rng.uniform(-4, 1)).astype(np.float32)
        codes, scales, _ = enc(g, np.zeros(n, np.float32), bucket=B, s=s, worker=w)
        msgs.append(codes); scl.append(scales)
        acc += (np_unpack(codes, n, oracle.code_bits(s)) - s) * np.repeat(scales.astype(np.float64), B)[:n] / s
    out = oracle.decode_mean(msgs, scl, n=n, bucket=B, s=s)
    # fp32 partial sums carry rounding errors relative to the largest scale
    top = max(float(x.max()) for x in scl)
    assert np.allclose(out, acc / W, rtol=1e-6, atol=2.0 ** -22 * top)


# ------------------------------------------------- fused model update --------
def test_decode_mean_update_is_algorithm1_last_line():
    # w <- w - eta * mean: eta = 0 leaves w alone; power-of-two data makes every operation
    # exact (compare with integers); otherwise compare with an independent fp64 evaluation
    rng = np.random.default_rng(31)
    n, B, s, W = 512, 64, 4, 4
    msgs, scl, ints = [], [], []
    for w in range(W):
        g = rng.integers(-s, s + 1, n).astype(np.float32)
        g[::B] = s                                     # scale = s exactly -> level step 1
        c, sc, _ = enc(g, np.zeros(n, np.float32), bucket=B, s=s, worker=w)
        msgs.append(c); scl.append(sc); ints.append(g.astype(np.int64))
    mean = oracle.decode_mean(msgs, scl, n=n, bucket=B, s=s)
    p0 = rng.integers(-100, 100, n).astype(np.float32)
    p = p0.copy()
    out = oracle.decode_mean_update(msgs, scl, p, eta=0.0, bucket=B, s=s)
    assert np.array_equal(p, p0) and np.array_equal(out, mean)
    p = p0.copy()
    oracle.decode_mean_update(msgs, scl, p, eta=0.5, bucket=B, s=s)
    assert np.array_equal(p * 8, p0 * 8 - sum(ints).astype(np.float32))     # 0.5 * (sum / 4) exact
    # generic values: one rounding away from the exact w - eta * mean
    msgs, scl = [], []
    for w in range(W):
        g = (rng.standard_normal(n) * 0.05).astype(np.float32)
        c, sc, _ = enc(g, np.zeros(n, np.float32), bucket=B, s=s, worker=w)
        msgs.append(c); scl.append(sc)
    mean = oracle.decode_mean(msgs, scl, n=n, bucket=B, s=s).astype(np.float64)
    p0 = rng.standard_normal(n).astype(np.float32)
    p = p0.copy()
    eta = np.float32(0.02)
    oracle.decode_mean_update(msgs, scl, p, eta=float(eta), bucket=B, s=s)
    exact = p0.astype(np.float64) - float(eta) * mean
    assert np.all(np.abs(p - exact) <= 0.5 * np.spacing(np.abs(exact).astype(np.float32)) * 1.0001)
    assert not np.array_equal(p, p0)


# ------------------------------------------------- level statistics ----------
def test_code_histogram_and_entropy_bound():
    rng = np.random.default_rng(41)
    for s, B, n in ((1, 128, 1000), (4, 512, 5000), (8, 96, 4001), (128, 4096, 9000)):
        g = (rng.standard_normal(n) * 0.01).astype(np.float32)
        codes, _, _ = enc(g, np.zeros(n, np.float32), bucket=B, s=s)
        counts = oracle.code_histogram(codes, n=n, s=s)
        ref = np.bincount(np_unpack(codes, n, oracle.code_bits(s)), minlength=2 * s + 1)
        assert counts.sum() == n and np.array_equal(counts.astype(np.int64), ref)   # library bincount
        d = counts.astype(np.float64)
        nz = d > 0
        assert abs(oracle.entropy_bound_bits(counts) - (d[nz] * np.log2(n / d[nz])).sum()) < 1e-6 * n
    # closed forms: 2^k equally likely levels cost k bits per entry; one level costs nothing;
    # and the bound never exceeds the fixed-width cost d * r
    assert oracle.entropy_bound_bits(np.array([256] * 8, np.uint64)) == 8 * 256 * 3.0
    assert oracle.entropy_bound_bits(np.array([0, 12345, 0], np.uint64)) == 0.0
    assert oracle.entropy_bound_bits(np.array([10, 980, 10], np.uint64)) < 1000 * 2


# ------------------------------------------------------- l2-norm scale -------
def _parse_positions(txt, cast):
    pos, out = 0, {}
    for tok in txt.split(","):
        tok = tok.strip()
        if tok.startswith("@"):
            pos = int(tok[1:])
        else:
            out[pos] = cast(tok); pos += 1
    return out


def test_l2_scale_golden():
    for row in _rows("l2_scale_cases.txt"):
        s, B, vals, scale, levels = [x.strip() for x in row.split("|")]
        s, B = int(s), int(B)
        g = np.zeros(B, np.float32)
        for k, v in _parse_positions(vals, float).items():
            g[k] = v
        codes, scales, st = enc(g, np.zeros(B, np.float32), bucket=B, s=s, norm=1)
        q = oracle.unpack_levels(codes, n=B, s=s)
        want = np.zeros(B, np.int64)
        for k, v in _parse_positions(levels, int).items():
            want[k] = v
        assert st == 0 and scales[0] == np.float32(scale) and np.array_equal(q, want)


def test_l2_scale_against_fp64_and_its_invariants():
    rng = np.random.default_rng(51)
    n, B, s = 5 * 512 + 100, 512, 4
    g = (rng.standard_normal(n) * 0.01).astype(np.float32)
    h = (rng.standard_normal(n) * 0.003).astype(np.float32)
    v = np.float32(g + h)                                # alpha = 1: one rounded sum
    codes, scales, st = enc(g, h.copy(), bucket=B, s=s, norm=1)
    q = oracle.unpack_levels(codes, n=n, s=s)
    for b in range(-(-n // B)):
        vb = v[b * B:(b + 1) * B].astype(np.float64)
        ref = np.sqrt((vb * vb).sum())                   # library norm in fp64
        assert abs(float(scales[b]) - ref) <= 2.0 ** -21 * ref
        a = float(scales[b]) / s
        sl = slice(b * B, min((b + 1) * B, n))
        assert np.all(np.abs(q[sl] * a - v[sl]) <= a * (1 + 2.0 ** -20))     # one level step
        assert np.all(q[sl] * v[sl] >= 0)
    # the l2 norm dominates the l-infinity norm, so levels sit lower than with norm = 0
    c0, s0, _ = enc(g, h.copy(), bucket=B, s=s, norm=0)
    assert np.all(scales >= s0) and np.abs(q).sum() < np.abs(oracle.unpack_levels(c0, n=n, s=s)).sum()


def test_l2_quantiser_is_qsgd_lemma1():
    # with the l2 scale the quantiser is QSGD's: unbiased, and
    # E||eps||^2 <= min(d/s^2, sqrt(d)/s) ||v||^2  (Lemma 1)
    rng = np.random.default_rng(61)
    d, N = 256, 1500
    g = (rng.standard_normal(d)).astype(np.float32)
    for s in (1, 4, 16):
        acc = np.zeros(d); err2 = 0.0
        for k in range(N):
            codes, scales, _ = enc(g, np.zeros(d, np.float32), bucket=d, s=s, norm=1, seed=k, step=k % 5)
            gq = oracle.unpack_levels(codes, n=d, s=s) * (float(scales[0]) / s)
            acc += gq; err2 += ((gq - g) ** 2).sum()
        norm2 = float((g.astype(np.float64) ** 2).sum())
        bound = min(d / s ** 2, np.sqrt(d) / s) * norm2
        assert err2 / N <= bound
        a = float(scales[0]) / s
        assert np.all(np.abs(acc / N - g) <= 5 * a / (2 * np.sqrt(N)))


def test_l2_summation_order_is_the_stated_one():
    # integers up to 2^12 keep every partial sum exact in fp32 (< 2^24 * ...): any order gives
    # the same sum; with wide-ranging values the stated order is reproduced step by step here
    rng = np.random.default_rng(71)
    B = 32 * 5                                            # five runs: the odd one is carried up
    for trial in range(40):
        v = (rng.standard_normal(B) * 10.0 ** rng.uniform(-3, 3, B)).astype(np.float32)
        runs = []
        for r0 in range(0, B, 32):
            acc = np.float32(0)
            for x in v[r0:r0 + 32]:
                acc = np.float32(np.float64(x) * np.float64(x) + np.float64(acc))    # fma: one rounding
            runs.append(acc)
        while len(runs) > 1:
            runs = [np.float32(runs[k] + runs[k + 1]) if k + 1 < len(runs) else runs[k]
                    for k in range(0, len(runs), 2)]
        _, scales, _ = enc(v, np.zeros(B, np.float32), bucket=B, s=4, norm=1)
        assert scales[0] == np.sqrt(runs[0], dtype=np.float32), trial
