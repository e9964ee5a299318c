"""Helpers of the GPU parity tests: run the CUDA codec through its C ABI and the
CPU oracle on the same inputs and compare them element by element.

Tolerances (stated once, used everywhere):
  codes, scales : bit-exact
  err, out      : |x - y| <= 1e-7 + 1e-6 * |y|   (y = oracle)
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
from typing import List, Sequence, Tuple

import numpy as np
import torch

import oracle
import paper_1806_08054_b200 as ecq

ATOL, RTOL = 1e-7, 1e-6


def close(x: np.ndarray, y: np.ndarray) -> bool:
    return bool(np.all(np.abs(x.astype(np.float64) - y.astype(np.float64))
                       <= ATOL + RTOL * np.abs(y.astype(np.float64))))


class GpuCodec:
    """Owns a context and the per-worker device buffers of one configuration."""

    def __init__(self, d, bucket, s, alpha, beta, seed, W, mode=0, norm=0, decode_plan=None):
        self.d, self.bucket, self.s, self.W = d, bucket, s, W
        self.ctx = ecq.ecq_create(d, bucket, s, alpha, beta, seed)
        if mode:
            ecq.ecq_set_error_mode(self.ctx, mode)
        if norm:
            ecq.ecq_set_norm(self.ctx, norm)
        if decode_plan is not None:
            ecq.ecq_set_decode_plan(self.ctx, *decode_plan)
        self.r = ecq.ecq_code_bits(self.ctx)
        self.nb = ecq.ecq_num_buckets(self.ctx)
        self.nw = ecq.ecq_codes_words(self.ctx)
        dev = "cuda"
        # guard words around every output so that a stray write is caught
        self.pad = 64
        self.err = [self._guarded(d, torch.float32, 0.0) for _ in range(W)]
        self.codes = [self._guarded(self.nw, torch.int32, 0x5A5A5A5A) for _ in range(W)]
        self.scales = [self._guarded(self.nb, torch.float32, -7.0) for _ in range(W)]
        self.out = self._guarded(d, torch.float32, -7.0)
        self.dev = dev

    def _guarded(self, n, dtype, fill):
        buf = torch.empty(n + 2 * self.pad, dtype=dtype, device="cuda")
        buf.fill_(123456789 if dtype == torch.int32 else 12345.678)
        view = buf[self.pad:self.pad + n]
        view.fill_(fill)
        return (buf, view)

    def check_guards(self):
        for buf, view in self.err + self.codes + self.scales + [self.out]:
            want = 123456789 if buf.dtype == torch.int32 else np.float32(12345.678)
            a = buf[:self.pad].cpu().numpy()
            b = buf[self.pad + view.numel():].cpu().numpy()
            assert np.all(a == want) and np.all(b == want), "write outside an output buffer"

    def encode(self, worker, step, grad):
        ecq.ecq_encode(self.ctx, worker, step, grad, self.err[worker][1],
                       self.codes[worker][1], self.scales[worker][1])

    def encode_batch(self, step, grads):
        W = len(grads)
        ecq.ecq_encode_batch(self.ctx, step, grads, [e[1] for e in self.err[:W]],
                             [c[1] for c in self.codes[:W]], [s[1] for s in self.scales[:W]])

    def decode(self, W=None):
        W = W or self.W
        ecq.ecq_decode_mean(self.ctx, [c[1] for c in self.codes[:W]],
                            [s[1] for s in self.scales[:W]], self.out[1])

    def status(self):
        return ecq.ecq_status(self.ctx)

    def close(self):
        ecq.ecq_destroy(self.ctx)


def codes_np(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint32)


def full_parity(d, bucket, s, alpha, beta, seed, W, steps, grad_fn, mode=0, err0=None,
                expect_status=ecq.ECQ_OK, check_decode=True, batch=False, norm=0, decode_plan=None):
    """Element-by-element comparison over whole vectors.

    ``grad_fn(worker, step)`` returns a float32 CUDA tensor of d entries.
    """
    gpu = GpuCodec(d, bucket, s, alpha, beta, seed, W, mode, norm, decode_plan)
    try:
        h_or = [np.zeros(d, np.float32) for _ in range(W)]
        if err0 is not None:
            for w in range(W):
                gpu.err[w][1].copy_(err0[w])
                h_or[w] = err0[w].cpu().numpy().copy()
        for t in range(steps):
            grads = [grad_fn(w, t) for w in range(W)]
            if batch:
                gpu.encode_batch(t, grads)
            else:
                for w in range(W):
                    gpu.encode(w, t, grads[w])
            if check_decode:
                gpu.decode()
            st = gpu.status()
            assert st == expect_status, "status %d (%s)" % (st, ecq.binding.strerror(st))
            g_host = [g.cpu().numpy() for g in grads]

            def one(w):
                return oracle.encode(g_host[w], h_or[w], bucket=bucket, s=s, alpha=alpha,
                                     beta=beta, seed=seed, worker=w, step=t, mode=mode, norm=norm)
            with ThreadPoolExecutor(max_workers=min(W, 8)) as ex:
                res = list(ex.map(one, range(W)))
            for w in range(W):
                c_or, s_or, _ = res[w]
                c_gpu = codes_np(gpu.codes[w][1])
                assert np.array_equal(gpu.scales[w][1].cpu().numpy().view(np.uint32),
                                      s_or.view(np.uint32)), "scales differ (w=%d t=%d)" % (w, t)
                if not np.array_equal(c_gpu, c_or):
                    bad = np.nonzero(c_gpu != c_or)[0]
                    raise AssertionError("codes differ (w=%d t=%d): %d words, first at %d"
                                         % (w, t, bad.size, bad[0]))
                assert close(gpu.err[w][1].cpu().numpy(), h_or[w]), "err differs (w=%d t=%d)" % (w, t)
            if check_decode:
                out_or = oracle.decode_mean([r[0] for r in res], [r[1] for r in res],
                                            n=d, bucket=bucket, s=s)
                assert close(gpu.out[1].cpu().numpy(), out_or), "decoded mean differs (t=%d)" % t
            gpu.check_guards()
    finally:
        gpu.close()


def sample_ranges(d: int, bucket: int, span: int = 1 << 16, count: int = 3,
                  seed: int = 0) -> List[Tuple[int, int]]:
    """Whole-bucket index ranges: the head, the ragged end, and some in between."""
    nb = -(-d // bucket)
    per = max(span // bucket, 1)
    rng = np.random.default_rng(seed)
    starts = {0, max(nb - per, 0)}
    while len(starts) < min(count + 2, max(nb // per, 1)):
        starts.add(int(rng.integers(0, max(nb - per, 1))))
    out = []
    for b0 in sorted(starts):
        lo = b0 * bucket
        hi = min((b0 + per) * bucket, d)
        out.append((lo, hi))
    return out


def placed_ranges(d: int, bucket: int, W: int, span: int = 8192, count: int = 64,
                  seed: int = 0) -> List[Tuple[int, int]]:
    """Whole-bucket windows of about ``span`` entries, placed where the kernels change what
    they do rather than at random only: the first and last tiles of a vector (in the batched
    encode launch those are where a CTA passes from one worker's vector to the next), the
    tiles either side of the points where the grid of CTAs wraps around (encode: 592 and 296
    CTAs over tiles of 4096 and 8192 entries; receiver: 148 CTAs over tiles of 30720 and 1184
    warps over tiles of 1024), the last whole tile and the ragged end behind it; random
    windows fill up to ``count``."""
    per = max(span // bucket, 1)                       # buckets per window
    nb = -(-d // bucket)
    points = [0, d]                                    # entry positions of interest
    for tile, ctas in ((4096, 592), (8192, 296), (30720, 148), (1024, 1184)):
        n_t = d // tile
        points += [tile, tile * ctas, tile * (ctas + 1), 2 * tile * ctas, n_t * tile, (n_t - 1) * tile]
        # where worker w's share of the launch's global tile sequence meets the grid's stride
        for w in range(1, min(W, 4)):
            first = (-(w * n_t)) % ctas                # first tile of worker w that CTA 0 takes
            points += [first * tile, (first + 1) * tile]
    starts = set()
    for pnt in points:
        b = min(max(pnt // bucket, 0), nb - 1)
        for b0 in (b - per, b):                        # the window before and the one from the point
            starts.add(min(max(b0, 0), max(nb - per, 0)))
    starts.add(max(nb - per, 0))
    rng = np.random.default_rng(seed)
    while len(starts) < min(count, max(nb // per, 1)):
        starts.add(int(rng.integers(0, max(nb - per, 1))))
    return [(b0 * bucket, min((b0 + per) * bucket, d)) for b0 in sorted(starts)]


class SampledOracle:
    """Follows the oracle on sampled whole-bucket ranges of a large vector."""

    def __init__(self, d, bucket, s, alpha, beta, seed, W, ranges, mode=0, norm=0):
        self.d, self.bucket, self.s, self.W = d, bucket, s, W
        self.alpha, self.beta, self.seed, self.mode, self.norm = alpha, beta, seed, mode, norm
        self.ranges = ranges
        self.r = oracle.code_bits(s)
        self.h = [[np.zeros(hi - lo, np.float32) for (lo, hi) in ranges] for _ in range(W)]
        self.msgs = [[None] * len(ranges) for _ in range(W)]

    def encode_and_compare(self, gpu: GpuCodec, w: int, step: int, grad: torch.Tensor):
        for k, (lo, hi) in enumerate(self.ranges):
            g = grad[lo:hi].cpu().numpy()
            c_or, s_or, _ = oracle.encode(g, self.h[w][k], bucket=self.bucket, s=self.s,
                                          alpha=self.alpha, beta=self.beta, seed=self.seed,
                                          worker=w, step=step, mode=self.mode, first_index=lo,
                                          norm=self.norm)
            self.msgs[w][k] = (c_or, s_or)
            w0 = lo * self.r // 32
            c_gpu = codes_np(gpu.codes[w][1][w0:w0 + c_or.size])
            s_gpu = gpu.scales[w][1][lo // self.bucket: lo // self.bucket + s_or.size].cpu().numpy()
            assert np.array_equal(s_gpu.view(np.uint32), s_or.view(np.uint32)), \
                "scales differ (w=%d t=%d range %d)" % (w, step, k)
            assert np.array_equal(c_gpu, c_or), "codes differ (w=%d t=%d range %d)" % (w, step, k)
            assert close(gpu.err[w][1][lo:hi].cpu().numpy(), self.h[w][k]), \
                "err differs (w=%d t=%d range %d)" % (w, step, k)

    def decode_and_compare(self, gpu: GpuCodec):
        for k, (lo, hi) in enumerate(self.ranges):
            out_or = oracle.decode_mean([self.msgs[w][k][0] for w in range(self.W)],
                                        [self.msgs[w][k][1] for w in range(self.W)],
                                        n=hi - lo, bucket=self.bucket, s=self.s)
            assert close(gpu.out[1][lo:hi].cpu().numpy(), out_or), "decoded mean differs (range %d)" % k


def whole_message_properties(gpu: GpuCodec, w: int, grad: torch.Tensor, beta: float,
                             scratch: torch.Tensor, sum64: torch.Tensor = None):
    """Worker w's whole message and accumulator after its FIRST encode (h was zero, so the
    compensated value is the gradient itself), checked on the device over every entry:
    the dequantised entries g~ (a one-message decode of the codes) are whole multiples q of the
    bucket's level step a = scale / s with |q| <= s (Eq. 8: every code is in range), lie within
    one level step of the input (Eq. 9 rounds to a neighbouring level), and the new
    accumulator is the rounded g - g~ (Eq. 6 with h = 0).  ``sum64`` collects g~ in fp64 for a
    later check of the decoded mean."""
    d, B, s = gpu.d, gpu.bucket, gpu.s
    ecq.ecq_decode_mean(gpu.ctx, [gpu.codes[w][1]], [gpu.scales[w][1]], scratch)
    assert gpu.status() == ecq.ECQ_OK
    gq = scratch
    a = (gpu.scales[w][1] / float(s)).repeat_interleave(B)[:d]
    live = a > 0
    # within one level step: Eq. 9 rounds to a neighbouring level; the fp32 roundings of
    # s/scale, |v| s/scale and q a move the ratio by a few 2^-24 of s levels at most
    assert bool(((gq - grad).abs() <= a * (1 + s * 2.0 ** -21)).logical_or(~live).all()), "beyond one level step"
    assert bool((gq[~live] == 0).all())
    q = torch.where(live, gq / torch.where(live, a, torch.ones_like(a)), torch.zeros_like(gq))
    qr = q.round()
    assert bool(((q - qr).abs() <= 1e-4).all()), "a dequantised entry is no multiple of the level step"
    assert bool((qr.abs() <= s).all()), "level out of range"
    assert bool((qr * grad >= 0).logical_or(qr == 0).all()), "level with the wrong sign"
    # Eq. 6 from a zero accumulator: h' = beta * 0 + (g - g~)
    e = grad - gq
    h = gpu.err[w][1]
    assert bool(((h - e).abs() <= ATOL + RTOL * e.abs()).all()), "accumulator is not g - g~"
    if sum64 is not None:
        sum64 += gq.double()


def whole_vector_properties(gpu: GpuCodec, w: int, grad: torch.Tensor, err_before: torch.Tensor,
                            alpha: float):
    """Checks that hold at any size, evaluated on the device over the whole vector.

    With alpha == 1 the compensated value is the single rounded sum g + h, so the
    scales must equal the library max-abs per bucket exactly.
    """
    d, B = gpu.d, gpu.bucket
    assert alpha == 1.0
    v = grad + err_before
    nb_full = d // B
    sc = gpu.scales[w][1]
    if nb_full:
        ref = v[: nb_full * B].abs().view(nb_full, B).amax(dim=1)
        finite = ref * (gpu.s / ref) < float("inf")
        assert torch.equal(torch.where(finite, ref, torch.zeros_like(ref)).view(torch.int32),
                           sc[:nb_full].view(torch.int32)), "scales != library max-abs"
    if d % B:
        assert sc[-1].item() == v[nb_full * B:].abs().max().item()
