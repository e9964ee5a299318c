"""CPU oracle of the ECQ-SGD gradient codec -- TEST INFRASTRUCTURE ONLY.

Thin numpy/ctypes wrapper around ``ecq_oracle.cpp`` (plain single-threaded C++,
built with ``g++ -O2 -ffp-contract=off``).  Only the tests, the smoke check and
the CPU-baseline leg of the benchmark may import this package; the CUDA library
and its Python binding never do, and this package imports nothing of theirs.

Functions follow the paper's Section 4: ``encode`` is Eq. 7 + Eq. 8 (l-infinity
scale per bucket) + Eq. 9 + Eq. 6 + the fixed-width code; ``decode_mean`` is
Eq. 4 / the global-gradient step of Algorithm 1's phase 2.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRCS = [os.path.join(_HERE, "ecq_oracle.cpp"), os.path.join(_HERE, "ecq_entropy_oracle.cpp")]
_LIB = os.path.join(_HERE, "libecq_oracle.so")

STATUS_NONFINITE = 1


def build(force: bool = False) -> str:
    """Compile the oracle (no optimisation that changes fp32 results)."""
    with _build_lock:          # callers may be pool threads that all find the library missing
        if force or not os.path.exists(_LIB) or \
                os.path.getmtime(_LIB) < max(os.path.getmtime(p) for p in _SRCS):
            tmp = _LIB + ".tmp.%d.%d" % (os.getpid(), threading.get_ident())
            subprocess.check_call([
                "g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math",
                "-shared", "-fPIC", "-o", tmp] + _SRCS)
            os.replace(tmp, _LIB)
    return _LIB


_build_lock = threading.Lock()
_load_lock = threading.Lock()
_lib = None


def _load():
    global _lib
    with _load_lock:
        return _load_locked()


def _load_locked():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u32, u64, f32, i32 = ctypes.c_uint32, ctypes.c_uint64, ctypes.c_float, ctypes.c_int
        vp = ctypes.c_void_p
        lib.ecqo_philox4x32_10.argtypes = [vp, vp, vp]
        lib.ecqo_philox4x32_10.restype = None
        lib.ecqo_draw_word.argtypes = [u64, u32, u32, u64]
        lib.ecqo_draw_word.restype = u32
        lib.ecqo_code_bits.argtypes = [u32]
        lib.ecqo_code_bits.restype = u32
        lib.ecqo_num_buckets.argtypes = [u64, u32]
        lib.ecqo_num_buckets.restype = u64
        lib.ecqo_codes_words.argtypes = [u64, u32]
        lib.ecqo_codes_words.restype = u64
        lib.ecqo_encode.argtypes = [u64, u32, u32, f32, f32, u64, i32, i32, u32, u32, u64,
                                    vp, vp, vp, vp, vp]
        lib.ecqo_encode.restype = i32
        lib.ecqo_encode_given_draws.argtypes = [u64, u32, u32, f32, f32, i32, i32,
                                                vp, vp, vp, vp, vp, vp]
        lib.ecqo_encode_given_draws.restype = i32
        lib.ecqo_decode_mean.argtypes = [u64, u32, u32, u32, vp, vp, vp]
        lib.ecqo_decode_mean.restype = i32
        lib.ecqo_decode_mean_update.argtypes = [u64, u32, u32, u32, vp, vp, f32, vp, vp]
        lib.ecqo_decode_mean_update.restype = i32
        lib.ecqo_code_histogram.argtypes = [u64, u32, vp, vp]
        lib.ecqo_code_histogram.restype = None
        lib.ecqo_entropy_bound_bits.argtypes = [vp, u32]
        lib.ecqo_entropy_bound_bits.restype = ctypes.c_double
        lib.ecqo_unpack_levels.argtypes = [u64, u32, vp, vp]
        lib.ecqo_unpack_levels.restype = None
        lib.ecqo_huffman_lengths.argtypes = [vp, u32, u32, vp]
        lib.ecqo_huffman_lengths.restype = i32
        lib.ecqo_huffman_words.argtypes = [vp, u32, vp]
        lib.ecqo_huffman_words.restype = i32
        lib.ecqo_huffman_chunks.argtypes = [u64]
        lib.ecqo_huffman_chunks.restype = u64
        lib.ecqo_huffman_encode.argtypes = [u64, u32, vp, u32, vp, vp, u64, vp, vp]
        lib.ecqo_huffman_encode.restype = i32
        lib.ecqo_huffman_decode.argtypes = [u64, u32, vp, u32, vp, vp, vp, vp]
        lib.ecqo_huffman_decode.restype = i32
        _lib = lib
    return _lib


def _ptr(a: np.ndarray) -> int:
    return a.ctypes.data


def philox4x32_10(ctr: Sequence[int], key: Sequence[int]) -> np.ndarray:
    """Philox4x32-10 of one 128-bit counter under one 64-bit key (SC'11)."""
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    _load().ecqo_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def draw_word(seed: int, worker: int, step: int, i: int) -> int:
    """The 32-bit word element ``i`` of ``worker`` draws at iteration ``step``."""
    return int(_load().ecqo_draw_word(seed, worker, step, i))


def code_bits(s: int) -> int:
    """r = ceil(log2(2s+1)) (paragraph after Eq. 9)."""
    return int(_load().ecqo_code_bits(s))


def num_buckets(d: int, bucket: int) -> int:
    return int(_load().ecqo_num_buckets(d, bucket))


def codes_words(d: int, s: int) -> int:
    """32-bit words of one worker's code stream."""
    return int(_load().ecqo_codes_words(d, s))


def encode(g: np.ndarray, h: np.ndarray, *, bucket: int, s: int, alpha: float,
           beta: float, seed: int, worker: int, step: int, mode: int = 0,
           first_index: int = 0, draws: Optional[np.ndarray] = None, norm: int = 0):
    """Encode one worker's slice; ``h`` is updated IN PLACE (Eq. 6).

    ``norm`` 0 takes the l-infinity norm of the bucket as the scale of Eq. 8, 1 the l2 norm.
    Returns ``(codes uint32[words], scales float32[nb], status)``.  ``draws``
    (one uint32 per element) replaces the Philox stream when given.
    """
    assert g.dtype == np.float32 and h.dtype == np.float32
    assert g.flags.c_contiguous and h.flags.c_contiguous and g.shape == h.shape
    n = g.size
    codes = np.zeros(max(codes_words(n, s), 1), dtype=np.uint32)
    scales = np.zeros(max(num_buckets(n, bucket), 1), dtype=np.float32)
    status = np.zeros(1, dtype=np.uint32)
    lib = _load()
    if draws is None:
        rc = lib.ecqo_encode(n, bucket, s, alpha, beta, seed, mode, norm, worker, step,
                             first_index, _ptr(g), _ptr(h), _ptr(codes), _ptr(scales),
                             _ptr(status))
    else:
        dr = np.ascontiguousarray(draws, dtype=np.uint32)
        assert dr.size == n
        rc = lib.ecqo_encode_given_draws(n, bucket, s, alpha, beta, mode, norm, _ptr(dr),
                                         _ptr(g), _ptr(h), _ptr(codes), _ptr(scales),
                                         _ptr(status))
    if rc != 0:
        raise ValueError("oracle encode: bad arguments")
    return codes[:codes_words(n, s)], scales[:num_buckets(n, bucket)], int(status[0])


def decode_mean(codes: Sequence[np.ndarray], scales: Sequence[np.ndarray], *,
                n: int, bucket: int, s: int) -> np.ndarray:
    """Mean of the W dequantised messages (Eq. 4)."""
    W = len(codes)
    assert W == len(scales) and W >= 1
    cs = [np.ascontiguousarray(c, dtype=np.uint32) for c in codes]
    ss = [np.ascontiguousarray(x, dtype=np.float32) for x in scales]
    cp = (ctypes.c_void_p * W)(*[_ptr(c) for c in cs])
    sp = (ctypes.c_void_p * W)(*[_ptr(x) for x in ss])
    out = np.zeros(n, dtype=np.float32)
    rc = _load().ecqo_decode_mean(n, bucket, s, W, cp, sp, _ptr(out))
    if rc != 0:
        raise ValueError("oracle decode_mean: bad arguments")
    return out


def decode_mean_update(codes: Sequence[np.ndarray], scales: Sequence[np.ndarray], params: np.ndarray,
                       *, eta: float, bucket: int, s: int) -> np.ndarray:
    """Eq. 4 then Algorithm 1's update: ``params`` is updated IN PLACE to
    ``params - eta * mean`` (one fused multiply-add per entry); returns the mean."""
    W, n = len(codes), params.size
    assert params.dtype == np.float32 and params.flags.c_contiguous
    cs = [np.ascontiguousarray(c, dtype=np.uint32) for c in codes]
    ss = [np.ascontiguousarray(x, dtype=np.float32) for x in scales]
    cp = (ctypes.c_void_p * W)(*[_ptr(c) for c in cs])
    sp = (ctypes.c_void_p * W)(*[_ptr(x) for x in ss])
    out = np.zeros(n, dtype=np.float32)
    rc = _load().ecqo_decode_mean_update(n, bucket, s, W, cp, sp, eta, _ptr(params), _ptr(out))
    if rc != 0:
        raise ValueError("oracle decode_mean_update: bad arguments")
    return out


def code_histogram(codes: np.ndarray, *, n: int, s: int) -> np.ndarray:
    """d_k, k < 2s+1: entries of the message on level k - s."""
    c = np.ascontiguousarray(codes, dtype=np.uint32)
    counts = np.zeros(2 * s + 1, dtype=np.uint64)
    _load().ecqo_code_histogram(n, s, _ptr(c), _ptr(counts))
    return counts


def entropy_bound_bits(counts: np.ndarray) -> float:
    """sum_k d_k log2(d / d_k) (paragraph after Eq. 9)."""
    c = np.ascontiguousarray(counts, dtype=np.uint64)
    return float(_load().ecqo_entropy_bound_bits(_ptr(c), c.size))


def unpack_levels(codes: np.ndarray, *, n: int, s: int) -> np.ndarray:
    """Signed levels q_i in [-s, s] of one message."""
    c = np.ascontiguousarray(codes, dtype=np.uint32)
    q = np.zeros(n, dtype=np.int32)
    _load().ecqo_unpack_levels(n, s, _ptr(c), _ptr(q))
    return q


# ---- entropy-coded message (paragraph after Eq. 9: "e.g. Huffman") ----------
HUFFMAN_CHUNK = 1024


def huffman_lengths(counts: np.ndarray, *, max_len: int = 12) -> np.ndarray:
    """Word lengths of an optimal prefix code limited to ``max_len`` bits (0 = absent)."""
    c = np.ascontiguousarray(counts, dtype=np.uint64)
    out = np.zeros(c.size, dtype=np.uint8)
    rc = _load().ecqo_huffman_lengths(_ptr(c), c.size, max_len, _ptr(out))
    if rc != 0:
        raise ValueError("alphabet does not fit the length limit")
    return out


def huffman_words(lengths: np.ndarray) -> np.ndarray:
    """Canonical code words for the given lengths."""
    L = np.ascontiguousarray(lengths, dtype=np.uint8)
    out = np.zeros(L.size, dtype=np.uint32)
    if _load().ecqo_huffman_words(_ptr(L), L.size, _ptr(out)) != 0:
        raise ValueError("lengths are not those of a prefix code")
    return out


def huffman_chunks(n: int) -> int:
    return int(_load().ecqo_huffman_chunks(n))


def huffman_encode(codes: np.ndarray, lengths: np.ndarray, *, n: int, s: int,
                   capacity: Optional[int] = None):
    """Entropy-code one message.  Returns (stream words, chunk offsets, quarter positions)."""
    r = code_bits(s)
    c = np.ascontiguousarray(codes, dtype=np.uint32)
    L = np.ascontiguousarray(lengths, dtype=np.uint8)
    n_chunks = huffman_chunks(n)
    cap = capacity if capacity is not None else (n * 32 + 31) // 32 + n_chunks
    stream = np.zeros(max(cap, 1), dtype=np.uint32)
    offsets = np.zeros(n_chunks + 1, dtype=np.uint32)
    quarters = np.zeros(3 * n_chunks, dtype=np.uint16)
    rc = _load().ecqo_huffman_encode(n, r, _ptr(L), L.size, _ptr(c), _ptr(stream), cap, _ptr(offsets),
                                     _ptr(quarters))
    if rc == 2:
        raise OverflowError("stream does not fit the capacity")
    if rc != 0:
        raise ValueError("lengths do not cover the message")
    return stream[:int(offsets[-1])].copy(), offsets, quarters


def huffman_decode(stream: np.ndarray, offsets: np.ndarray, quarters: np.ndarray,
                   lengths: np.ndarray, *, n: int, s: int) -> np.ndarray:
    """Inverse of :func:`huffman_encode`: the r-bit code words of the message."""
    r = code_bits(s)
    st = np.ascontiguousarray(stream, dtype=np.uint32)
    if st.size == 0:
        st = np.zeros(1, dtype=np.uint32)
    off = np.ascontiguousarray(offsets, dtype=np.uint32)
    qt = np.ascontiguousarray(quarters, dtype=np.uint16)
    if qt.size == 0:
        qt = np.zeros(3, dtype=np.uint16)
    L = np.ascontiguousarray(lengths, dtype=np.uint8)
    out = np.zeros(codes_words(n, s), dtype=np.uint32)
    if _load().ecqo_huffman_decode(n, r, _ptr(L), L.size, _ptr(st), _ptr(off), _ptr(qt), _ptr(out)) != 0:
        raise ValueError("stream holds a bit pattern that is no code word")
    return out
