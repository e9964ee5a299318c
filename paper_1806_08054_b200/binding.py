"""ctypes binding of ``libecq.so``: argument marshalling only.

Every step of the codec runs in the CUDA kernels behind the C ABI declared in
``include/ecq.h``; the functions here have the same names and only turn torch
tensors into pointers.  There is no CPU fallback: if the library is missing or a
tensor is not on a CUDA device the call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Sequence

import torch

from .build import LIB

ECQ_OK, ECQ_ERR_ARG, ECQ_ERR_CUDA, ECQ_ERR_NONFINITE, ECQ_ERR_TIMEOUT, ECQ_ERR_ALLOC = range(6)
ECQ_ERR_TOO_LARGE = 6
ECQ_ERR_CAPACITY = 7
ECQ_ERR_SYMBOL = 8
ECQ_HUFFMAN_MAX_LEN = 12
ECQ_HUFFMAN_CHUNK = 1024
ECQ_HUFFMAN_TABLE_BYTES = 4096 * 4 + 4096 * 4 + 16
ECQ_STATIC_SCRATCH_BYTES = 4 << 20
ECQ_MAX_WORKERS = 64
ECQ_WAIT_LIMIT_DEFAULT = 1 << 22
ECQ_MAX_WORKERS_TOTAL = 1024

_lib = None


class EcqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (status %d)" % (where, strerror(status), status))


def lib() -> ctypes.CDLL:
    """Load the compiled library; raise if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB):
            raise RuntimeError(
                "libecq.so is not built: run `python -m paper_1806_08054_b200.build` "
                "(there is no fallback implementation)")
        L = ctypes.CDLL(LIB)
        u32, u64, f32, i32, vp = (ctypes.c_uint32, ctypes.c_uint64, ctypes.c_float,
                                  ctypes.c_int, ctypes.c_void_p)
        L.ecq_create.argtypes = [ctypes.POINTER(vp), u64, u32, u32, f32, f32, u64]
        L.ecq_create.restype = i32
        L.ecq_destroy.argtypes = [vp]
        L.ecq_destroy.restype = None
        L.ecq_set_error_mode.argtypes = [vp, i32]
        L.ecq_set_error_mode.restype = i32
        L.ecq_set_norm.argtypes = [vp, i32]
        L.ecq_set_norm.restype = i32
        L.ecq_set_decode_plan.argtypes = [vp, i32, ctypes.c_uint32]
        L.ecq_set_decode_plan.restype = i32
        L.ecq_set_wait_limit.argtypes = [vp, ctypes.c_uint32]
        L.ecq_set_wait_limit.restype = i32
        L.ecq_code_bits.argtypes = [vp]
        L.ecq_code_bits.restype = u32
        L.ecq_num_buckets.argtypes = [vp]
        L.ecq_num_buckets.restype = u64
        L.ecq_codes_words.argtypes = [vp]
        L.ecq_codes_words.restype = u64
        L.ecq_encode.argtypes = [vp, u32, u32, vp, vp, vp, vp, vp]
        L.ecq_encode.restype = i32
        L.ecq_encode_batch.argtypes = [vp, u32, u32, vp, vp, vp, vp, vp]
        L.ecq_encode_batch.restype = i32
        L.ecq_decode_mean.argtypes = [vp, u32, vp, vp, vp, vp]
        L.ecq_decode_mean.restype = i32
        L.ecq_decode_mean_update.argtypes = [vp, u32, vp, vp, f32, vp, vp, vp]
        L.ecq_decode_mean_update.restype = i32
        L.ecq_code_histogram.argtypes = [vp, vp, vp, vp]
        L.ecq_code_histogram.restype = i32
        L.ecq_entropy_bound_bits.argtypes = [vp, u32]
        L.ecq_entropy_bound_bits.restype = ctypes.c_double
        L.ecq_step_host_workspace_bytes.argtypes = [vp, u32]
        L.ecq_step_host_workspace_bytes.restype = u64
        L.ecq_step_host.argtypes = [vp, u32, u32, vp, vp, vp, u64, vp, vp]
        L.ecq_step_host.restype = i32
        L.ecq_step_static.argtypes = [u64, u32, u32, f32, f32, u64, u32, u32, vp, vp, vp, vp]
        L.ecq_step_static.restype = i32
        L.ecq_huffman_lengths.argtypes = [vp, vp, vp]
        L.ecq_huffman_lengths.restype = i32
        L.ecq_huffman_chunks.argtypes = [vp]
        L.ecq_huffman_chunks.restype = u64
        L.ecq_huffman_stream_bound.argtypes = [vp, vp, vp]
        L.ecq_huffman_stream_bound.restype = u64
        L.ecq_huffman_tables.argtypes = [vp, vp, vp, vp]
        L.ecq_huffman_tables.restype = i32
        L.ecq_huffman_encode.argtypes = [vp, vp, vp, vp, u64, vp, vp, vp]
        L.ecq_huffman_encode.restype = i32
        L.ecq_huffman_decode.argtypes = [vp, vp, vp, u64, vp, vp, vp, vp]
        L.ecq_huffman_decode.restype = i32
        L.ecq_status.argtypes = [vp, vp]
        L.ecq_status.restype = i32
        L.ecq_launch_count.argtypes = []
        L.ecq_launch_count.restype = u64
        L.ecq_strerror.argtypes = [i32]
        L.ecq_strerror.restype = ctypes.c_char_p
        _lib = L
    return _lib


def strerror(status: int) -> str:
    return lib().ecq_strerror(status).decode()


def _stream(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream


def _dev(t: torch.Tensor, dtype, name: str) -> int:
    if not t.is_cuda:
        raise ValueError("%s must be a CUDA tensor (the codec has no CPU path)" % name)
    if t.dtype != dtype or not t.is_contiguous():
        raise ValueError("%s must be contiguous %s" % (name, dtype))
    return t.data_ptr()


class PointerTable:
    """Device addresses of a fixed list of tensors, checked and marshalled once.  The calls
    that take one tensor per worker accept a table in place of the sequence, which saves the
    per-tensor checks on every call when the same buffers serve every step.  The table keeps
    its tensors alive; it holds addresses, so a tensor that is resized or replaced needs a new
    table."""
    __slots__ = ("array", "n", "dtype", "_keep")

    def __init__(self, tensors: Sequence[torch.Tensor], dtype, name: str = "tensors"):
        self._keep = list(tensors)
        self.n = len(self._keep)
        self.dtype = dtype
        self.array = (ctypes.c_void_p * self.n)(*[_dev(x, dtype, name) for x in self._keep])

    def __len__(self) -> int:
        return self.n


def pointer_table(tensors: Sequence[torch.Tensor], dtype, name: str = "tensors") -> PointerTable:
    """Marshal a list of CUDA tensors of one dtype once, for use in many calls."""
    return PointerTable(tensors, dtype, name)


def _table(ts, dtype, name: str) -> PointerTable:
    if isinstance(ts, PointerTable):
        if ts.dtype != dtype:
            raise ValueError("%s must be a table of %s tensors" % (name, dtype))
        return ts
    return PointerTable(ts, dtype, name)


def ecq_create(d: int, bucket: int, levels: int, alpha: float, beta: float, seed: int) -> int:
    """Return an opaque context handle (see ``ecq_create`` in ecq.h)."""
    h = ctypes.c_void_p()
    rc = lib().ecq_create(ctypes.byref(h), d, bucket, levels, alpha, beta, seed)
    if rc != ECQ_OK:
        raise EcqError(rc, "ecq_create")
    return h.value


def ecq_destroy(ctx: int) -> None:
    lib().ecq_destroy(ctx)


def ecq_set_error_mode(ctx: int, mode: int) -> None:
    rc = lib().ecq_set_error_mode(ctx, mode)
    if rc != ECQ_OK:
        raise EcqError(rc, "ecq_set_error_mode")


def ecq_set_norm(ctx: int, norm: int) -> None:
    """0: l-infinity scale per bucket (default); 1: l2 scale (Eq. 8 allows either)."""
    rc = lib().ecq_set_norm(ctx, norm)
    if rc != ECQ_OK:
        raise EcqError(rc, "ecq_set_norm")


ECQ_DECODE_AUTO, ECQ_DECODE_WARP, ECQ_DECODE_RING = 0, 1, 2


def ecq_set_decode_plan(ctx: int, kernel: int = ECQ_DECODE_AUTO, max_ctas: int = 0) -> None:
    """Which receiver kernel a launch takes and how many CTAs at most (0: fill the device)."""
    rc = lib().ecq_set_decode_plan(ctx, kernel, max_ctas)
    if rc != ECQ_OK:
        raise EcqError(rc, "ecq_set_decode_plan")


def ecq_set_wait_limit(ctx: int, polls: int) -> None:
    """Polls an in-kernel wait for an asynchronous copy makes before it gives up (default 2**22)."""
    rc = lib().ecq_set_wait_limit(ctx, polls)
    if rc != ECQ_OK:
        raise EcqError(rc, "ecq_set_wait_limit")


def ecq_code_bits(ctx: int) -> int:
    return int(lib().ecq_code_bits(ctx))


def ecq_num_buckets(ctx: int) -> int:
    return int(lib().ecq_num_buckets(ctx))


def ecq_codes_words(ctx: int) -> int:
    return int(lib().ecq_codes_words(ctx))


def ecq_encode(ctx: int, worker: int, step: int, grad: torch.Tensor, err: torch.Tensor,
               codes: torch.Tensor, scales: torch.Tensor, stream=None) -> None:
    """Enqueue the fused sender-side kernel; ``err`` is updated in place."""
    rc = lib().ecq_encode(ctx, worker, step, _dev(grad, torch.float32, "grad"),
                          _dev(err, torch.float32, "err"), _dev(codes, torch.int32, "codes"),
                          _dev(scales, torch.float32, "scales"), _stream(stream))
    if rc != ECQ_OK:
        raise EcqError(rc, "ecq_encode")


def ecq_encode_batch(ctx: int, step: int, grads: Sequence[torch.Tensor],
                     errs: Sequence[torch.Tensor], codes: Sequence[torch.Tensor],
                     scales: Sequence[torch.Tensor], stream=None) -> None:
    """Enqueue the sender-side kernel for workers 0..len(grads)-1 as one launch.  Each of the
    four arguments is a sequence of tensors or a ``pointer_table`` of them."""
    W = len(grads)
    if not (len(errs) == len(codes) == len(scales) == W):
        raise ValueError("grads, errs, codes and scales must have one entry per worker")
    rc = lib().ecq_encode_batch(ctx, W, step, _table(grads, torch.float32, "grads").array,
                                _table(errs, torch.float32, "errs").array,
                                _table(codes, torch.int32, "codes").array,
                                _table(scales, torch.float32, "scales").array, _stream(stream))
    if rc != ECQ_OK:
        raise EcqError(rc, "ecq_encode_batch")


def ecq_decode_mean(ctx: int, codes: Sequence[torch.Tensor], scales: Sequence[torch.Tensor],
                    out: torch.Tensor, stream=None) -> None:
    """Enqueue the fused receiver-side kernel over ``len(codes)`` messages (sequences of
    tensors or ``pointer_table``s)."""
    W = len(codes)
    if len(scales) != W:
        raise ValueError("codes and scales must have one entry per message")
    cp = _table(codes, torch.int32, "codes").array
    sp = _table(scales, torch.float32, "scales").array
    rc = lib().ecq_decode_mean(ctx, W, cp, sp, _dev(out, torch.float32, "out"), _stream(stream))
    if rc != ECQ_OK:
        raise EcqError(rc, "ecq_decode_mean")


def ecq_decode_mean_update(ctx: int, codes: Sequence[torch.Tensor], scales: Sequence[torch.Tensor],
                           eta: float, params: torch.Tensor, out=None, stream=None) -> None:
    """Receiver-side kernel with ``params <- params - eta * mean`` fused in."""
    W = len(codes)
    if len(scales) != W:
        raise ValueError("codes and scales must have one entry per message")
    cp = _table(codes, torch.int32, "codes").array
    sp = _table(scales, torch.float32, "scales").array
    rc = lib().ecq_decode_mean_update(ctx, W, cp, sp, eta, _dev(params, torch.float32, "params"),
                                      None if out is None else _dev(out, torch.float32, "out"),
                                      _stream(stream))
    if rc != ECQ_OK:
        raise EcqError(rc, "ecq_decode_mean_update")


def ecq_code_histogram(ctx: int, codes: torch.Tensor, counts: torch.Tensor, stream=None) -> None:
    """Fill ``counts`` (int64 CUDA tensor of 2s+1 entries) with the level counts of one message."""
    rc = lib().ecq_code_histogram(ctx, _dev(codes, torch.int32, "codes"),
                                  _dev(counts, torch.int64, "counts"), _stream(stream))
    if rc != ECQ_OK:
        raise EcqError(rc, "ecq_code_histogram")


def ecq_entropy_bound_bits(counts_host) -> float:
    """sum_k d_k log2(d / d_k) from host counts (any integer sequence)."""
    n = len(counts_host)
    arr = (ctypes.c_uint64 * n)(*[int(x) for x in counts_host])
    return float(lib().ecq_entropy_bound_bits(arr, n))


def ecq_step_host_workspace_bytes(ctx: int, W: int) -> int:
    return int(lib().ecq_step_host_workspace_bytes(ctx, W))


def ecq_step_host(ctx: int, step: int, grads_host: Sequence[torch.Tensor], err: torch.Tensor,
                  workspace: torch.Tensor, out_host: torch.Tensor, stream=None) -> None:
    """One iteration from host gradients to a host mean (blocking)."""
    W = len(grads_host)
    for g in grads_host:
        if g.is_cuda or g.dtype != torch.float32 or not g.is_contiguous():
            raise ValueError("grads_host must be contiguous float32 host tensors")
    if out_host.is_cuda or out_host.dtype != torch.float32 or not out_host.is_contiguous():
        raise ValueError("out_host must be a contiguous float32 host tensor")
    gp = (ctypes.c_void_p * W)(*[g.data_ptr() for g in grads_host])
    if not workspace.is_cuda:
        raise ValueError("workspace must be a CUDA tensor")
    rc = lib().ecq_step_host(ctx, W, step, gp, _dev(err, torch.float32, "err"),
                             workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                             out_host.data_ptr(), _stream(stream))
    if rc != ECQ_OK:
        raise EcqError(rc, "ecq_step_host")


def ecq_step_static(d: int, bucket: int, levels: int, alpha: float, beta: float, seed: int,
                    step: int, grads: Sequence[torch.Tensor], err: torch.Tensor,
                    out: torch.Tensor, stream=None) -> int:
    """One iteration (W encodes + decode-mean) that allocates nothing: no context, and the
    messages live in the scratch array built into the library.  For callers that are not
    allowed to allocate device memory (see ``ecq_step_static`` in ecq.h).  Blocking; returns
    the device status (ECQ_OK / ECQ_ERR_NONFINITE / ECQ_ERR_TIMEOUT) and raises on argument
    errors, among them ECQ_ERR_TOO_LARGE when the messages exceed the built-in scratch."""
    W = len(grads)
    if any(g.numel() < d for g in grads) or err.numel() < W * d or out.numel() < d:
        raise ValueError("ecq_step_static: grads need d entries each, err W*d, out d")
    gp = (ctypes.c_void_p * W)(*[_dev(g, torch.float32, "grads") for g in grads])
    rc = lib().ecq_step_static(d, bucket, levels, alpha, beta, seed, W, step, gp,
                               _dev(err, torch.float32, "err"), _dev(out, torch.float32, "out"),
                               _stream(stream))
    if rc not in (ECQ_OK, ECQ_ERR_NONFINITE, ECQ_ERR_TIMEOUT):
        raise EcqError(rc, "ecq_step_static")
    return rc


def ecq_status(ctx: int, stream=None) -> int:
    """Synchronise the stream and return (and clear) the sticky device status."""
    return int(lib().ecq_status(ctx, _stream(stream)))


def ecq_launch_count() -> int:
    return int(lib().ecq_launch_count())


# ---- entropy-coded message ----------------------------------------------------
def _host_u64(counts, n):
    arr = (ctypes.c_uint64 * n)(*[int(x) for x in counts])
    return arr


def ecq_huffman_lengths(ctx: int, counts) -> list:
    """Code-word lengths (host list of 2s+1 ints) from the level counts of a message."""
    n = len(counts)
    c = _host_u64(counts, n)
    out = (ctypes.c_uint8 * n)()
    rc = lib().ecq_huffman_lengths(ctx, c, out)
    if rc != ECQ_OK:
        raise EcqError(rc, "ecq_huffman_lengths")
    return list(out)


def ecq_huffman_chunks(ctx: int) -> int:
    return int(lib().ecq_huffman_chunks(ctx))


def ecq_huffman_stream_bound(ctx: int, counts, lengths) -> int:
    """Stream words that always suffice for a message with these counts and lengths."""
    n = len(counts)
    return int(lib().ecq_huffman_stream_bound(ctx, _host_u64(counts, n),
                                               (ctypes.c_uint8 * n)(*[int(x) for x in lengths])))


def ecq_huffman_tables(ctx: int, lengths, tables: torch.Tensor, stream=None) -> None:
    """Build the tables of the code with these lengths into ``tables`` (uint8 CUDA tensor
    of ECQ_HUFFMAN_TABLE_BYTES)."""
    if tables.numel() < ECQ_HUFFMAN_TABLE_BYTES:
        raise ValueError("tables must hold ECQ_HUFFMAN_TABLE_BYTES bytes")
    n = len(lengths)
    rc = lib().ecq_huffman_tables(ctx, (ctypes.c_uint8 * n)(*[int(x) for x in lengths]),
                                  _dev(tables, torch.uint8, "tables"), _stream(stream))
    if rc != ECQ_OK:
        raise EcqError(rc, "ecq_huffman_tables")


def ecq_huffman_encode(ctx: int, tables: torch.Tensor, codes: torch.Tensor, stream_words: torch.Tensor,
                       offsets: torch.Tensor, quarters: torch.Tensor, stream=None) -> None:
    """Enqueue the entropy coder: ``codes`` -> ``stream_words`` (its size is the capacity),
    ``offsets`` (ecq_huffman_chunks() + 1 words) and ``quarters`` (3 int16 per chunk)."""
    rc = lib().ecq_huffman_encode(ctx, _dev(tables, torch.uint8, "tables"), _dev(codes, torch.int32, "codes"),
                                  _dev(stream_words, torch.int32, "stream_words"), stream_words.numel(),
                                  _dev(offsets, torch.int32, "offsets"),
                                  _dev(quarters, torch.int16, "quarters"), _stream(stream))
    if rc != ECQ_OK:
        raise EcqError(rc, "ecq_huffman_encode")


def ecq_huffman_decode(ctx: int, tables: torch.Tensor, stream_words: torch.Tensor, offsets: torch.Tensor,
                       quarters: torch.Tensor, codes: torch.Tensor, stream=None) -> None:
    """Enqueue the inverse of :func:`ecq_huffman_encode`."""
    rc = lib().ecq_huffman_decode(ctx, _dev(tables, torch.uint8, "tables"),
                                  _dev(stream_words, torch.int32, "stream_words"), stream_words.numel(),
                                  _dev(offsets, torch.int32, "offsets"),
                                  _dev(quarters, torch.int16, "quarters"), _dev(codes, torch.int32, "codes"),
                                  _stream(stream))
    if rc != ECQ_OK:
        raise EcqError(rc, "ecq_huffman_decode")
