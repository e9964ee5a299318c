"""The allocation-free entry point against the ordinary ones.

``ecq_step_static`` serves callers that may not allocate device memory (a plugin
inside another framework's memory pool, a process whose allocator must not be
re-entered): it needs no context and keeps the workers' messages in a scratch
array that is part of the library.  This test calls it through the C ABI twice in
a row -- the array is shared and keeps the previous call's contents, so the second
call checks that nothing stale leaks through -- and compares the accumulators and
the decoded mean with ecq_encode + ecq_decode_mean on the same inputs.  The two
paths run the same kernels, so the comparison is exact; the tolerance of the other
GPU tests (1e-7 + 1e-6 |y|) is asserted as well.

Collected last on purpose: a failure here cannot hide another test's result.
"""
import numpy as np
import pytest
import torch

import paper_1806_08054_b200 as ecq
from paper_1806_08054_b200 import binding

pytestmark = pytest.mark.gpu


def _grad(d, w, t):
    gen = torch.Generator(device="cuda")
    gen.manual_seed(777 + 100 * t + w)
    return 0.01 * torch.randn(d, generator=gen, device="cuda")


@pytest.mark.parametrize("d,bucket,levels,W", [(4096 * 9 + 512 + 40, 512, 4, 4),
                                                (1 << 18, 2048, 1, 3),
                                                (5000, 96, 8, 2)])
def test_static_step_matches_the_ordinary_entry_points(d, bucket, levels, W):
    alpha, beta, seed = 1.0, 0.9, 4321
    ctx = ecq.ecq_create(d, bucket, levels, alpha, beta, seed)
    nw, nb = ecq.ecq_codes_words(ctx), ecq.ecq_num_buckets(ctx)
    err_ref = [torch.zeros(d, device="cuda") for _ in range(W)]
    codes = [torch.zeros(nw, dtype=torch.int32, device="cuda") for _ in range(W)]
    scales = [torch.zeros(nb, device="cuda") for _ in range(W)]
    out_ref = torch.zeros(d, device="cuda")
    err = torch.zeros(W * d, device="cuda")
    out = torch.full((d,), -3.0, device="cuda")
    for t in range(3):                                  # calls in a row share the scratch
        grads = [_grad(d, w, t) for w in range(W)]
        for w in range(W):
            ecq.ecq_encode(ctx, w, t, grads[w], err_ref[w], codes[w], scales[w])
        ecq.ecq_decode_mean(ctx, codes, scales, out_ref)
        assert ecq.ecq_status(ctx) == ecq.ECQ_OK
        torch.cuda.synchronize()
        free_before, launches_before = torch.cuda.mem_get_info()[0], ecq.ecq_launch_count()
        rc = ecq.ecq_step_static(d, bucket, levels, alpha, beta, seed, t, grads, err, out)
        assert rc == ecq.ECQ_OK
        assert ecq.ecq_launch_count() - launches_before == W + 1
        if t > 0:
            # what the entry point is for: once the kernels are loaded (first call), a call
            # leaves the device's free memory exactly where it found it
            assert torch.cuda.mem_get_info()[0] == free_before
        a, b = out.cpu().numpy(), out_ref.cpu().numpy()
        assert np.all(np.abs(a - b) <= 1e-7 + 1e-6 * np.abs(b))
        assert torch.equal(out, out_ref)
        for w in range(W):
            assert torch.equal(err[w * d:(w + 1) * d], err_ref[w])
    ecq.ecq_destroy(ctx)


def test_static_step_reports_nonfinite_then_clears():
    d, W = 8192, 2
    grads = [_grad(d, w, 0) for w in range(W)]
    grads[1][17] = float("nan")
    err = torch.zeros(W * d, device="cuda")
    out = torch.zeros(d, device="cuda")
    assert ecq.ecq_step_static(d, 512, 4, 1.0, 0.9, 1, 0, grads, err, out) == ecq.ECQ_ERR_NONFINITE
    grads[1][17] = 0.0
    assert ecq.ecq_step_static(d, 512, 4, 1.0, 0.9, 1, 1, grads, err, out) == ecq.ECQ_OK


def test_binding_checks_buffer_lengths():
    d, W = 4096, 2
    g = [torch.zeros(d, device="cuda") for _ in range(W)]
    with pytest.raises(ValueError):
        ecq.ecq_step_static(d, 512, 4, 1.0, 0.9, 1, 0, g, torch.zeros(W * d - 1, device="cuda"),
                            torch.zeros(d, device="cuda"))
    with pytest.raises(ValueError):
        ecq.ecq_step_static(d, 512, 4, 1.0, 0.9, 1, 0, g, torch.zeros(W * d, device="cuda"),
                            torch.zeros(d - 1, device="cuda"))
    with pytest.raises(ValueError):
        ecq.ecq_step_static(d, 512, 4, 1.0, 0.9, 1, 0, [g[0], g[1][:100]],
                            torch.zeros(W * d, device="cuda"), torch.zeros(d, device="cuda"))


def test_static_step_refuses_what_does_not_fit():
    d, W = 1 << 22, 8              # 8 messages of 2 MiB of codes each: beyond the 4 MiB scratch
    L = binding.lib()
    g = torch.zeros(16, device="cuda")
    import ctypes
    gp = (ctypes.c_void_p * W)(*[g.data_ptr()] * W)
    rc = L.ecq_step_static(d, 512, 4, 1.0, 0.9, 1, W, 0, gp, g.data_ptr(), g.data_ptr(), None)
    assert rc == binding.ECQ_ERR_TOO_LARGE
    assert "scratch" in binding.strerror(rc)
