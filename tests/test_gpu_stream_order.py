"""Stream order between the library's own kernels.

The persistent kernels are launched so that a launch may be scheduled while its predecessor in
the stream is still draining (programmatic dependent launch); each waits for the predecessor
to complete before its first global access.  These tests enqueue several whole iterations
(Algorithm 1: encode, then decode + model update) back to back on one stream with no host
synchronisation, re-using the same message buffers every step, so that a sender kernel that
started writing before the receiver kernel ahead of it had read the messages (or a receiver
that read before the sender had written) would change the result.  The oracle replays the
loop; parameters, accumulators and the last messages must match bit for bit.
"""
from __future__ import annotations

import numpy as np
import pytest
import torch

import oracle
import paper_1806_08054_b200 as ecq
from parity_util import GpuCodec, codes_np

pytestmark = pytest.mark.gpu

SEED = 99


@pytest.mark.parametrize("kernel", [ecq.ECQ_DECODE_WARP, ecq.ECQ_DECODE_RING])
def test_iterations_enqueued_back_to_back(kernel):
    # long enough for every launch to fill the GPU (148 ring tiles of 30720 outputs and more
    # warp tiles than 2 CTAs x 8 warps per SM), with a ragged end
    d, bucket, s, W, T, eta = 148 * 30720 + 5000, 512, 4, 3, 5, 0.05
    gpu = GpuCodec(d, bucket, s, 1.0, 0.9, SEED, W, decode_plan=(kernel, 0))
    gen = torch.Generator(device="cuda")
    gen.manual_seed(5)
    grads = [[0.01 * torch.randn(d, generator=gen, device="cuda") for _ in range(W)] for _ in range(T)]
    p0 = torch.randn(d, generator=gen, device="cuda")
    params = p0.clone()
    errs = [e[1] for e in gpu.err]
    codes, scales = [c[1] for c in gpu.codes], [x[1] for x in gpu.scales]
    t_g = [ecq.pointer_table(g, torch.float32, "grads") for g in grads]
    t_h = ecq.pointer_table(errs, torch.float32, "errs")
    t_c, t_s = ecq.pointer_table(codes, torch.int32, "codes"), ecq.pointer_table(scales, torch.float32, "scales")
    torch.cuda.synchronize()
    n0 = ecq.ecq_launch_count()
    for t in range(T):
        ecq.ecq_encode_batch(gpu.ctx, t, t_g[t], t_h, t_c, t_s)
        ecq.ecq_decode_mean_update(gpu.ctx, t_c, t_s, eta, params, gpu.out[1])
    assert ecq.ecq_launch_count() - n0 == 2 * T
    assert gpu.status() == ecq.ECQ_OK

    p_or = p0.cpu().numpy().copy()
    h_or = [np.zeros(d, np.float32) for _ in range(W)]
    for t in range(T):
        msgs = [oracle.encode(grads[t][w].cpu().numpy(), h_or[w], bucket=bucket, s=s, alpha=1.0, beta=0.9,
                              seed=SEED, worker=w, step=t) for w in range(W)]
        mean = oracle.decode_mean_update([m[0] for m in msgs], [m[1] for m in msgs], p_or, eta=eta,
                                         bucket=bucket, s=s)
    assert np.array_equal(params.cpu().numpy().view(np.uint32), p_or.view(np.uint32))
    assert np.array_equal(gpu.out[1].cpu().numpy().view(np.uint32), mean.view(np.uint32))
    for w in range(W):
        assert np.array_equal(codes_np(codes[w]), msgs[w][0])
        assert np.array_equal(scales[w].cpu().numpy().view(np.uint32), msgs[w][1].view(np.uint32))
        assert np.array_equal(errs[w].cpu().numpy().view(np.uint32), h_or[w].view(np.uint32))
    gpu.check_guards()
    gpu.close()
