"""The bounded in-kernel waits at work, without any fault: with the context's poll limit set
to zero every wait for an asynchronous copy gives up at once while the copy is still on its
way.  The kernel must then stop, report ECQ_ERR_TIMEOUT through the sticky status word, let
the copies in flight land (that last wait keeps the built-in limit) and leave the context
usable: the same call with the default limit is then checked against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_1806_08054_b200 as ecq
from paper_1806_08054_b200 import workloads as wl

from parity_util import GpuCodec, close, codes_np

pytestmark = pytest.mark.gpu
SEED = wl.CODEC_SEED


def _grads(d, W, base):
    out = []
    for w in range(W):
        gen = torch.Generator(device="cuda")
        gen.manual_seed(base + w)
        out.append(0.01 * torch.randn(d, generator=gen, device="cuda"))
    return out


def _oracle_messages(grads, d, bucket, s):
    msgs, hs = [], []
    for w, g in enumerate(grads):
        h = np.zeros(d, np.float32)
        c, sc, _ = oracle.encode(g.cpu().numpy(), h, bucket=bucket, s=s, alpha=1.0, beta=0.9,
                                 seed=SEED, worker=w, step=0)
        msgs.append((c, sc))
        hs.append(h)
    return msgs, hs


@pytest.mark.parametrize("bucket,s", [(512, 4), (128, 1), (4096, 8)])
def test_tiled_encode_gives_up_and_recovers(bucket, s):
    d, W = 8192 * 40 + 4096 + 512 + 40, 4           # whole tiles of both shapes and a ragged end
    gpu = GpuCodec(d, bucket, s, 1.0, 0.9, SEED, W)
    grads = _grads(d, W, 300)
    ecq.ecq_set_wait_limit(gpu.ctx, 0)
    gpu.encode_batch(0, grads)
    assert gpu.status() == ecq.ECQ_ERR_TIMEOUT
    gpu.check_guards()
    assert gpu.status() == ecq.ECQ_OK               # the status word was cleared by the read
    # nothing was booked: the accumulators of the whole tiles are untouched
    for w in range(W):
        assert torch.count_nonzero(gpu.err[w][1][:8192 * 40]) == 0
    ecq.ecq_set_wait_limit(gpu.ctx, ecq.ECQ_WAIT_LIMIT_DEFAULT)
    for w in range(W):
        gpu.err[w][1].zero_()
    gpu.encode_batch(0, grads)
    assert gpu.status() == ecq.ECQ_OK
    msgs, hs = _oracle_messages(grads, d, bucket, s)
    for w in range(W):
        assert np.array_equal(codes_np(gpu.codes[w][1]), msgs[w][0])
        assert np.array_equal(gpu.scales[w][1].cpu().numpy(), msgs[w][1])
        assert close(gpu.err[w][1].cpu().numpy(), hs[w])
    gpu.check_guards()
    gpu.close()


@pytest.mark.parametrize("bucket,s,W", [(512, 4, 6), (2048, 1, 16), (4096, 8, 3)])
def test_ring_decode_gives_up_and_recovers(bucket, s, W):
    d = 30720 * 7 + 1024 * 5 + 33
    gpu = GpuCodec(d, bucket, s, 1.0, 0.9, SEED, W, decode_plan=(ecq.ECQ_DECODE_RING, 3))
    grads = _grads(d, W, 500)
    gpu.encode_batch(0, grads)
    assert gpu.status() == ecq.ECQ_OK
    ecq.ecq_set_wait_limit(gpu.ctx, 0)
    gpu.decode()
    assert gpu.status() == ecq.ECQ_ERR_TIMEOUT
    gpu.check_guards()
    # again, to see that a launch which gave up leaves nothing behind that trips the next one
    gpu.decode()
    assert gpu.status() == ecq.ECQ_ERR_TIMEOUT
    ecq.ecq_set_wait_limit(gpu.ctx, ecq.ECQ_WAIT_LIMIT_DEFAULT)
    gpu.decode()
    assert gpu.status() == ecq.ECQ_OK
    msgs, _ = _oracle_messages(grads, d, bucket, s)
    mean = oracle.decode_mean([m[0] for m in msgs], [m[1] for m in msgs], n=d, bucket=bucket, s=s)
    assert close(gpu.out[1].cpu().numpy(), mean)
    gpu.check_guards()
    gpu.close()


def test_argument_check():
    with pytest.raises(ecq.EcqError):
        ecq.ecq_set_wait_limit(0, 5)
