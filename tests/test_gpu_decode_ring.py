"""GPU parity of the receiver kernels by name: the ring kernel (bulk copies shared by a
CTA, tiles of 30720 outputs) and the warp-tiled kernel, each forced through
ecq_set_decode_plan, against the CPU oracle of Eq. 4 -- at sizes with several tiles per
CTA, a partly filled last tile and a ragged end of fewer than 1024 outputs."""
import numpy as np
import pytest
import torch

import oracle
import paper_1806_08054_b200 as ecq
from paper_1806_08054_b200 import workloads as wl

from parity_util import GpuCodec, close, full_parity

pytestmark = pytest.mark.gpu
SEED = wl.CODEC_SEED
TILE = 30720


def randn_fn(d, scale=0.01, base=0):
    def fn(w, t):
        gen = torch.Generator(device="cuda")
        gen.manual_seed(base + 1000 * t + w)
        return scale * torch.randn(d, generator=gen, device="cuda")
    return fn


@pytest.mark.parametrize("bucket,s,W", [(512, 4, 4), (128, 1, 8), (2048, 1, 16), (4096, 8, 3), (1024, 128, 5),
                                        (32, 2, 8), (512, 3, 32), (64, 8, 16), (256, 16, 7), (128, 7, 32),
                                        (8192, 32, 6), (512, 64, 9), (512, 2, 64)])
@pytest.mark.parametrize("max_ctas", [2, 0])
def test_ring_kernel_against_the_oracle(bucket, s, W, max_ctas):
    # two CTAs walk six tiles (every ring stage is reused); the last tile holds 3 of its 30
    # sub-tiles, and 100 outputs are left for the one-thread-per-output end
    d = TILE * 5 + 1024 * 3 + 100
    full_parity(d, bucket, s, 1.0, 0.9, SEED, W=W, steps=2, grad_fn=randn_fn(d, base=W + bucket),
                batch=True, decode_plan=(ecq.ECQ_DECODE_RING, max_ctas))


@pytest.mark.parametrize("d", [1024, 1024 + 5, 1024 * 8, 1024 * 17 + 31, TILE, TILE + 1024 * 29 + 1023, 1000])
def test_ring_kernel_short_vectors(d):
    # from one sub-tile up; d < 1024 has no tile at all and takes another kernel
    for bucket, s, W in ((512, 4, 4), (1024, 1, 3)):
        full_parity(d, bucket, s, 1.0, 0.9, SEED, W=W, steps=1, grad_fn=randn_fn(d, base=d),
                    decode_plan=(ecq.ECQ_DECODE_RING, 0))


@pytest.mark.parametrize("bucket,s,W", [(512, 4, 100), (2048, 1, 130), (128, 8, 65)])
def test_ring_kernel_carries_running_sums_beyond_64_workers(bucket, s, W):
    d = TILE * 2 + 1024 * 9 + 77
    full_parity(d, bucket, s, 1.0, 0.9, SEED, W=W, steps=1, grad_fn=randn_fn(d, base=W),
                batch=True, decode_plan=(ecq.ECQ_DECODE_RING, 3))


@pytest.mark.parametrize("plan", [(ecq.ECQ_DECODE_RING, 2), (ecq.ECQ_DECODE_WARP, 0), (ecq.ECQ_DECODE_AUTO, 0)])
def test_fused_model_update_in_every_kernel(plan):
    d, bucket, s, W = TILE * 3 + 1024 * 5 + 300, 512, 4, 6
    gpu = GpuCodec(d, bucket, s, 1.0, 0.9, SEED, W, decode_plan=plan)
    fn = randn_fn(d, base=23)
    grads = [fn(w, 0) for w in range(W)]
    gpu.encode_batch(0, grads)
    msgs = []
    for w in range(W):
        h = np.zeros(d, np.float32)
        c, sc, _ = oracle.encode(grads[w].cpu().numpy(), h, bucket=bucket, s=s, alpha=1.0, beta=0.9,
                                 seed=SEED, worker=w, step=0)
        msgs.append((c, sc))
    gen = torch.Generator(device="cuda"); gen.manual_seed(5)
    p0 = torch.randn(d, generator=gen, device="cuda")
    params = p0.clone()
    ecq.ecq_decode_mean_update(gpu.ctx, [c[1] for c in gpu.codes], [x[1] for x in gpu.scales], 0.05,
                               params, gpu.out[1])
    assert gpu.status() == ecq.ECQ_OK
    p_or = p0.cpu().numpy().copy()
    mean = oracle.decode_mean_update([m[0] for m in msgs], [m[1] for m in msgs], p_or, eta=0.05,
                                     bucket=bucket, s=s)
    assert close(gpu.out[1].cpu().numpy(), mean)
    assert close(params.cpu().numpy(), p_or)
    gpu.check_guards()
    gpu.close()


def test_scales_near_one_stay_within_tolerance():
    # level steps of order one are where a reordered sum would leave the absolute tolerance
    d, bucket, s, W = TILE * 2 + 1024 + 17, 1024, 2, 8
    full_parity(d, bucket, s, 1.0, 0.95, SEED, W=W, steps=2, grad_fn=randn_fn(d, scale=0.7, base=1),
                decode_plan=(ecq.ECQ_DECODE_RING, 2))


@pytest.mark.parametrize("scale", [1e30, 1e-33])
@pytest.mark.parametrize("plan", [(ecq.ECQ_DECODE_RING, 2), (ecq.ECQ_DECODE_WARP, 0)])
def test_very_large_and_very_small_gradients(scale, plan):
    # the kernels carry the level steps times 2^-22 / W: sums near the top of the fp32 range must
    # not overflow on the way, and level steps that fall below the normal range may lose bits
    # only far under the absolute tolerance
    d, bucket, s, W = TILE * 2 + 1024 * 7 + 3, 512, 4, 8
    full_parity(d, bucket, s, 1.0, 0.9, SEED, W=W, steps=1, grad_fn=randn_fn(d, scale=scale, base=9),
                decode_plan=plan)


def test_every_kernel_gives_the_same_bits_on_a_long_vector():
    # any size: the kernels sum in the same order, so their outputs are bit-identical
    w = wl.WORKLOADS["resnet50"]
    d, W = w.d, w.W
    outs = []
    for plan in ((ecq.ECQ_DECODE_WARP, 0), (ecq.ECQ_DECODE_RING, 0), (ecq.ECQ_DECODE_AUTO, 0)):
        gpu = GpuCodec(d, w.bucket, w.s, w.alpha, w.beta, SEED, W, decode_plan=plan)
        gpu.encode_batch(0, [wl.gradient(w, p, 0, "cuda") for p in range(W)])
        gpu.decode()
        assert gpu.status() == ecq.ECQ_OK
        gpu.check_guards()
        outs.append(gpu.out[1].clone())
        gpu.close()
    assert torch.equal(outs[0].view(torch.int32), outs[1].view(torch.int32))
    assert torch.equal(outs[0].view(torch.int32), outs[2].view(torch.int32))


@pytest.mark.parametrize("bucket,s,W", [(512, 4, 16), (512, 1, 8), (4096, 8, 12)])
def test_automatic_choice_gives_the_same_bits_on_vectors_of_a_few_tiles_per_cta(bucket, s, W):
    # 5.6 ring tiles per CTA: with this many messages of these widths the automatic choice takes
    # the ring kernel, with fewer or wider ones the warp-tiled kernel; the bits are the same,
    # ragged end of 40 outputs included
    d = wl.WORKLOADS["resnet50"].d
    fn = randn_fn(d, base=3 * W + s)
    grads = [fn(w, 0) for w in range(W)]
    outs = []
    for plan in ((ecq.ECQ_DECODE_WARP, 0), (ecq.ECQ_DECODE_RING, 0), (ecq.ECQ_DECODE_AUTO, 0)):
        gpu = GpuCodec(d, bucket, s, 1.0, 0.9, SEED, W, decode_plan=plan)
        gpu.encode_batch(0, grads)
        gpu.decode()
        assert gpu.status() == ecq.ECQ_OK
        gpu.check_guards()
        outs.append(gpu.out[1].clone())
        gpu.close()
    assert torch.equal(outs[0].view(torch.int32), outs[1].view(torch.int32))
    assert torch.equal(outs[0].view(torch.int32), outs[2].view(torch.int32))


def test_plan_argument_errors():
    ctx = ecq.ecq_create(4096, 512, 4, 1.0, 0.9, SEED)
    with pytest.raises(ecq.EcqError):
        ecq.ecq_set_decode_plan(ctx, 3, 0)
    with pytest.raises(ecq.EcqError):
        ecq.ecq_set_decode_plan(ctx, -1, 0)
    ecq.ecq_set_decode_plan(ctx, ecq.ECQ_DECODE_AUTO, 0)
    ecq.ecq_destroy(ctx)


@pytest.mark.parametrize("bucket,s,W", [(32, 2, 8), (32, 8, 8), (64, 1, 16), (512, 4, 32)])
def test_ring_kernel_repeated_on_one_context(bucket, s, W):
    # the same launch many times over: a stage handed back before its words were read, or read
    # before they had landed, shows as a few wrong rows in some repetition
    d = TILE * 7 + 1024 * 11 + 5
    gpu = GpuCodec(d, bucket, s, 1.0, 0.9, SEED, W, decode_plan=(ecq.ECQ_DECODE_RING, 3))
    fn = randn_fn(d, base=77)
    grads = [fn(w, 0) for w in range(W)]
    gpu.encode_batch(0, grads)
    msgs = []
    for w in range(W):
        h = np.zeros(d, np.float32)
        c, sc, _ = oracle.encode(grads[w].cpu().numpy(), h, bucket=bucket, s=s, alpha=1.0, beta=0.9,
                                 seed=SEED, worker=w, step=0)
        msgs.append((c, sc))
    mean = oracle.decode_mean([m[0] for m in msgs], [m[1] for m in msgs], n=d, bucket=bucket, s=s)
    want = torch.from_numpy(mean).cuda()
    for rep in range(40):
        gpu.out[1].fill_(-7.0)
        gpu.decode()
        assert torch.equal(gpu.out[1].view(torch.int32), want.view(torch.int32)), "repetition %d" % rep
    assert gpu.status() == ecq.ECQ_OK
    gpu.check_guards()
    gpu.close()


def test_output_that_is_only_16_byte_aligned_takes_another_kernel():
    # the ring kernel stores 32 bytes at a time; the interface only asks for 16-byte alignment
    d, bucket, s, W = TILE * 2 + 1024 * 3 + 9, 512, 4, 4
    gpu = GpuCodec(d, bucket, s, 1.0, 0.9, SEED, W, decode_plan=(ecq.ECQ_DECODE_RING, 0))
    fn = randn_fn(d, base=41)
    grads = [fn(w, 0) for w in range(W)]
    gpu.encode_batch(0, grads)
    msgs = []
    for w in range(W):
        h = np.zeros(d, np.float32)
        c, sc, _ = oracle.encode(grads[w].cpu().numpy(), h, bucket=bucket, s=s, alpha=1.0, beta=0.9,
                                 seed=SEED, worker=w, step=0)
        msgs.append((c, sc))
    buf = torch.full((d + 16,), -3.0, device="cuda")
    out = buf[4:4 + d]
    assert out.data_ptr() % 32 == 16
    ecq.ecq_decode_mean(gpu.ctx, [c[1] for c in gpu.codes], [x[1] for x in gpu.scales], out)
    assert gpu.status() == ecq.ECQ_OK
    mean = oracle.decode_mean([m[0] for m in msgs], [m[1] for m in msgs], n=d, bucket=bucket, s=s)
    assert close(out.cpu().numpy(), mean)
    assert torch.all(buf[:4] == -3.0) and torch.all(buf[4 + d:] == -3.0)
    gpu.close()
