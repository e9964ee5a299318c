"""GPU parity: the CUDA codec, called through its C ABI, against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_1806_08054_b200 as ecq
from paper_1806_08054_b200 import workloads as wl

from parity_util import (GpuCodec, SampledOracle, close, codes_np, full_parity, placed_ranges,
                         sample_ranges, whole_message_properties, whole_vector_properties)

pytestmark = pytest.mark.gpu
SEED = wl.CODEC_SEED


def randn_fn(d, scale=0.01, base=0):
    def fn(w, t):
        gen = torch.Generator(device="cuda")
        gen.manual_seed(base + 1000 * t + w)
        return scale * torch.randn(d, generator=gen, device="cuda")
    return fn


# ------------------------------------------------------------ small shapes ---
@pytest.mark.parametrize("s", [1, 2, 4, 8, 16, 64, 128, 300, 32767])
@pytest.mark.parametrize("bucket", [32, 128, 512, 4096, 96, 8192])
def test_small_shapes_every_width(s, bucket):
    # several tiles of the tiled kernel plus a ragged end, and the any-shape path
    sizes = [1, 8, 31, 32, 33, bucket - 1, bucket, bucket + 1, 4096, 3 * 4096 + 5 * 32 + 7]
    if s in (4, 128):
        sizes.append(9 * 4096 + bucket + 40)
    for d in sorted(set(sizes)):
        full_parity(d, bucket, s, 1.0, 0.9, SEED, W=2, steps=2, grad_fn=randn_fn(d, base=d))


@pytest.mark.parametrize("bucket,s", [(512, 4), (2048, 1), (4096, 8), (128, 128), (1024, 2)])
def test_many_tiles_more_than_one_wave(bucket, s):
    # more tiles than resident CTAs so that every ring stage is reused
    d = 4096 * 1500 + 3 * bucket + 24
    full_parity(d, bucket, s, 1.0, 0.9, SEED, W=1, steps=2, grad_fn=randn_fn(d, base=7),
                check_decode=True)


@pytest.mark.parametrize("bucket,s,W", [(512, 4, 4), (4096, 8, 3), (128, 1, 8), (96, 2, 2), (1024, 128, 64)])
def test_batched_encode_is_one_launch_with_the_same_result(bucket, s, W):
    d = 4096 * 7 + 2 * bucket + 12
    before = ecq.ecq_launch_count()
    full_parity(d, bucket, s, 1.0, 0.9, SEED, W=W, steps=2, grad_fn=randn_fn(d, base=W), batch=True)
    launches = ecq.ecq_launch_count() - before
    tiled = (bucket & (bucket - 1)) == 0 and bucket <= 4096
    assert launches == 2 * ((1 if tiled else W) + 1)


def test_alpha_beta_variants_and_mode1():
    d = 4096 * 3 + 777
    for alpha, beta in ((0.0, 0.0), (0.2, 0.9), (0.01, 1.0), (1.0, 0.99), (2.5, 0.5)):
        for mode in (0, 1):
            full_parity(d, 512, 4, alpha, beta, 99, W=2, steps=4, grad_fn=randn_fn(d, base=3),
                        mode=mode, batch=(mode == 1))


def test_worker_step_seed_select_the_stream():
    d, B, s = 8192, 512, 4
    g = randn_fn(d)(0, 0)
    outs = {}
    for seed, worker, step in ((1, 0, 0), (2, 0, 0), (1, 1, 0), (1, 0, 1), (1 << 40, 0, 0)):
        gpu = GpuCodec(d, B, s, 1.0, 0.9, seed, 1)
        ecq.ecq_encode(gpu.ctx, worker, step, g, gpu.err[0][1], gpu.codes[0][1], gpu.scales[0][1])
        assert gpu.status() == 0
        h = np.zeros(d, np.float32)
        c_or, _, _ = oracle.encode(g.cpu().numpy(), h, bucket=B, s=s, alpha=1.0, beta=0.9,
                                   seed=seed, worker=worker, step=step)
        assert np.array_equal(codes_np(gpu.codes[0][1]), c_or)
        outs[(seed, worker, step)] = c_or
        gpu.close()
    vals = list(outs.values())
    for i in range(len(vals)):
        for j in range(i):
            assert not np.array_equal(vals[i], vals[j])


# ------------------------------------------------------------- edge inputs ---
@pytest.mark.parametrize("bucket", [128, 1024, 4096, 96])
def test_degenerate_buckets(bucket):
    d = 4096 * 2 + 3 * bucket + 11
    gen = torch.Generator(device="cuda")
    gen.manual_seed(5)
    g = torch.randn(d, generator=gen, device="cuda")
    h0 = 0.1 * torch.randn(d, generator=gen, device="cuda")
    B = bucket
    g[0:B] = 0; h0[0:B] = 0                       # all-zero bucket
    g[B:2 * B] = 1e-39; h0[B:2 * B] = 0           # denormal bucket: s/scale overflows
    g[2 * B] = -0.0; h0[2 * B] = 0                # negative zero among regular entries
    g[3 * B] = 3.0; g[3 * B + 1] = -3.0; g[3 * B + 2] = 3.0   # ties for the max
    h0[3 * B:3 * B + 3] = 0
    g[4 * B - 1] = 50.0                            # max in the last slot
    g[4 * B] = -60.0                               # max in the first slot
    g[5 * B:6 * B] = 1e-30                         # tiny but regular scale
    g[6 * B: 7 * B] = 1e30                         # huge scale
    full_parity(d, bucket, 4, 1.0, 0.9, SEED, W=1, steps=2, grad_fn=lambda w, t: g, err0=[h0])


@pytest.mark.parametrize("bucket", [512, 4096, 96])
def test_nonfinite_bucket_is_flagged_and_kept(bucket):
    d = 4096 * 2 + bucket + 5
    g = randn_fn(d)(0, 0)
    g[5] = float("nan")
    g[4096 + 7] = float("inf")
    g[d - 1] = float("-inf")
    full_parity(d, bucket, 8, 1.0, 0.9, SEED, W=1, steps=1, grad_fn=lambda w, t: g,
                expect_status=ecq.ECQ_ERR_NONFINITE)
    # the sticky status is cleared by reading it
    gpu = GpuCodec(d, bucket, 8, 1.0, 0.9, SEED, 1)
    gpu.encode(0, 0, g)
    assert gpu.status() == ecq.ECQ_ERR_NONFINITE and gpu.status() == ecq.ECQ_OK
    gpu.close()


def test_decode_worker_counts():
    d, B, s = 4096 * 2 + 100, 512, 4
    for W in (1, 2, 3, 5, 8, 17, 64):
        full_parity(d, B, s, 1.0, 0.9, SEED, W=W, steps=1, grad_fn=randn_fn(d, base=W))


@pytest.mark.parametrize("bucket,s,W,d", [(512, 4, 65, 4096 * 2 + 600), (512, 4, 128, 4096 + 36),
                                            (2048, 1, 150, 4096 * 3 + 24), (96, 8, 70, 3001),
                                            (128, 300, 129, 2500), (32, 2, 66, 4096 + 40),
                                            (4096, 128, 200, 4096 * 2 + 5)])
def test_more_workers_than_one_launch_serves(bucket, s, W, d):
    # beyond 64 messages the receiver sums 64 per launch and carries the running sums in
    # `out`; the sender batches 64 workers per launch.  Same chain of operations as one pass.
    before = ecq.ecq_launch_count()
    full_parity(d, bucket, s, 1.0, 0.9, SEED, W=W, steps=2, grad_fn=randn_fn(d, base=W), batch=True)
    launches = ecq.ecq_launch_count() - before
    chunks = -(-W // ecq.binding.ECQ_MAX_WORKERS)
    tiled = (bucket & (bucket - 1)) == 0 and bucket <= 4096 and d >= 4096
    assert launches == 2 * ((chunks if tiled else W) + chunks)


def test_fused_model_update_with_more_workers_than_one_launch_serves():
    d, bucket, s, W = 4096 * 2 + 77, 512, 4, 100
    gpu = GpuCodec(d, bucket, s, 1.0, 0.9, SEED, W)
    fn = randn_fn(d, base=11)
    grads = [fn(w, 0) for w in range(W)]
    gpu.encode_batch(0, grads)
    msgs = []
    for w in range(W):
        h = np.zeros(d, np.float32)
        c, sc, _ = oracle.encode(grads[w].cpu().numpy(), h, bucket=bucket, s=s, alpha=1.0, beta=0.9,
                                 seed=SEED, worker=w, step=0)
        msgs.append((c, sc))
    gen = torch.Generator(device="cuda"); gen.manual_seed(3)
    p0 = torch.randn(d, generator=gen, device="cuda")
    params = p0.clone()
    codes, scales = [c[1] for c in gpu.codes], [x[1] for x in gpu.scales]
    ecq.ecq_decode_mean_update(gpu.ctx, codes, scales, 0.05, params, gpu.out[1])
    assert gpu.status() == ecq.ECQ_OK
    p_or = p0.cpu().numpy().copy()
    mean = oracle.decode_mean_update([m[0] for m in msgs], [m[1] for m in msgs], p_or, eta=0.05,
                                     bucket=bucket, s=s)
    assert np.array_equal(params.cpu().numpy().view(np.uint32), p_or.view(np.uint32))
    assert np.array_equal(gpu.out[1].cpu().numpy().view(np.uint32), mean.view(np.uint32))
    gpu.check_guards()
    with pytest.raises(ecq.EcqError):       # the running sums need `out` between launches
        ecq.ecq_decode_mean_update(gpu.ctx, codes, scales, 0.05, params, None)
    gpu.close()


@pytest.mark.parametrize("bucket,s,W,d", [(512, 4, 4, 4096 * 5 + 700), (2048, 1, 16, 4096 * 3 + 2048 + 24),
                                            (96, 8, 3, 5000), (128, 300, 2, 3000), (512, 8, 8, 777)])
def test_fused_model_update(bucket, s, W, d):
    # Algorithm 1, last line, fused into the receiver kernel: bit-exact against the oracle
    # (same operations in the same order), with and without the mean being written out
    gpu = GpuCodec(d, bucket, s, 1.0, 0.9, SEED, W)
    fn = randn_fn(d, base=d + W)
    grads = [fn(w, 0) for w in range(W)]
    gpu.encode_batch(0, grads)
    msgs = []
    for w in range(W):
        h = np.zeros(d, np.float32)
        c, sc, _ = oracle.encode(grads[w].cpu().numpy(), h, bucket=bucket, s=s, alpha=1.0, beta=0.9,
                                 seed=SEED, worker=w, step=0)
        msgs.append((c, sc))
    gen = torch.Generator(device="cuda"); gen.manual_seed(3)
    p0 = torch.randn(d, generator=gen, device="cuda")
    for eta, with_out in ((0.02, True), (1.0, False), (0.0, True)):
        params = p0.clone()
        if with_out:
            gpu.out[1].fill_(-7.0)
        ecq.ecq_decode_mean_update(gpu.ctx, [c[1] for c in gpu.codes], [x[1] for x in gpu.scales], eta,
                                   params, gpu.out[1] if with_out else None)
        assert gpu.status() == ecq.ECQ_OK
        p_or = p0.cpu().numpy().copy()
        mean = oracle.decode_mean_update([m[0] for m in msgs], [m[1] for m in msgs], p_or, eta=eta,
                                         bucket=bucket, s=s)
        assert np.array_equal(params.cpu().numpy().view(np.uint32), p_or.view(np.uint32))
        if with_out:
            assert close(gpu.out[1].cpu().numpy(), mean)
    gpu.check_guards()
    L = ecq.binding.lib()
    assert L.ecq_decode_mean_update(gpu.ctx, W, None, None, 0.1, None, None, None) == ecq.ECQ_ERR_ARG
    gpu.close()


@pytest.mark.parametrize("bucket,s,d", [(512, 1, 4096 * 9 + 77), (512, 4, 4096 * 9 + 512 + 40), (96, 8, 5003),
                                        (1024, 16, 33000), (4096, 128, 4096 * 6 + 1), (128, 300, 9000),
                                        (32, 32767, 4099)])
def test_code_histogram_and_entropy(bucket, s, d):
    gpu = GpuCodec(d, bucket, s, 1.0, 0.9, SEED, 1)
    gpu.encode(0, 0, randn_fn(d, base=s)(0, 0))
    counts = torch.full((2 * s + 1,), -1, dtype=torch.int64, device="cuda")
    ecq.ecq_code_histogram(gpu.ctx, gpu.codes[0][1], counts)
    assert gpu.status() == ecq.ECQ_OK
    ref = oracle.code_histogram(codes_np(gpu.codes[0][1]), n=d, s=s)
    got = counts.cpu().numpy()
    assert got.sum() == d and np.array_equal(got.astype(np.uint64), ref)
    bits = ecq.ecq_entropy_bound_bits(got)
    assert abs(bits - oracle.entropy_bound_bits(ref)) <= 1e-9 * max(bits, 1.0)
    assert bits <= d * gpu.r + 1e-6
    gpu.close()


# ------------------------------------------------------------ l2-norm scale ---
@pytest.mark.parametrize("bucket", [32, 128, 512, 2048, 4096, 96, 8192, 32768])
@pytest.mark.parametrize("s", [1, 4, 8, 128])
def test_l2_scale_small_shapes(bucket, s):
    for d in sorted({1, 33, bucket - 1, bucket + 1, 4096, 3 * 4096 + 5 * 32 + 7, 9 * 4096 + bucket + 40}):
        full_parity(d, bucket, s, 1.0, 0.9, SEED, W=2, steps=2, grad_fn=randn_fn(d, base=d), norm=1,
                    batch=(s == 4))


def test_l2_scale_degenerate_and_wide_range_buckets():
    B = 512
    d = 4096 * 2 + 3 * B + 11
    gen = torch.Generator(device="cuda"); gen.manual_seed(6)
    g = torch.randn(d, generator=gen, device="cuda") * torch.pow(
        10.0, torch.empty(d, device="cuda").uniform_(-4, 2, generator=gen))
    h0 = 0.1 * torch.randn(d, generator=gen, device="cuda")
    g[0:B] = 0; h0[0:B] = 0                          # all-zero bucket
    g[B:2 * B] = 1e-25; h0[B:2 * B] = 0              # squares underflow to zero
    g[2 * B:3 * B] = 0; h0[2 * B:3 * B] = 0; g[2 * B + 7] = -2.5      # a single entry
    full_parity(d, B, 4, 1.0, 0.9, SEED, W=1, steps=2, grad_fn=lambda w, t: g, err0=[h0], norm=1)
    g[4096 + 5] = 3e19                                 # the sum of squares overflows
    full_parity(d, B, 4, 1.0, 0.9, SEED, W=1, steps=1, grad_fn=lambda w, t: g, err0=[h0], norm=1,
                expect_status=ecq.ECQ_ERR_NONFINITE)


def test_l2_scale_limits_of_the_any_shape_path():
    ctx = ecq.ecq_create(1 << 20, 65536, 4, 1.0, 0.9, 1)
    with pytest.raises(ecq.EcqError):
        ecq.ecq_set_norm(ctx, 1)
    with pytest.raises(ecq.EcqError):
        ecq.ecq_set_norm(ctx, 2)
    ecq.ecq_set_norm(ctx, 0)
    ecq.ecq_destroy(ctx)


def test_l2_scale_on_resnet50_with_the_papers_cifar_setting():
    # bucket 4096, l2 scale, s = 4, alpha = 0.01, beta = 1.0 (the paper's CIFAR-10 footnote)
    base = wl.WORKLOADS["resnet50"]
    w = wl.Workload(base.name, base.index, 4, base.d, 4096, 4, 0.01, 1.0, 2, base.kind, base.layers)
    ranges = sample_ranges(w.d, w.bucket, seed=9)
    gpu = GpuCodec(w.d, w.bucket, w.s, w.alpha, w.beta, SEED, w.W, norm=1)
    so = SampledOracle(w.d, w.bucket, w.s, w.alpha, w.beta, SEED, w.W, ranges, norm=1)
    for t in range(w.steps):
        gs = [wl.gradient(w, p, t, "cuda") for p in range(w.W)]
        gpu.encode_batch(t, gs)
        for p in range(w.W):
            so.encode_and_compare(gpu, p, t, gs[p])
        gpu.decode(w.W)
        assert gpu.status() == ecq.ECQ_OK
        so.decode_and_compare(gpu)
    gpu.check_guards()
    gpu.close()


def test_one_context_from_two_host_threads_on_two_streams():
    # a context is immutable: concurrent encodes of different workers on different streams
    # give what serial calls give
    import threading
    d, B, s, W = 4096 * 40 + 72, 512, 4, 4
    fn = randn_fn(d, base=31)
    grads = [fn(w, 0) for w in range(W)]
    ref = GpuCodec(d, B, s, 1.0, 0.9, SEED, W)
    for w in range(W):
        ref.encode(w, 0, grads[w])
    par = GpuCodec(d, B, s, 1.0, 0.9, SEED, W)
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream() for _ in range(2)]

    def work(k):
        for rep in range(20):
            for w in range(k, W, 2):
                if rep:
                    par.err[w][1].zero_()
                ecq.ecq_encode(par.ctx, w, 0, grads[w], par.err[w][1], par.codes[w][1],
                               par.scales[w][1], stream=streams[k])
        streams[k].synchronize()

    def zeroing_stream(k):
        with torch.cuda.stream(streams[k]):
            work(k)
    ts = [threading.Thread(target=zeroing_stream, args=(k,)) for k in range(2)]
    [t.start() for t in ts]; [t.join() for t in ts]
    torch.cuda.synchronize()
    assert par.status() == ecq.ECQ_OK
    for w in range(W):
        assert torch.equal(par.codes[w][1], ref.codes[w][1]) and torch.equal(par.err[w][1], ref.err[w][1])
        assert torch.equal(par.scales[w][1], ref.scales[w][1])
    ref.close(); par.close()


def test_argument_errors():
    with pytest.raises(ecq.EcqError):
        ecq.ecq_create(0, 512, 4, 1.0, 0.9, 1)
    for bad in ((100, 48, 4, 1.0, 0.9), (100, 512, 0, 1.0, 0.9), (100, 512, 40000, 1.0, 0.9),
                (100, 512, 4, -1.0, 0.9), (100, 512, 4, 1.0, 1.5), (100, 512, 4, float("nan"), 0.9)):
        with pytest.raises(ecq.EcqError):
            ecq.ecq_create(*bad, 1)
    gpu = GpuCodec(1024, 512, 4, 1.0, 0.9, 1, 1)
    g = torch.zeros(1025, device="cuda")
    with pytest.raises(ecq.EcqError):       # misaligned gradient pointer
        ecq.ecq_encode(gpu.ctx, 0, 0, g[1:], gpu.err[0][1], gpu.codes[0][1], gpu.scales[0][1])
    with pytest.raises(ValueError):         # host tensor: there is no CPU path
        ecq.ecq_encode(gpu.ctx, 0, 0, torch.zeros(1024), gpu.err[0][1], gpu.codes[0][1],
                       gpu.scales[0][1])
    L = ecq.binding.lib()
    assert L.ecq_decode_mean(gpu.ctx, 0, None, None, None, None) == ecq.ECQ_ERR_ARG
    assert L.ecq_decode_mean(gpu.ctx, ecq.binding.ECQ_MAX_WORKERS_TOTAL + 1, None, None, None, None) == ecq.ECQ_ERR_ARG
    gpu.close()


def test_checkpoint_resume_is_bit_identical():
    # the only state is err (+ the caller's step counter)
    d, B, s = 4096 * 4 + 9, 512, 4
    fn = randn_fn(d, base=11)
    a = GpuCodec(d, B, s, 1.0, 0.9, SEED, 1)
    for t in range(10):
        a.encode(0, t, fn(0, t))
    b = GpuCodec(d, B, s, 1.0, 0.9, SEED, 1)
    for t in range(5):
        b.encode(0, t, fn(0, t))
    saved = b.err[0][1].clone()
    b.close()
    c = GpuCodec(d, B, s, 1.0, 0.9, SEED, 1)
    c.err[0][1].copy_(saved)
    for t in range(5, 10):
        c.encode(0, t, fn(0, t))
    assert torch.equal(a.err[0][1], c.err[0][1]) and torch.equal(a.codes[0][1], c.codes[0][1])
    a.close(); c.close()


def test_step_host_matches_device_calls():
    d, B, s, W = 4096 * 6 + 512 + 8, 512, 4, 5
    fn = randn_fn(d, base=21)
    ref = GpuCodec(d, B, s, 1.0, 0.9, SEED, W)
    ctx = ecq.ecq_create(d, B, s, 1.0, 0.9, SEED)
    err = torch.zeros(W * d, device="cuda")
    ws = torch.empty(ecq.ecq_step_host_workspace_bytes(ctx, W), dtype=torch.uint8, device="cuda")
    out_host = torch.empty(d).pin_memory()
    for t in range(3):
        grads = [fn(w, t) for w in range(W)]
        for w in range(W):
            ref.encode(w, t, grads[w])
        ref.decode()
        hosts = [g.cpu().pin_memory() for g in grads]
        ecq.ecq_step_host(ctx, t, hosts, err, ws, out_host)
        assert torch.equal(out_host, ref.out[1].cpu())
        for w in range(W):
            assert torch.equal(err[w * d:(w + 1) * d], ref.err[w][1])
    ecq.ecq_destroy(ctx)
    ref.close()


# --------------------------------------------------- the five configurations --
def test_config1_gauss_1m_every_element():
    w = wl.WORKLOADS["gauss_1m"]
    full_parity(w.d, w.bucket, w.s, w.alpha, w.beta, SEED, w.W, w.steps,
                lambda p, t: wl.gradient(w, p, t, "cuda"))


def _sampled_config(w, steps, W=None, ranges=None, grads=None):
    """Full-size run in the launch configuration bench.py times.  The oracle follows placed
    and random whole-bucket windows of every worker element by element; on the device, over
    the WHOLE vector of EVERY worker: scales against the library max-abs, and after the first
    step the message and the accumulator against what Eq. 6, 8 and 9 fix (levels in range,
    within one level step, accumulator = g - g~), and the decoded mean against the fp64 mean
    of the dequantised messages."""
    W = W or w.W
    ranges = ranges or placed_ranges(w.d, w.bucket, W, seed=w.index)
    gpu = GpuCodec(w.d, w.bucket, w.s, w.alpha, w.beta, SEED, W)
    so = SampledOracle(w.d, w.bucket, w.s, w.alpha, w.beta, SEED, W, ranges)
    try:
        for t in range(steps):
            gs = [grads(p, t) if grads else wl.gradient(w, p, t, "cuda") for p in range(W)]
            before = gpu.err[0][1].clone()
            gpu.encode_batch(t, gs)                 # the launch configuration bench.py times
            if t == 0:
                zero = torch.zeros_like(before)
                for p in range(W):
                    whole_vector_properties(gpu, p, gs[p], zero, w.alpha)
                del zero
            else:
                whole_vector_properties(gpu, 0, gs[0], before, w.alpha)
            del before
            sum64 = None
            if t == 0:
                scratch = torch.empty(w.d, device="cuda")
                sum64 = torch.zeros(w.d, dtype=torch.float64, device="cuda")
                for p in range(W):
                    whole_message_properties(gpu, p, gs[p], w.beta, scratch, sum64)
                del scratch
            for p in range(W):
                so.encode_and_compare(gpu, p, t, gs[p])
            del gs
            gpu.decode(W)
            assert gpu.status() == ecq.ECQ_OK
            if sum64 is not None:
                mean = sum64 / W
                assert bool(((gpu.out[1].double() - mean).abs() <= 1e-7 + 1e-6 * mean.abs()).all()), \
                    "decoded mean is not the mean of the dequantised messages"
                del sum64, mean
            so.decode_and_compare(gpu)
            gpu.check_guards()
    finally:
        gpu.close()
        wl.clear_cache()
        torch.cuda.empty_cache()


def test_config2_lsq_4m():
    w = wl.WORKLOADS["lsq_4m"]
    _sampled_config(w, steps=w.steps)


def test_config3_resnet50():
    w = wl.WORKLOADS["resnet50"]
    _sampled_config(w, steps=w.steps)


def test_config4_alexnet():
    w = wl.WORKLOADS["alexnet"]
    _sampled_config(w, steps=w.steps)


@pytest.mark.parametrize("name", ["resnet50", "alexnet"])
def test_config3_and_4_every_element_of_every_worker(name):
    # one step of the whole configuration against the oracle, element by element, in the
    # launch configuration bench.py times (batched encode, automatic receiver kernel)
    w = wl.WORKLOADS[name]
    full_parity(w.d, w.bucket, w.s, w.alpha, w.beta, SEED, w.W, 1,
                lambda p, t: wl.gradient(w, p, t, "cuda"), batch=True)
    torch.cuda.empty_cache()


@pytest.mark.parametrize("bucket", wl.LM_SWEEP_BUCKETS)
@pytest.mark.parametrize("s", wl.LM_SWEEP_LEVELS)
def test_config5_lm_350m_sweep(bucket, s):
    base = wl.WORKLOADS["lm_350m"]
    w = wl.with_codec(base, bucket, s)
    free, _ = torch.cuda.mem_get_info()
    need = (w.W * w.d * 4) + 4 * w.d * 4 + w.W * w.d * 9 // 8 + 6 * w.d * 4
    if free < need * 1.05:
        pytest.skip("needs %.0f GB of free device memory" % (need / 1e9))
    # four distinct gradient buffers per step; worker p reads buffer p mod 4
    # (its Philox stream and its accumulator are still its own)
    cache = {}

    def grads(p, t):
        key = (p % 4, t)
        if key not in cache:
            for k in [k for k in cache if k[1] != t]:
                del cache[k]
            cache[key] = wl.gradient(w, p % 4, t, "cuda")
        return cache[key]
    steps = w.steps if (bucket, s) == (512, 4) else 1
    _sampled_config(w, steps=steps, grads=grads)
    cache.clear()
    torch.cuda.empty_cache()


@pytest.mark.parametrize("s", [3, 7, 127])
def test_code_width_matched_levels_on_lm_350m(s):
    # the same width-matched quantisers at the benchmark's full size (B = 512, 4 workers)
    w = wl.with_codec(wl.WORKLOADS["lm_350m"], 512, s)
    free, _ = torch.cuda.mem_get_info()
    if free < 4 * w.d * 4 * 3.5:
        pytest.skip("needs %.0f GB of free device memory" % (4 * w.d * 4 * 3.5 / 1e9))
    cache = {}

    def grads(p, t):
        if (p, t) not in cache:
            cache[(p, t)] = wl.gradient(w, p, t, "cuda")
        return cache[(p, t)]
    _sampled_config(w, steps=1, W=4, grads=grads)
    cache.clear()
    torch.cuda.empty_cache()


def test_code_width_matched_levels_on_resnet50():
    # the quantiser whose 2s+1 levels exactly fill b bits: s = 2^(b-1) - 1
    base = wl.WORKLOADS["resnet50"]
    for s in (3, 7, 127):
        _sampled_config(wl.with_codec(base, base.bucket, s), steps=1, W=2)


def test_pointer_tables_give_the_same_launches_as_tensor_lists():
    # the binding marshals a fixed list of tensors once; the calls are the same
    d, bucket, s_, W = 300_000 + 40, 512, 4, 4
    gpu = GpuCodec(d, bucket, s_, 1.0, 0.9, SEED, W)
    gen = torch.Generator(device="cuda"); gen.manual_seed(3)
    grads = [0.01 * torch.randn(d, generator=gen, device="cuda") for _ in range(W)]
    gpu.encode_batch(0, grads)
    gpu.decode()
    want_codes = [c[1].clone() for c in gpu.codes]
    want_err = [e[1].clone() for e in gpu.err]
    want_out = gpu.out[1].clone()
    for e in gpu.err:
        e[1].zero_()
    tg = ecq.pointer_table(grads, torch.float32, "grads")
    te = ecq.pointer_table([e[1] for e in gpu.err], torch.float32, "errs")
    tc = ecq.pointer_table([c[1] for c in gpu.codes], torch.int32, "codes")
    ts = ecq.pointer_table([x[1] for x in gpu.scales], torch.float32, "scales")
    assert len(tc) == W
    for c in gpu.codes:
        c[1].zero_()
    gpu.out[1].zero_()
    ecq.ecq_encode_batch(gpu.ctx, 0, tg, te, tc, ts)
    ecq.ecq_decode_mean(gpu.ctx, tc, ts, gpu.out[1])
    assert gpu.status() == ecq.ECQ_OK
    for w in range(W):
        assert torch.equal(gpu.codes[w][1], want_codes[w])
        assert torch.equal(gpu.err[w][1].view(torch.int32), want_err[w].view(torch.int32))
    assert torch.equal(gpu.out[1].view(torch.int32), want_out.view(torch.int32))
    with pytest.raises(ValueError):
        ecq.ecq_decode_mean(gpu.ctx, ts, ts, gpu.out[1])           # a table of the wrong type
    gpu.check_guards()
    gpu.close()
