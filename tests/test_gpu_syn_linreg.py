"""End-to-end use of the codec on the paper's kind of synthetic linear regression
(Section 6.1, the Syn-256 / Syn-512 / Syn-1024 runs): 10k samples split over W workers,
mini-batch SGD with learning rate 0.02, gradients exchanged through ecq_encode_batch and
applied with ecq_decode_mean_update.  Three arms as in the paper: 32-bit exchange, plain
stochastic quantisation (alpha = 0, the special case the paper identifies with QSGD) and
error compensation with the paper's setting for these runs (l2-norm scale over the whole
vector, s = 4, alpha = 0.2, beta = 0.9).  The paper's curves are in a figure the source
does not contain; its qualitative claim -- the distance to the optimum of the compensated
run stays closer to the full-precision run than the uncompensated one -- is what is
checked.  The loop is also followed by the CPU oracle, step by step and element by element."""
import numpy as np
import pytest
import torch

import oracle
import paper_1806_08054_b200 as ecq
from paper_1806_08054_b200 import workloads as wl

from parity_util import close, codes_np

pytestmark = pytest.mark.gpu
L_INF, L2 = 0, 1


def train(d, seed, alpha, beta, levels, norm=L2, W=4, steps=600, lr=0.02):
    prob = wl.SynLinReg(d, W, seed)
    w = torch.zeros(d, device="cuda")
    if levels == 0:                                   # 32-bit full-precision exchange
        for t in range(steps):
            g = [prob.minibatch_gradient(p, w) for p in range(W)]
            w -= lr * torch.stack(g).mean(0)
        return (w - prob.w_star).norm().item()
    ctx = ecq.ecq_create(d, d, levels, alpha, beta, wl.CODEC_SEED)   # one scale for the whole vector
    ecq.ecq_set_norm(ctx, norm)
    nw, nb = ecq.ecq_codes_words(ctx), ecq.ecq_num_buckets(ctx)
    errs = [torch.zeros(d, device="cuda") for _ in range(W)]
    codes = [torch.zeros(nw, dtype=torch.int32, device="cuda") for _ in range(W)]
    scales = [torch.zeros(nb, device="cuda") for _ in range(W)]
    for t in range(steps):
        g = [prob.minibatch_gradient(p, w) for p in range(W)]
        ecq.ecq_encode_batch(ctx, t, g, errs, codes, scales)
        ecq.ecq_decode_mean_update(ctx, codes, scales, lr, w)
    assert ecq.ecq_status(ctx) == ecq.ECQ_OK
    ecq.ecq_destroy(ctx)
    return (w - prob.w_star).norm().item()


@pytest.mark.parametrize("d", [256, 512, 1024])
def test_papers_setting_error_compensation_closes_the_gap(d):
    seeds = range(4)
    fp32 = np.array([train(d, k, 0.0, 0.0, 0) for k in seeds])
    qsgd = np.array([train(d, k, 0.0, 0.0, 4) for k in seeds])       # alpha = 0: no compensation
    ecq_ = np.array([train(d, k, 0.2, 0.9, 4) for k in seeds])
    print("d=%d  |w-w*|: 32-bit %s  alpha=0 %s  alpha=0.2 %s" % (d, fp32.round(4), qsgd.round(4), ecq_.round(4)))
    assert np.all(fp32 < 0.1) and np.all(qsgd < 0.3) and np.all(ecq_ < 0.3)   # everything converges
    assert np.all(ecq_ < qsgd)                                                # in every run
    assert (ecq_ - fp32).mean() < 0.6 * (qsgd - fp32).mean()                  # the gap shrinks by a margin


def test_ternary_levels_with_the_max_abs_scale():
    # the coarsest quantiser (s = 1, l-infinity scale): the same claim, in every run
    d, seeds = 256, range(4)
    fp32 = np.array([train(d, k, 0.0, 0.0, 0) for k in seeds])
    qsgd = np.array([train(d, k, 0.0, 0.0, 1, norm=L_INF) for k in seeds])
    ecq_ = np.array([train(d, k, 0.2, 0.9, 1, norm=L_INF) for k in seeds])
    assert np.all(fp32 < 0.05) and np.all(qsgd < 0.06)
    assert np.all(ecq_ < qsgd)
    assert (ecq_ - fp32).mean() < 0.5 * (qsgd - fp32).mean()


@pytest.mark.parametrize("alpha,beta", [(0.2, 0.9), (0.0, 0.0)])
def test_the_loop_against_the_oracle_step_by_step(alpha, beta):
    # 20 iterations on Syn-256 in the paper's setting; both sides get the same mini-batch
    # gradients (computed from the GPU's parameters) and are compared after every step:
    # codes and scales bit for bit, accumulators and parameters within 1e-7 + 1e-6 |y|
    d, W, s, lr, steps = 256, 4, 4, 0.02, 20
    prob = wl.SynLinReg(d, W, 11)
    ctx = ecq.ecq_create(d, d, s, alpha, beta, wl.CODEC_SEED)
    ecq.ecq_set_norm(ctx, L2)
    nw, nb = ecq.ecq_codes_words(ctx), ecq.ecq_num_buckets(ctx)
    w_gpu = torch.zeros(d, device="cuda")
    errs = [torch.zeros(d, device="cuda") for _ in range(W)]
    codes = [torch.zeros(nw, dtype=torch.int32, device="cuda") for _ in range(W)]
    scales = [torch.zeros(nb, device="cuda") for _ in range(W)]
    w_or = np.zeros(d, np.float32)
    h_or = [np.zeros(d, np.float32) for _ in range(W)]
    for t in range(steps):
        g = [prob.minibatch_gradient(p, w_gpu) for p in range(W)]
        ecq.ecq_encode_batch(ctx, t, g, errs, codes, scales)
        ecq.ecq_decode_mean_update(ctx, codes, scales, lr, w_gpu)
        assert ecq.ecq_status(ctx) == ecq.ECQ_OK
        msgs = []
        for p in range(W):
            c, sc, _ = oracle.encode(g[p].cpu().numpy(), h_or[p], bucket=d, s=s, alpha=alpha, beta=beta,
                                     seed=wl.CODEC_SEED, worker=p, step=t, norm=L2)
            assert np.array_equal(codes_np(codes[p]), c), "codes differ (worker %d, step %d)" % (p, t)
            assert np.array_equal(scales[p].cpu().numpy().view(np.uint32), sc.view(np.uint32))
            assert close(errs[p].cpu().numpy(), h_or[p]), "accumulator differs (worker %d, step %d)" % (p, t)
            msgs.append((c, sc))
        oracle.decode_mean_update([m[0] for m in msgs], [m[1] for m in msgs], w_or, eta=lr, bucket=d, s=s)
        assert close(w_gpu.cpu().numpy(), w_or), "parameters differ (step %d)" % t
        # the next gradients come from the GPU's parameters on both sides
        w_or = w_gpu.cpu().numpy().copy()
    ecq.ecq_destroy(ctx)
