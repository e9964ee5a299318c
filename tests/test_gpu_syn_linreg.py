"""End-to-end use of the codec on the paper's kind of synthetic linear regression
(Section 6.1): W workers, mini-batch SGD with lr 0.02, gradients exchanged through
ecq_encode_batch and applied with ecq_decode_mean_update.  The paper's qualitative claim is
checked through the kernels: with the same quantiser, error compensation (alpha = 0.2,
beta = 0.9, the paper's setting for these runs) ends closer to the full-precision result
than plain stochastic quantisation (alpha = 0, i.e. QSGD-style)."""
import numpy as np
import pytest
import torch

import paper_1806_08054_b200 as ecq
from paper_1806_08054_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def train(d, seed, alpha, beta, levels, W=4, steps=600, lr=0.02):
    prob = wl.SynLinReg(d, W, seed)
    w = torch.zeros(d, device="cuda")
    if levels == 0:                                   # 32-bit full-precision exchange
        for t in range(steps):
            g = [prob.minibatch_gradient(p, w) for p in range(W)]
            w -= lr * torch.stack(g).mean(0)
        return (w - prob.w_star).norm().item()
    ctx = ecq.ecq_create(d, d, levels, alpha, beta, wl.CODEC_SEED)
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


def test_error_compensation_closes_the_gap_to_full_precision():
    d, seeds = 256, range(4)
    fp32 = np.array([train(d, k, 0.0, 0.0, 0) for k in seeds])
    qsgd = np.array([train(d, k, 0.0, 0.0, 1) for k in seeds])       # alpha = 0: no compensation
    ecq_ = np.array([train(d, k, 0.2, 0.9, 1) for k in seeds])
    assert np.all(fp32 < 0.05) and np.all(qsgd < 0.06)              # everything converges
    assert np.all(ecq_ < qsgd)                                       # in every run
    assert (ecq_ - fp32).mean() < 0.5 * (qsgd - fp32).mean()         # and by a wide margin
