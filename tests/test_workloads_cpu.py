"""The seeded input generators: shapes, determinism and the stated value recipes (CPU)."""
import numpy as np
import torch

from paper_1806_08054_b200 import workloads as wl


def test_layer_tables_match_the_architectures():
    assert len(wl.WORKLOADS["resnet50"].layers) == 161 and wl.WORKLOADS["resnet50"].d == 25_557_032
    assert len(wl.WORKLOADS["alexnet"].layers) == 16 and wl.WORKLOADS["alexnet"].d == 61_100_840
    assert wl.WORKLOADS["lm_350m"].d == 24 * (2 * 1024 * 4096 + 1024 * 3072 + 1024 * 1024) + 50257 * 1024
    assert [w.W for w in wl.WORKLOADS.values()] == [4, 8, 8, 16, 32]


def test_gradients_are_deterministic_and_distinct():
    for name in ("gauss_1m", "lsq_4m", "resnet50", "alexnet", "lm_350m"):
        w = wl.scaled(wl.WORKLOADS[name], 20_000)
        a = wl.gradient(w, 1, 2, "cpu")
        b = wl.gradient(w, 1, 2, "cpu")
        c = wl.gradient(w, 2, 2, "cpu")
        e = wl.gradient(w, 1, 3, "cpu")
        assert a.dtype == torch.float32 and a.shape == (20_000,) and torch.isfinite(a).all()
        assert torch.equal(a, b) and not torch.equal(a, c) and not torch.equal(a, e)
    wl.clear_cache()


def test_value_recipes():
    g = wl.gradient(wl.scaled(wl.WORKLOADS["gauss_1m"], 200_000), 0, 0, "cpu").numpy()
    assert abs(g.std() - 0.01) < 2e-4 and abs(g.mean()) < 1e-4
    a = wl.gradient(wl.scaled(wl.WORKLOADS["alexnet"], 400_000), 0, 0, "cpu").numpy()
    assert abs((a == 0).mean() - 0.01) < 2e-3                        # 1 % exact zeros
    assert np.abs(a).max() > 20 * np.median(np.abs(a))              # heavy tails (Student-t, nu = 3)
    o = wl.gradient(wl.scaled(wl.WORKLOADS["lm_350m"], 1_000_000), 0, 0, "cpu").numpy()
    out = np.abs(np.abs(o) - 0.1) < 1e-9
    assert abs(out.mean() - 1e-3) < 3e-4 and abs(o[~out].std() - 1e-3) < 2e-5
    r = wl.gradient(wl.scaled(wl.WORKLOADS["resnet50"], 40_960), 0, 0, "cpu").numpy().reshape(10, 4096)
    sig = r.std(axis=1)
    assert sig.min() > 5e-6 and sig.max() < 2e-2 and sig.max() / sig.min() > 3   # per-layer scales differ
    l = wl.gradient(wl.scaled(wl.WORKLOADS["lsq_4m"], 50_000), 0, 0, "cpu").numpy()
    assert (l == 0).mean() > 0.5                                     # most columns of a sparse X are empty
    wl.clear_cache()


def test_with_codec_and_scaled_keep_the_inputs():
    base = wl.WORKLOADS["lm_350m"]
    v = wl.with_codec(base, 4096, 128)
    assert (v.bucket, v.s, v.d, v.index) == (4096, 128, base.d, base.index)
    assert torch.equal(wl.gradient(wl.scaled(base, 5000), 0, 0, "cpu"),
                       wl.gradient(wl.scaled(v, 5000), 0, 0, "cpu"))


def test_syn_linreg_shapes():
    p = wl.SynLinReg(32, 4, seed=1, n_samples=400, device="cpu")
    g = p.minibatch_gradient(2, torch.zeros(32), batch=16)
    assert g.shape == (32,) and torch.isfinite(g).all() and len(p.shards) == 4
