"""rad_mlp_step against the oracle on the MNIST-shaped nets and the bf16 cut of the wide net."""
import numpy as np
import pytest
import torch

from oracle import rad as orc
from workloads import get_config, mlp_inputs

from gpu_util import TOL, rel_err, to_dev, to_host_f32

pytestmark = pytest.mark.gpu


def _run(cfg, variant, p, seed, act=None, step=0, law="bernoulli"):
    import paper_2007_10412_b200 as rad
    act = act or cfg.act
    X, y, Ws, bs = mlp_inputs(cfg.dims, cfg.batch, cfg.dtype, cfg.x_dist, cfg.data_seed, bias_zero=False)
    ctx = rad.MLPStep(cfg.dims, cfg.batch, cfg.dtype, act, variant, p, law=law)
    dX = to_dev(X, cfg.dtype)
    dy = torch.from_numpy(y).cuda()
    dWs = [to_dev(W, cfg.dtype) for W in Ws]
    dbs = [to_dev(b, "f32") for b in bs]
    ctx(dX, dy, dWs, dbs, seed=seed, step=step)
    torch.cuda.synchronize()
    assert ctx.dev_status.item() == 0
    ref = orc.mlp_step(X, y, Ws, bs, act=act, dtype=cfg.dtype, variant=variant, p=p, seed=seed, step=step, law=law)
    return ctx, ref, (X, y, Ws, bs)


@pytest.mark.parametrize("name,variant", [("mlp_small_different", "different"), ("mlp_small_same", "same"),
                                          ("mlp_wide_cut", "different"), ("mlp_wide_cut", "same")])
@pytest.mark.parametrize("law", ["replace", "fixed"])
def test_step_with_the_other_sampling_laws_matches_oracle(name, variant, law):
    """The whole step with the paper's own sampling law (k = ceil(0.1 d) draws with replacement per layer
    input) and with the fixed-count law without replacement: loss and bias gradients as in exact backprop,
    weight gradients from the stores."""
    cfg = get_config(name)
    ctx, ref, _ = _run(cfg, variant, 0.1, seed=3, step=2, law=law)
    tol = TOL[cfg.dtype]
    assert abs(ctx.loss.item() - ref.loss) <= (1e-5 if cfg.dtype == "f32" else 2e-3) * abs(ref.loss)
    nnz = ctx.nnz.cpu().numpy().reshape(-1, 2)
    for l in range(len(cfg.dims) - 1):
        assert nnz[l, 0] == (ref.stores[l].nnz if variant == "different" else ref.stores[l].idx.size)
        for got, want in ((ctx.dW[l], ref.dW[l]), (ctx.db[l], ref.db[l])):
            fro, mx = rel_err(to_host_f32(got), want)
            assert fro <= tol and mx <= tol, (l, fro, mx)


@pytest.mark.parametrize("name,variant", [("mlp_small_different", "different"), ("mlp_small_same", "same"),
                                          ("mlp_wide_cut", "different"), ("mlp_wide_cut", "same")])
@pytest.mark.parametrize("p", [0.1, 1.0])
@pytest.mark.parametrize("act", ["relu", "gelu"])
def test_step_matches_oracle(name, variant, p, act):
    cfg = get_config(name)
    ctx, ref, _ = _run(cfg, variant, p, seed=0, act=act)
    tol = TOL[cfg.dtype]
    assert abs(ctx.loss.item() - ref.loss) <= 1e-5 * abs(ref.loss) if cfg.dtype == "f32" else \
        abs(ctx.loss.item() - ref.loss) <= 2e-3 * abs(ref.loss)
    nnz = ctx.nnz.cpu().numpy().reshape(-1, 2)
    for l in range(len(cfg.dims) - 1):
        assert nnz[l, 0] == (ref.stores[l].nnz if variant == "different" else ref.stores[l].idx.size)
        for got, want in ((ctx.dW[l], ref.dW[l]), (ctx.db[l], ref.db[l])):
            fro, mx = rel_err(to_host_f32(got), want)
            assert fro <= tol and mx <= tol, (l, fro, mx)


def test_stored_bytes_report():
    import paper_2007_10412_b200 as rad
    cfg = get_config("mlp_small_different")
    ctx = rad.MLPStep(cfg.dims, cfg.batch, "f32", "relu", "different", 0.1)
    s = ctx.stats
    assert s.full_backprop_bytes == 150 * 1384 * 4 + 6000
    assert s.unsampled_bytes == 6000 and s.relu_bytes == 150 * 20 * 4 and s.preact_bytes == 0
    assert 0.1 * 150 * 1384 * 4 < s.value_bytes < 0.16 * 150 * 1384 * 4
    g = rad.MLPStep(cfg.dims, cfg.batch, "f32", "gelu", "different", 0.1)
    assert g.stats.preact_bytes == 150 * 600 * 4 and g.stats.relu_bytes == 0


@pytest.mark.parametrize("p", [0.01, 0.05, 0.1, 0.2, 0.5, 1.0])
def test_same_sample_statistics_over_seeds(p):
    """Mean over seeds approaches the exact gradient and the variance follows q * dW^2 (same sample)."""
    import paper_2007_10412_b200 as rad
    cfg = get_config("mlp_small_same")
    X, y, Ws, bs = mlp_inputs(cfg.dims, cfg.batch, "f32", cfg.x_dist, cfg.data_seed)
    exact = orc.mlp_step(X, y, Ws, bs)
    ctx = rad.MLPStep(cfg.dims, cfg.batch, "f32", "relu", "same", p)
    dX, dy = to_dev(X, "f32"), torch.from_numpy(y).cuda()
    dWs, dbs = [to_dev(W, "f32") for W in Ws], [to_dev(b, "f32") for b in bs]
    S = 1000
    L = len(Ws)
    acc = [torch.zeros_like(w, dtype=torch.float64) for w in ctx.dW]
    sq = [torch.zeros((), dtype=torch.float64, device="cuda") for _ in range(L)]
    ex = [torch.from_numpy(g).cuda() for g in exact.dW]
    for seed in range(S):
        ctx(dX, dy, dWs, dbs, seed=seed)
        for l in range(L):
            g = ctx.dW[l].double()
            acc[l] += g
            sq[l] += ((g - ex[l]) ** 2).sum()
    torch.cuda.synchronize()
    assert ctx.dev_status.item() == 0
    pe = orc.effective_p(p)
    q = (1 - pe) / pe
    for l in range(L):
        var_sum = q * float((exact.dW[l] ** 2).sum())
        err = float(((acc[l] / S - ex[l]) ** 2).sum())
        norm = float((exact.dW[l] ** 2).sum())
        if p == 1.0:
            assert err <= 1e-10 * norm
        else:
            assert err <= 2.0 * var_sum / S + 1e-10 * norm
            assert abs(float(sq[l]) / S - var_sum) <= 0.15 * var_sum


@pytest.mark.parametrize("name", ["mlp_small_different", "mlp_wide_cut"])
def test_step_with_the_projection_variant_matches_oracle(name):
    """The whole step with P = R R^T (Rademacher projection, k = ceil(0.25 d)): loss and bias gradients as in
    exact backprop, weight gradients R' ((S^T dZ) / k) from the stored blocks."""
    cfg = get_config(name)
    ctx, ref, _ = _run(cfg, "project", 0.25, seed=5, step=1)
    tol = TOL[cfg.dtype]
    assert abs(ctx.loss.item() - ref.loss) <= (1e-5 if cfg.dtype == "f32" else 2e-3) * abs(ref.loss)
    nnz = ctx.nnz.cpu().numpy().reshape(-1, 2)
    for l in range(len(cfg.dims) - 1):
        assert nnz[l, 0] == ref.stores[l].T
        for got, want in ((ctx.dW[l], ref.dW[l]), (ctx.db[l], ref.db[l])):
            fro, mx = rel_err(to_host_f32(got), want)
            assert fro <= tol and mx <= tol, (l, fro, mx)
