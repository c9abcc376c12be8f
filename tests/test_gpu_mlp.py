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


@pytest.mark.parametrize("name,variant,act,launches", [("mlp_small_different", "different", "relu", 10),
                                                       ("mlp_small_different", "redrawn", "relu", None),
                                                       ("mlp_small_different", "different", "gelu", 10),
                                                       ("mlp_small_same", "same", "relu", 15)])
def test_small_net_step_equals_the_layer_calls_and_counts_its_launches(name, variant, act, launches):
    """On the nets that run on CUDA cores a layer's dW and the gradient of its input share one launch inside
    rad_mlp_step (Sec. 4.2: both are contractions of the same dZ).  The step's weight gradients and loss equal,
    bit for bit, those of the same step made of the public layer calls, one launch per contraction; the bias
    gradients agree to rounding (the step sums them in the dW kernel); and the MNIST-shaped net takes ten launches
    (fifteen with same-sample stores, whose store is three kernels)."""
    import paper_2007_10412_b200 as rad
    cfg = get_config(name)
    dims, B, L = cfg.dims, cfg.batch, len(cfg.dims) - 1
    X, y, Ws, bs = mlp_inputs(dims, B, cfg.dtype, cfg.x_dist, cfg.data_seed, bias_zero=False)
    dX, dy = to_dev(X, cfg.dtype), torch.from_numpy(y).cuda()
    dWs, dbs = [to_dev(W, cfg.dtype) for W in Ws], [to_dev(b, "f32") for b in bs]
    ctx = rad.MLPStep(dims, B, cfg.dtype, act, variant, 0.1)
    ctx(dX, dy, dWs, dbs, seed=21, step=5)                      # first call: one-time setup outside the count
    torch.cuda.synchronize()
    n0 = rad.rad_launch_count()
    ctx(dX, dy, dWs, dbs, seed=21, step=5)
    torch.cuda.synchronize()
    assert ctx.dev_status.item() == 0
    if launches is not None:
        assert rad.rad_launch_count() - n0 == launches
    # the same step, call by call
    tdt = dX.dtype
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    stores = [rad.Store("same" if variant == "same" else "different", cfg.dtype, B, dims[l], 0.1, seed=21, layer=l, step=5,
                        relu_bits=False) for l in range(L)]
    rbits = [None] + [torch.empty(B * ((dims[l] + 31) // 32), dtype=torch.int32, device="cuda") if act == "relu" else None
                      for l in range(1, L)]
    pre = [None] + [torch.empty(B, dims[l], dtype=tdt, device="cuda") if act == "gelu" else None for l in range(1, L)]
    a = dX
    rad.rad_linear_forward_store(a, stores[0], status)
    for l in range(L - 1):
        out = torch.empty(B, dims[l + 1], dtype=tdt, device="cuda")
        rad.rad_linear_forward(a, dWs[l], dbs[l], act, out_act=out, out_zlow=pre[l + 1], relubits=rbits[l + 1], dev_status=status)
        rad.rad_linear_forward_store(out, stores[l + 1], status)
        a = out
    logits = torch.empty(B, dims[L], dtype=torch.float32, device="cuda")
    rad.rad_linear_forward(a, dWs[L - 1], dbs[L - 1], "none", out_z=logits, dev_status=status)
    loss = torch.zeros(1, dtype=torch.float32, device="cuda")
    dz = torch.empty(B, dims[L], dtype=tdt, device="cuda")
    rad.rad_softmax_xent(logits, dy, loss, dz)
    for l in range(L - 1, -1, -1):
        dW = torch.full((dims[l], dims[l + 1]), float("nan"), dtype=torch.float32, device="cuda")
        db = torch.empty(dims[l + 1], dtype=torch.float32, device="cuda")
        rad.rad_linear_weight_grad(stores[l], dz, dW, dev_status=status)
        dzp = torch.empty(B, dims[l], dtype=tdt, device="cuda") if l > 0 else None
        rad.rad_linear_input_grad(dz, dWs[l], relubits_prev=rbits[l], z_prev=pre[l], dZ_prev=dzp, db=db, dev_status=status)
        torch.cuda.synchronize()
        assert status.item() == 0
        assert torch.equal(dW, ctx.dW[l]), l
        fro, mx = rel_err(to_host_f32(ctx.db[l]), to_host_f32(db).astype(np.float64))
        assert fro <= 1e-5 and mx <= 1e-5, (l, fro, mx)
        dz = dzp
    assert torch.equal(loss, ctx.loss)
