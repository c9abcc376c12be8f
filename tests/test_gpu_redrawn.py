"""The different-sample store held without its keep bits (Sec. 3.2: the random matrix does not depend on the
data, so the backward pass can draw it again): values, tile offsets and counts against the oracle's
different-sample store, the weight gradient against the oracle and, bit for bit, against the one computed
from a store that holds its index."""
import numpy as np
import pytest
import torch

from oracle import rad as orc
from workloads import get_config, layer_inputs, mlp_inputs

from gpu_util import TOL, bits_host, rel_err, to_dev, to_host_f32, u32
from layout import bits_of, tile_major

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,D,H,dtype", [(150, 300, 40, "f32"), (257, 1160, 72, "bf16"), (2100, 8200, 136, "bf16")])
@pytest.mark.parametrize("p,law", [(0.1, "bernoulli"), (0.5, "bernoulli"), (0.1, "fixed")])
def test_store_and_weight_grad_without_held_keep_bits(B, D, H, dtype, p, law):
    import paper_2007_10412_b200 as rad
    A, dZ = layer_inputs(B, D, H, dtype=dtype, seed=B + D + H, relu_like=True)
    seed, layer, step = (5 << 35) + 99, 1, 4
    ref = orc.forward_store(A, dtype, "different", p, seed, layer, step, law=law)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Ad, dZd = to_dev(A, dtype), to_dev(dZ, dtype)
    held = rad.Store("redrawn", dtype, B, D, p, seed=seed, layer=layer, step=step, capacity="worst", law=law)
    assert held.keepbits.numel() == 0 and held.c.keepbits is None
    rad.rad_linear_forward_store(Ad, held, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    _, vals, offs = tile_major(ref)
    assert np.array_equal(u32(held.offsets), offs)
    nnz = held.nnz.cpu().numpy()
    assert nnz[0] == ref.nnz and nnz[1] == offs[-1]
    assert np.array_equal(bits_host(held.values[:int(offs[-1])]), bits_of(vals, dtype))
    assert np.array_equal(u32(held.relubits).reshape(B, -1), ref.relubits)

    def weight_grad(st):
        dW = torch.full((D, H), float("nan"), dtype=torch.float32, device="cuda")
        ws = torch.empty(max(rad.rad_weight_grad_workspace(st, H), 256), dtype=torch.uint8, device="cuda")
        ws.fill_(0xA5)                                   # nothing of the index may be taken from old contents
        rad.rad_linear_weight_grad(st, dZd, dW, ws, status)
        torch.cuda.synchronize()
        assert status.item() == 0
        return dW

    dW_held = weight_grad(held)
    want = orc.weight_grad(ref, dZ)
    fro, mx = rel_err(to_host_f32(dW_held), want)
    assert fro <= TOL[dtype] and mx <= TOL[dtype], (fro, mx)
    # the same contraction from a store that holds its index: identical bits
    full = rad.Store("different", dtype, B, D, p, seed=seed, layer=layer, step=step, capacity="worst", law=law)
    rad.rad_linear_forward_store(Ad, full, status)
    assert torch.equal(weight_grad(full), dW_held)
    # what is held between the passes
    assert held.held_bytes()["index_bytes"] == 4 * (len(offs))
    assert full.held_bytes()["index_bytes"] == 4 * (len(offs) + 288 * (len(offs) - 1))


@pytest.mark.parametrize("name,act,law", [("mlp_small_different", "relu", "bernoulli"), ("mlp_wide_cut", "relu", "bernoulli"),
                                          ("mlp_wide_cut", "gelu", "bernoulli"), ("mlp_wide_cut", "relu", "fixed"),
                                          ("mlp_small_different", "relu", "fixed")])
def test_step_without_held_keep_bits_equals_the_step_that_holds_them(name, act, law):
    """rad_mlp_step with variant "redrawn": the hidden layers' stores come out of the forward epilogue with
    their index in the scratch area, the backward pass draws every index again; loss and all gradients equal
    those of the different-sample step bit for bit, the oracle's within tolerance, and the index bytes held
    shrink to the tile offsets."""
    import paper_2007_10412_b200 as rad
    cfg = get_config(name)
    X, y, Ws, bs = mlp_inputs(cfg.dims, cfg.batch, cfg.dtype, cfg.x_dist, cfg.data_seed, bias_zero=False)
    dX, dy = to_dev(X, cfg.dtype), torch.from_numpy(y).cuda()
    dWs, dbs = [to_dev(W, cfg.dtype) for W in Ws], [to_dev(b, "f32") for b in bs]
    out = {}
    for variant in ("different", "redrawn"):
        ctx = rad.MLPStep(cfg.dims, cfg.batch, cfg.dtype, act, variant, 0.1, law=law)
        ctx.workspace.fill_(0x5A)
        ctx(dX, dy, dWs, dbs, seed=11, step=3)
        torch.cuda.synchronize()
        assert ctx.dev_status.item() == 0
        out[variant] = ctx
    a, b = out["different"], out["redrawn"]
    assert torch.equal(a.loss, b.loss) and torch.equal(a.nnz, b.nnz)
    for l in range(len(cfg.dims) - 1):
        assert torch.equal(a.dW[l], b.dW[l]) and torch.equal(a.db[l], b.db[l]), l
    ref = orc.mlp_step(X, y, Ws, bs, act=act, dtype=cfg.dtype, variant="different", p=0.1, seed=11, step=3, law=law)
    for l in range(len(cfg.dims) - 1):
        fro, mx = rel_err(to_host_f32(b.dW[l]), ref.dW[l])
        assert fro <= TOL[cfg.dtype] and mx <= TOL[cfg.dtype], (l, fro, mx)
    ntiles = sum(((cfg.batch + 63) // 64) * ((d + 127) // 128) for d in cfg.dims[:-1])
    assert b.stats.index_bytes == 4 * (ntiles + len(cfg.dims) - 1)
    assert a.stats.index_bytes == b.stats.index_bytes + 4 * 288 * ntiles
    assert a.stats.value_bytes == b.stats.value_bytes


def test_redrawn_store_rejects_what_it_cannot_do():
    import paper_2007_10412_b200 as rad
    with pytest.raises(rad.RadError, match="invalid"):
        rad.Store("redrawn", "bf16", 64, 128, 0.1, law="replace")
    st = rad.Store("redrawn", "bf16", 64, 128, 0.1)
    with pytest.raises(rad.RadError, match="unsupported"):
        rad.rad_store_index(st)
