"""Per-layer backward calls against the oracle: dW from the store, exact dX / db, forward, loss."""
import numpy as np
import pytest
import torch

from oracle import rad as orc
from workloads import layer_inputs, mlp_inputs

from gpu_util import TOL, rel_err, to_dev, to_host_f32, u32

pytestmark = pytest.mark.gpu

LAYERS = [
    (150, 784, 300, "f32"),
    (150, 300, 10, "f32"),
    (150, 300, 10, "bf16"),     # unaligned bf16: CUDA-core kernels
    (33, 17, 5, "f32"),
    (328, 640, 520, "bf16"),    # aligned bf16: tensor-core kernels
    (328, 392, 200, "bf16"),
    (1024, 256, 512, "bf16"),
    (900, 520, 600, "f32"),     # float32 with enough tiles for the CUDA-core GEMM's larger tile
]


@pytest.mark.parametrize("B,D,H,dtype", LAYERS)
@pytest.mark.parametrize("variant", ["different", "same"])
@pytest.mark.parametrize("p", [0.1, 1.0, 0.5])
def test_weight_grad_matches_oracle(B, D, H, dtype, variant, p):
    import paper_2007_10412_b200 as rad
    A, dZ = layer_inputs(B, D, H, dtype=dtype, seed=B + D + H)
    ref_st = orc.forward_store(A, dtype, variant, p, 11, 2, 0)
    ref = orc.weight_grad(ref_st, dZ)
    st = rad.Store(variant, dtype, B, D, p, seed=11, layer=2, step=0, relu_bits=False)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rad.rad_linear_forward_store(to_dev(A, dtype), st, status)
    dW = torch.full((D, H), float("nan"), dtype=torch.float32, device="cuda")
    rad.rad_linear_weight_grad(st, to_dev(dZ, dtype), dW, dev_status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    got = to_host_f32(dW)
    fro, mx = rel_err(got, ref)
    assert fro <= TOL[dtype] and mx <= TOL[dtype], (fro, mx)
    if variant == "same":
        kept = np.zeros(D, bool)
        kept[ref_st.idx] = True
        assert (got[~kept] == 0).all()          # Sec. 4.3: rows of unsampled columns are untouched
    # run to run reproducibility (fixed accumulation order)
    dW2 = torch.empty_like(dW)
    rad.rad_linear_weight_grad(st, to_dev(dZ, dtype), dW2, dev_status=status)
    torch.cuda.synchronize()
    assert torch.equal(dW, dW2)


@pytest.mark.parametrize("B,D,H,dtype", LAYERS)
@pytest.mark.parametrize("act", ["relu", "gelu"])
def test_input_grad_matches_oracle(B, D, H, dtype, act):
    import paper_2007_10412_b200 as rad
    rng = np.random.default_rng(B * 7 + D)
    _, dZ = layer_inputs(B, D, H, dtype=dtype, seed=5)
    W = rng.standard_normal((D, H), dtype=np.float32) * np.float32(np.sqrt(2.0 / D))
    Zp = rng.standard_normal((B, D), dtype=np.float32)
    if dtype == "bf16":
        from workloads import to_bf16_grid
        W, Zp = to_bf16_grid(W), to_bf16_grid(Zp)
    bits = orc.pack_bits(Zp > 0)
    if act == "relu":
        ref_dA, ref_db = orc.input_grad(dZ, W, relubits_prev=bits, dtype=dtype)
    else:
        ref_dA, ref_db = orc.input_grad(dZ, W, Z_prev=Zp, act="gelu", dtype=dtype)
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    out = torch.full((B, D), float("nan"), dtype=tdt, device="cuda")
    db = torch.full((H,), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rad.rad_linear_input_grad(to_dev(dZ, dtype), to_dev(W, dtype),
                              relubits_prev=torch.from_numpy(bits.view(np.int32)).cuda() if act == "relu" else None,
                              z_prev=to_dev(Zp, dtype) if act == "gelu" else None,
                              dZ_prev=out, db=db, dev_status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    fro, mx = rel_err(to_host_f32(out), ref_dA)
    assert fro <= TOL[dtype] and mx <= TOL[dtype], (fro, mx)
    fro, mx = rel_err(to_host_f32(db), ref_db)
    assert fro <= 1e-5 and mx <= 1e-5, (fro, mx)
    if act == "relu":
        assert (to_host_f32(out)[~(Zp > 0)] == 0).all()


@pytest.mark.parametrize("B,D,H,dtype", LAYERS)
@pytest.mark.parametrize("act", ["relu", "gelu", "none"])
def test_forward_matches_oracle(B, D, H, dtype, act):
    import paper_2007_10412_b200 as rad
    X, _, Ws, bs = mlp_inputs((D, H), B, dtype=dtype, x_dist="normal", seed=3, bias_zero=False)
    z = X.astype(np.float64) @ Ws[0].astype(np.float64) + bs[0]
    a = orc.act_forward(z, act)
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    out_act = torch.empty(B, H, dtype=tdt, device="cuda")
    out_z = torch.empty(B, H, dtype=torch.float32, device="cuda")
    out_zl = torch.empty(B, H, dtype=tdt, device="cuda")
    w32 = (H + 31) // 32
    rb = torch.zeros(B * w32, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rad.rad_linear_forward(to_dev(X, dtype), to_dev(Ws[0], dtype), to_dev(bs[0], "f32"), act, out_act=out_act,
                           out_z=out_z, out_zlow=out_zl, relubits=rb, dev_status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    tol = TOL[dtype]
    assert max(rel_err(to_host_f32(out_z), z)) <= 1e-5
    assert max(rel_err(to_host_f32(out_act), a)) <= (1e-5 if dtype == "f32" else 8e-3)
    assert max(rel_err(to_host_f32(out_zl), z)) <= (1e-5 if dtype == "f32" else 8e-3)
    assert tol >= 1e-5
    # the ReLU bits are those of the activation the call wrote
    assert np.array_equal(u32(rb).reshape(B, w32), orc.pack_bits(to_host_f32(out_act) > 0))


@pytest.mark.parametrize("B,C,dtype", [(150, 10, "f32"), (150, 10, "bf16"), (513, 1000, "bf16"), (3, 2, "f32")])
def test_softmax_xent_matches_oracle(B, C, dtype):
    import paper_2007_10412_b200 as rad
    rng = np.random.default_rng(C)
    logits = (rng.standard_normal((B, C)) * 3).astype(np.float32)
    labels = rng.integers(0, C, B).astype(np.int32)
    loss_ref, dz_ref = orc.softmax_xent(logits, labels)
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    dz = torch.empty(B, C, dtype=tdt, device="cuda")
    loss = torch.zeros(1, device="cuda")
    rad.rad_softmax_xent(torch.from_numpy(logits).cuda(), torch.from_numpy(labels).cuda(), loss, dz)
    torch.cuda.synchronize()
    assert abs(loss.item() - loss_ref) <= 1e-5 * abs(loss_ref)
    assert max(rel_err(to_host_f32(dz), dz_ref)) <= (1e-5 if dtype == "f32" else 8e-3)


@pytest.mark.parametrize("B,H,dtype", [(700, 10, "f32"), (700, 40, "bf16"), (5000, 64, "bf16"), (40000, 16, "bf16"),
                                       (700, 300, "f32"), (700, 301, "bf16"), (2100, 1000, "bf16"), (130, 1000, "bf16")])
def test_bias_gradient_alone_on_every_column_sum_route(B, H, dtype):
    """db = sum over the minibatch of dZ (Sec. 4.2: exact, never sampled), asked for without the input gradient:
    few rows (one launch), narrow matrices (row lanes x columns), wide bf16 matrices (16-byte loads) and the
    plain two-stage route, against float64 sums of the same numbers."""
    import paper_2007_10412_b200 as rad
    rng = np.random.default_rng(B + H)
    dZ = rng.standard_normal((B, H), dtype=np.float32)
    if dtype == "bf16":
        from workloads import to_bf16_grid
        dZ = to_bf16_grid(dZ)
    W = torch.zeros(8, H, dtype=torch.float32 if dtype == "f32" else torch.bfloat16, device="cuda")
    db = torch.full((H,), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rad.rad_linear_input_grad(to_dev(dZ, dtype), W, db=db, dev_status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    want = dZ.astype(np.float64).sum(axis=0)
    bound = 2e-6 * np.abs(dZ.astype(np.float64)).sum(axis=0)
    assert (np.abs(to_host_f32(db).astype(np.float64) - want) <= bound).all()
