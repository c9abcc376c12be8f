"""The static-shape store of the fixed-count law (exactly k columns per row, without replacement; App. A,
remark under the fraction sweep): B x k values and B x k 16-bit column numbers, bit for bit against the
oracle's Floyd sampling, and the weight gradient formed from it."""
import numpy as np
import pytest
import torch

from oracle import rad as orc
from workloads import layer_inputs

from gpu_util import TOL, bits_host, rel_err, to_dev, to_host_f32, u32
from layout import bits_of, tile_major

pytestmark = pytest.mark.gpu

SHAPES = [(150, 300, "f32"), (7, 5, "bf16"), (64, 128, "bf16"), (328, 640, "bf16"), (257, 1160, "f32"), (1000, 2200, "bf16")]


def _cols16(st, B, ld):
    return st.keepbits.view(torch.int16).cpu().numpy().view(np.uint16).reshape(B, ld)


@pytest.mark.parametrize("B,D,dtype", SHAPES)
@pytest.mark.parametrize("f", [0.1, 0.5, 1.0, 0.01])
def test_static_shape_store_is_bit_exact(B, D, dtype, f):
    import paper_2007_10412_b200 as rad
    A, _ = layer_inputs(B, D, 1, dtype=dtype, seed=B + D, relu_like=True)
    seed, layer, step = (3 << 35) + 77, 2, 5
    ref = orc.forward_store(A, dtype, "different", f, seed, layer, step, law="fixed")
    k = orc.draws_per_row(f, D)
    mask = orc.unpack_bits(ref.keepbits, D)
    assert (mask.sum(axis=1) == k).all()
    st = rad.Store("rows", dtype, B, D, f, seed=seed, layer=layer, step=step, law="fixed")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rad.rad_linear_forward_store(to_dev(A, dtype), st, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    ld = int(st.c.values_ld)
    assert ld % 8 == 0 and k <= ld < k + 8
    nnz = st.nnz.cpu().numpy()
    assert nnz[0] == B * k and nnz[1] == B * ld
    cols = _cols16(st, B, ld)
    want_cols = np.nonzero(mask)[1].reshape(B, k)
    assert np.array_equal(cols[:, :k], want_cols.astype(np.uint16))
    assert (cols[:, k:] == 0).all()
    vals = bits_host(st.values[:B * ld]).reshape(B, ld)
    assert np.array_equal(vals[:, :k], bits_of(ref.values, dtype).reshape(B, k))
    assert (vals[:, k:] == 0).all()
    assert np.array_equal(u32(st.relubits).reshape(B, -1), ref.relubits)


@pytest.mark.parametrize("B,D", [(150, 300), (328, 640), (1000, 2200)])
@pytest.mark.parametrize("f", [0.1, 0.5, 1.0])
def test_index_of_the_fixed_count_law_from_the_key_alone(B, D, f):
    import paper_2007_10412_b200 as rad
    seed, layer, step = 99, 1, 3
    ref = orc.forward_store(np.ones((B, D), np.float32), "f32", "different", f, seed, layer, step, with_relu_bits=False, law="fixed")
    st = rad.Store("different", "f32", B, D, f, seed=seed, layer=layer, step=step, relu_bits=False, law="fixed")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rad.rad_store_index(st, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    kb, _, offs = tile_major(ref)
    assert np.array_equal(u32(st.keepbits), kb)
    assert np.array_equal(u32(st.offsets), offs)
    nnz = st.nnz.cpu().numpy()
    assert nnz[0] == ref.nnz and nnz[1] == offs[-1]


@pytest.mark.parametrize("B,D,H,dtype", [(150, 784, 300, "f32"), (328, 640, 520, "bf16"), (1024, 256, 512, "bf16"), (33, 17, 5, "f32")])
@pytest.mark.parametrize("f", [0.1, 0.5])
def test_weight_grad_from_the_static_shape_store(B, D, H, dtype, f):
    import paper_2007_10412_b200 as rad
    A, dZ = layer_inputs(B, D, H, dtype=dtype, seed=B + H)
    ref_st = orc.forward_store(A, dtype, "different", f, 21, 0, 1, law="fixed")
    ref = orc.weight_grad(ref_st, dZ)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    st = rad.Store("rows", dtype, B, D, f, seed=21, layer=0, step=1, relu_bits=False, law="fixed")
    rad.rad_linear_forward_store(to_dev(A, dtype), st, status)
    dW = torch.full((D, H), float("nan"), dtype=torch.float32, device="cuda")
    rad.rad_linear_weight_grad(st, to_dev(dZ, dtype), dW, dev_status=status)
    # the bitmask form of the same law and key: same mask, same values, same contraction
    st2 = rad.Store("different", dtype, B, D, f, seed=21, layer=0, step=1, relu_bits=False, law="fixed")
    rad.rad_linear_forward_store(to_dev(A, dtype), st2, status)
    dW2 = torch.empty_like(dW)
    rad.rad_linear_weight_grad(st2, to_dev(dZ, dtype), dW2, dev_status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    fro, mx = rel_err(to_host_f32(dW), ref)
    assert fro <= TOL[dtype] and mx <= TOL[dtype], (fro, mx)
    assert torch.equal(dW, dW2)


def test_static_shape_store_at_the_bench_size():
    """65536 x 8192, fraction 0.1: sampled rows bit for bit (the oracle draws those rows alone), the static shape,
    and dW on sampled entries."""
    import paper_2007_10412_b200 as rad
    B, D, H, f = 65536, 8192, 8192, 0.1
    A, dZ = layer_inputs(B, D, H, dtype="bf16", seed=77)
    Ad, dZd = torch.from_numpy(A).to(torch.bfloat16).cuda(), torch.from_numpy(dZ).to(torch.bfloat16).cuda()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    st = rad.Store("rows", "bf16", B, D, f, seed=5, layer=1, step=3, relu_bits=False, law="fixed")
    rad.rad_linear_forward_store(Ad, st, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    k, ld = orc.draws_per_row(f, D), int(st.c.values_ld)
    assert k == 820 and ld == 824
    rng = np.random.default_rng(8)
    rows = np.concatenate([[0, 63, 64, B - 1], rng.integers(0, B, 28)])
    sub = orc.fixed_subset("different", B, D, f, 5, 1, 3, rows=rows).astype(bool)
    want_cols = np.nonzero(sub)[1].reshape(len(rows), k)
    ri = torch.from_numpy(rows).cuda()
    cols = st.keepbits.view(torch.int16).view(B, ld)[ri].cpu().numpy().view(np.uint16)
    assert np.array_equal(cols[:, :k], want_cols.astype(np.uint16)) and (cols[:, k:] == 0).all()
    s = orc.replace_scale(f, D)
    want = orc.bf16_bits(orc.round_bf16(np.take_along_axis(A[rows], want_cols, axis=1) * s))
    vals = st.values.view(B, ld)[ri].view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.array_equal(vals[:, :k], want) and (vals[:, k:] == 0).all()
    dW = torch.full((D, H), float("nan"), dtype=torch.float32, device="cuda")
    rad.rad_linear_weight_grad(st, dZd, dW, dev_status=status)
    torch.cuda.synchronize()
    assert status.item() == 0 and torch.isfinite(dW).all()
    ds = np.concatenate([[0, 127, 128, D - 1], rng.integers(0, D, 8)])
    hs = np.concatenate([[0, 255, 256, H - 1], rng.integers(0, H, 12)])
    full = orc.fixed_subset("different", B, D, f, 5, 1, 3).astype(bool)[:, ds]
    a_hat = np.where(full, orc.round_bf16(A[:, ds] * s), np.float32(0)).astype(np.float64)
    ref = a_hat.T @ dZ[:, hs].astype(np.float64)
    got = to_host_f32(dW[torch.from_numpy(ds).cuda()][:, torch.from_numpy(hs).cuda()])
    assert max(rel_err(got, ref)) <= 2e-2
