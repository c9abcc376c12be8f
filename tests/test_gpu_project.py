"""Random-projection variant on the GPU against the oracle: the sign matrix bit for bit, the stored block
S = A R' and the weight gradient R' ((S^T dZ) / k) within the floating-point tolerance, the whole step."""
import numpy as np
import pytest
import torch

from oracle import rad as orc
from workloads import get_config, layer_inputs, mlp_inputs

from gpu_util import TOL, rel_err, to_dev, to_host_f32

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("D,f,dtype", [(784, 0.1, "f32"), (300, 0.5, "bf16"), (5, 1.0, "f32"), (640, 0.3, "bf16"),
                                       (1, 1.0, "f32"), (200, 0.9, "bf16")])
def test_sign_matrix_is_bit_exact(D, f, dtype):
    import paper_2007_10412_b200 as rad
    k = orc.draws_per_row(f, D)
    ld = -(-k // 64) * 64
    want = np.zeros((D, ld), dtype=np.float32)
    want[:, :k] = orc.rademacher(D, k, 0xABCDEF12345, 3, 9)
    out = torch.full((D, ld), 7.0, dtype=torch.float32 if dtype == "f32" else torch.bfloat16, device="cuda")
    rad.rad_rademacher(dtype, D, f, ld, 0xABCDEF12345, 3, 9, out)
    torch.cuda.synchronize()
    assert np.array_equal(to_host_f32(out), want)


@pytest.mark.parametrize("B,D,H,dtype,f", [(150, 784, 300, "f32", 0.1), (328, 640, 520, "bf16", 0.2),
                                           (130, 264, 72, "bf16", 0.5), (150, 300, 10, "f32", 1.0),
                                           (512, 1024, 256, "bf16", 0.1)])
def test_store_and_weight_gradient(B, D, H, dtype, f):
    import paper_2007_10412_b200 as rad
    A, dZ = layer_inputs(B, D, H, dtype=dtype, seed=B + H)
    ref = orc.project_store(A, dtype, f, 21, 1, 4)
    k = ref.T
    st = rad.Store("project", dtype, B, D, f, seed=21, layer=1, step=4, relu_bits=False)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rad.rad_linear_forward_store(to_dev(A, dtype), st, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    nnz = st.nnz.cpu().numpy()
    assert nnz[0] == k and nnz[1] == B * k
    ld = st.c.values_ld
    S = to_host_f32(st.values[:B * ld]).reshape(B, ld)
    assert (S[:, k:] == 0).all()
    fro, mx = rel_err(S[:, :k], ref.values.reshape(B, k))
    assert fro <= TOL[dtype] and mx <= TOL[dtype], (fro, mx)
    dW = torch.empty(D, H, dtype=torch.float32, device="cuda")
    ws = torch.empty(max(rad.rad_weight_grad_workspace(st, H), 256), dtype=torch.uint8, device="cuda")
    rad.rad_linear_weight_grad(st, to_dev(dZ, dtype), dW, ws, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    fro, mx = rel_err(dW.cpu().numpy(), orc.weight_grad(ref, dZ))
    assert fro <= TOL[dtype] and mx <= TOL[dtype], (fro, mx)


def test_bad_arguments_are_refused():
    import paper_2007_10412_b200 as rad
    A, _ = layer_inputs(64, 128, 1, dtype="bf16", seed=1)
    st = rad.Store("project", "bf16", 64, 128, 0.5)
    st.c.values_ld = 8                                           # fewer columns than k = 64
    with pytest.raises(rad.RadError, match="invalid argument"):
        rad.rad_linear_forward_store(to_dev(A, "bf16"), st)
    st.c.values_ld = 64
    st.workspace = st.workspace[:256]
    with pytest.raises(rad.RadError, match="workspace"):
        rad.rad_linear_forward_store(to_dev(A, "bf16"), st)


def test_relu_bits_come_with_the_projected_store():
    """The 1-bit ReLU derivative of the layer that produced A (Sec. 4.2) is written by the same call."""
    import paper_2007_10412_b200 as rad
    B, D = 130, 264
    A, _ = layer_inputs(B, D, 1, dtype="bf16", seed=6, relu_like=True)
    st = rad.Store("project", "bf16", B, D, 0.25, seed=2, relu_bits=True)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rad.rad_linear_forward_store(to_dev(A, "bf16"), st, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    got = st.relubits.cpu().numpy().view(np.uint32).reshape(B, -1)
    assert np.array_equal(got, orc.pack_bits(A > 0))
