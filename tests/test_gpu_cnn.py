"""rad_cnn_step against the convolutional oracle: the 32x32x3 / 16-32-64 / 1024-128-10 net of the
CNN configuration (bf16, batch 128) and smaller nets in both types and both sampling variants."""
import numpy as np
import pytest
import torch

from oracle import cnn as orc
from workloads import cnn_inputs

from gpu_util import TOL, rel_err, to_dev

pytestmark = pytest.mark.gpu

CASES = [
    # B, hw, cin, channels, fc, dtype
    (5, 8, 3, (8, 16), (24, 5), "f32"),
    (70, 16, 3, (8, 8), (32, 10), "bf16"),          # two row slabs in the stores
    (128, 32, 3, (16, 32, 64), (128, 10), "bf16"),  # the CNN configuration
    (37, 16, 16, (32, 24, 8), (16, 4), "bf16"),     # ragged pixel tiles; tensor-core kernels from the first convolution on
]


@pytest.fixture
def conv_kernel(request):
    """Forces the CUDA-core or the tensor-core convolution kernels for the test, then restores the automatic choice."""
    import paper_2007_10412_b200 as rad
    prev = rad.rad_set_conv_kernel(request.param)
    yield request.param
    rad.rad_set_conv_kernel(prev)


@pytest.mark.parametrize("conv_kernel", ["simt", "tensor"], indirect=True)
@pytest.mark.parametrize("B,hw,cin,channels,fc,dtype", CASES)
@pytest.mark.parametrize("variant", ["different", "same"])
@pytest.mark.parametrize("p", [0.1, 1.0])
def test_cnn_step_matches_oracle(B, hw, cin, channels, fc, dtype, variant, p, conv_kernel):
    import paper_2007_10412_b200 as rad
    X, y, cW, cb, fW, fb = cnn_inputs(B, hw, cin, channels, fc, dtype, seed=B + hw, bias_zero=False)
    ref = orc.cnn_step(X, y, cW, cb, fW, fb, dtype=dtype, variant=variant, p=p, seed=3, step=2)
    ctx = rad.CNNStep(B, hw, cin, channels, fc, dtype, variant, p)
    ctx(to_dev(X, dtype), torch.from_numpy(y).cuda(), [to_dev(w, dtype) for w in cW], [to_dev(b, "f32") for b in cb],
        [to_dev(w, dtype) for w in fW], [to_dev(b, "f32") for b in fb], seed=3, step=2)
    torch.cuda.synchronize()
    assert ctx.dev_status.item() == 0
    tol = TOL[dtype]
    assert abs(ctx.loss.item() - ref.loss) <= (1e-5 if dtype == "f32" else 2e-3) * abs(ref.loss)
    nnz = ctx.nnz.cpu().numpy().reshape(-1, 2)
    for l, want in enumerate(ref.nnz):
        assert nnz[l, 0] == (want if variant == "different" else want // B)
    got_all = ctx.dconv_W + ctx.dconv_b + ctx.dfc_W + ctx.dfc_b
    want_all = ref.dW_conv + ref.db_conv + ref.dW_fc + ref.db_fc
    # Frobenius error within the stated tolerance.  The largest single deviation gets twice that in bf16: one ReLU
    # decision of the 16384 outputs of the first linear layer that falls the other way (its pre-activation is a
    # last-bit rounding away from zero, and a different but equally valid summation order in a convolution
    # before it is enough) moves single entries of a 128-term sum by a percent or two while the tensor as a
    # whole moves by a fraction of a percent; it happens with either set of convolution kernels.
    for i, (got, want) in enumerate(zip(got_all, want_all)):
        fro, mx = rel_err(got.double().cpu().numpy(), want)
        assert fro <= tol and mx <= (tol if dtype == "f32" else 2 * tol), (i, fro, mx)


def test_cnn_stored_bytes():
    import paper_2007_10412_b200 as rad
    ctx = rad.CNNStep(128, 32, 3, (16, 32, 64), (128, 10), "bf16", "different", 0.1)
    s = ctx.stats
    per_sample_inputs = 3072 + 4096 + 2048 + 1024 + 128
    assert s.full_backprop_bytes == 128 * per_sample_inputs * 2 + 128 * 10 * 4
    assert s.relu_bytes == 128 * (32 * 32 * 16 + 16 * 16 * 32 + 8 * 8 * 64) // 8 + 128 * 4 * 4
    assert s.value_bytes < 0.16 * 128 * per_sample_inputs * 2
