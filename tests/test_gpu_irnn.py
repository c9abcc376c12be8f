"""rad_irnn_step against the recurrent oracle: the Sequential-MNIST-shaped IRNN (batch 150, 784 steps,
hidden 100) and small random recurrent nets, both sampling variants."""
import numpy as np
import pytest
import torch

from oracle import irnn as orc
from workloads import irnn_inputs

from gpu_util import rel_err

pytestmark = pytest.mark.gpu

CASES = [
    # B, T, hidden, classes, identity-initialised
    (9, 23, 40, 5, False),
    (33, 50, 100, 10, False),
    (4, 7, 128, 3, False),
    (150, 784, 100, 10, True),        # the paper's IRNN shape and initialisation
]


@pytest.mark.parametrize("B,T,Hd,C,ident", CASES)
@pytest.mark.parametrize("variant", ["different", "same"])
@pytest.mark.parametrize("p", [0.1, 1.0])
def test_irnn_step_matches_oracle(B, T, Hd, C, ident, variant, p):
    import paper_2007_10412_b200 as rad
    args = irnn_inputs(B, T, Hd, C, seed=B + T, identity=ident)
    ref = orc.irnn_step(*args, variant=variant, p=p, seed=5, step0=1000)
    ctx = rad.IRNNStep(B, T, Hd, C, variant, p)
    dev = [torch.from_numpy(np.ascontiguousarray(a)).cuda() for a in args]
    ctx(*dev, seed=5, step0=1000)
    torch.cuda.synchronize()
    assert ctx.dev_status.item() == 0
    assert abs(ctx.loss.item() - ref.loss) <= 1e-5 * abs(ref.loss)
    nnz = ctx.nnz.cpu().numpy()
    assert nnz[0] == ref.nnz_steps.sum()                     # masks are data-independent: exact counts
    assert nnz[1] == (ref.nnz_out if variant == "different" else ref.nnz_out // B)
    for name, got, want in (("dW_hh", ctx.dW_hh, ref.dW_hh), ("dW_out", ctx.dW_out, ref.dW_out),
                            ("dW_ih", ctx.dW_ih, ref.dW_ih), ("db", ctx.db, ref.db), ("db_out", ctx.db_out, ref.db_out)):
        fro, mx = rel_err(got.double().cpu().numpy(), want)
        assert fro <= 1e-5 and mx <= 1e-5, (name, fro, mx)


def test_irnn_stored_bytes():
    import paper_2007_10412_b200 as rad
    ctx = rad.IRNNStep(150, 784, 100, 10, "different", 0.1)
    s = ctx.stats
    assert s.full_backprop_bytes == 150 * 317176               # App. A: 317.176 kBytes per element
    assert s.relu_bytes == 784 * 150 * 4 * 4                    # 1 bit per hidden unit and step, in 32-bit words
    held = s.value_bytes + s.index_bytes + s.relu_bytes + s.unsampled_bytes
    assert 4.5 < s.full_backprop_bytes / held < 8.0
    # without the keep bits and offsets, which the paper's count leaves out, the saving is near its 7.15x
    assert 6.0 < s.full_backprop_bytes / (held - s.index_bytes) < 7.2
