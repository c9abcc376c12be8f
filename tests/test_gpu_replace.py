"""The with-replacement law (the paper's own) and the fixed-count law without replacement on the GPU
against the oracle: store and weight gradient (different-sample and same-sample, float32 and bf16)."""
import numpy as np
import pytest
import torch

from oracle import rad as orc
from workloads import layer_inputs

from gpu_util import TOL, bits_host, rel_err, to_dev, u32
from layout import bits_of, tile_major

pytestmark = pytest.mark.gpu

SHAPES = [(150, 784, "f32"), (150, 300, "bf16"), (7, 5, "f32"), (64, 128, "bf16"), (328, 640, "bf16"),
          (257, 1160, "f32"), (1, 1, "f32")]


LAWS = ["replace", "fixed"]


@pytest.fixture
def store_kernel(request):
    """Forces one of the different-sample store kernels for the test, then restores the automatic choice."""
    import paper_2007_10412_b200 as rad
    prev = rad.rad_set_store_kernel(request.param)
    yield request.param
    rad.rad_set_store_kernel(prev)


# "pipelined": where the index part comes from the key alone (fixed-count law), the values are placed by the
# persistent kernel's loader and compaction warps instead of one CTA per tile; the last two shapes span several
# chunks with a ragged last chunk, slab and column block
@pytest.mark.parametrize("store_kernel", ["auto", "pipelined"], indirect=True)
@pytest.mark.parametrize("law", LAWS)
@pytest.mark.parametrize("B,D,dtype", SHAPES + [(1000, 1160, "bf16"), (449, 2200, "f32")])
@pytest.mark.parametrize("f", [0.1, 0.5, 1.0, 0.01])
def test_different_sample_store_is_bit_exact(B, D, dtype, f, law, store_kernel):
    import paper_2007_10412_b200 as rad
    A, _ = layer_inputs(B, D, 1, dtype=dtype, seed=B + D, relu_like=True)
    seed, layer, step = (1 << 40) + 777, 2, 5
    ref = orc.forward_store(A, dtype, "different", f, seed, layer, step, law=law)
    assert rad.rad_draws_per_row(f, D) == ref.T
    assert np.float32(rad.rad_replace_scale(f, D)) == ref.scale
    if law == "fixed":
        assert ref.nnz == B * ref.T                      # exactly k entries per row
    st = rad.Store("different", dtype, B, D, f, seed=seed, layer=layer, step=step, capacity="worst", law=law)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rad.rad_linear_forward_store(to_dev(A, dtype), st, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    kb, vals, offs = tile_major(ref)
    assert np.array_equal(u32(st.keepbits), kb)
    assert np.array_equal(u32(st.offsets), offs)
    nnz = st.nnz.cpu().numpy()
    assert nnz[0] == ref.nnz and nnz[1] == offs[-1]
    assert np.array_equal(bits_host(st.values[:int(offs[-1])]), bits_of(vals, dtype))
    assert np.array_equal(u32(st.relubits).reshape(B, -1), ref.relubits)


@pytest.mark.parametrize("law", LAWS)
@pytest.mark.parametrize("B,D,dtype", SHAPES)
@pytest.mark.parametrize("f", [0.1, 0.5, 1.0])
def test_same_sample_store_is_bit_exact(B, D, dtype, f, law):
    import paper_2007_10412_b200 as rad
    A, _ = layer_inputs(B, D, 1, dtype=dtype, seed=B + D + 1, relu_like=True)
    seed, layer, step = 99, 1, 3
    ref = orc.forward_store(A, dtype, "same", f, seed, layer, step, law=law)
    st = rad.Store("same", dtype, B, D, f, seed=seed, layer=layer, step=step, capacity="worst", law=law)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rad.rad_linear_forward_store(to_dev(A, dtype), st, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    k = ref.idx.size
    nnz = st.nnz.cpu().numpy()
    assert nnz[0] == k and nnz[1] == k * B
    assert np.array_equal(u32(st.offsets)[:k], ref.idx.astype(np.uint32))
    assert np.array_equal(u32(st.keepbits), ref.keepbits.reshape(-1))
    ld = st.c.values_ld
    got = bits_host(st.values[:B * ld]).reshape(B, ld)
    assert np.array_equal(got[:, :k], bits_of(ref.values, dtype).reshape(B, k))
    assert (got[:, k:] == 0).all()


@pytest.mark.parametrize("law", LAWS)
@pytest.mark.parametrize("variant", ["different", "same"])
@pytest.mark.parametrize("B,D,H,dtype", [(150, 784, 300, "f32"), (328, 640, 520, "bf16"), (130, 264, 72, "bf16")])
def test_weight_gradient_from_the_store(variant, B, D, H, dtype, law):
    """dW_hat = A_hat^T dZ from such a store through the same weight-gradient call."""
    import paper_2007_10412_b200 as rad
    f = 0.2
    A, dZ = layer_inputs(B, D, H, dtype=dtype, seed=B + H)
    ref = orc.forward_store(A, dtype, variant, f, 5, 0, 1, law=law)
    want = orc.weight_grad(ref, dZ)
    st = rad.Store(variant, dtype, B, D, f, seed=5, layer=0, step=1, law=law)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rad.rad_linear_forward_store(to_dev(A, dtype), st, status)
    dW = torch.empty(D, H, dtype=torch.float32, device="cuda")
    ws = torch.empty(max(rad.rad_weight_grad_workspace(st, H), 256), dtype=torch.uint8, device="cuda")
    rad.rad_linear_weight_grad(st, to_dev(dZ, dtype), dW, ws, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    fro, mx = rel_err(dW.cpu().numpy(), want)
    assert fro <= TOL[dtype] and mx <= TOL[dtype], (fro, mx)
    if variant == "same":
        unkept = np.setdiff1d(np.arange(D), ref.idx)
        assert (dW.cpu().numpy()[unkept] == 0).all()


def test_a_layer_of_many_tiles_and_the_typical_capacity():
    import paper_2007_10412_b200 as rad
    B, D, f = 1200, 4096, 0.1
    A, _ = layer_inputs(B, D, 1, dtype="bf16", seed=12)
    ref = orc.forward_store(A, "bf16", "different", f, 1, 0, 0, law="replace", with_relu_bits=False)
    st = rad.Store("different", "bf16", B, D, f, seed=1, relu_bits=False, law="replace")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rad.rad_linear_forward_store(to_dev(A, "bf16"), st, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    kb, vals, offs = tile_major(ref)
    assert np.array_equal(u32(st.keepbits), kb) and np.array_equal(u32(st.offsets), offs)
    assert np.array_equal(bits_host(st.values[:int(offs[-1])]), bits_of(vals, "bf16"))
    # distinct columns per row: D (1 - (1 - 1/D)^k) on average (Sec. 3.2 law), fewer than the k draws
    k = orc.draws_per_row(f, D)
    assert abs(ref.nnz / B - D * (1 - (1 - 1 / D) ** k)) < 3.0 and ref.nnz < B * k


@pytest.mark.parametrize("variant", ["different", "same"])
def test_fixed_count_law_at_fraction_one_is_exact_backprop(variant):
    """Without replacement a fraction of 1.0 keeps everything with weight 1 (App. A): dW equals A^T dZ."""
    import paper_2007_10412_b200 as rad
    B, D, H = 150, 300, 64
    A, dZ = layer_inputs(B, D, H, dtype="f32", seed=4)
    st = rad.Store(variant, "f32", B, D, 1.0, seed=8, law="fixed", capacity="worst")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rad.rad_linear_forward_store(to_dev(A, "f32"), st, status)
    dW = torch.empty(D, H, dtype=torch.float32, device="cuda")
    ws = torch.empty(max(rad.rad_weight_grad_workspace(st, H), 256), dtype=torch.uint8, device="cuda")
    rad.rad_linear_weight_grad(st, to_dev(dZ, "f32"), dW, ws, status)
    torch.cuda.synchronize()
    assert status.item() == 0 and st.nnz.cpu().numpy()[0] == (B * D if variant == "different" else D)
    fro, mx = rel_err(dW.cpu().numpy(), A.astype(np.float64).T @ dZ.astype(np.float64))
    assert fro <= 1e-5 and mx <= 1e-5


@pytest.mark.parametrize("store_kernel", ["auto", "pipelined"], indirect=True)
@pytest.mark.parametrize("law,variant", [("fixed", "different"), ("replace", "different"), ("bernoulli", "redrawn")])
def test_a_short_values_buffer_is_reported_and_nothing_is_written_past_it(law, variant, store_kernel):
    """The routes that place values into an index made from the key alone: with room for a part of the tiles
    only, the call reports it, the counts stay exact, the tiles that fit hold the oracle's values and nothing
    is written past the declared capacity."""
    import paper_2007_10412_b200 as rad
    B, D, f, dtype = 1000, 1160, 0.1, "bf16"
    A, _ = layer_inputs(B, D, 1, dtype=dtype, seed=5)
    ref = orc.forward_store(A, dtype, "different", f, 9, 1, 2, law=law, with_relu_bits=False)
    _, vals, offs = tile_major(ref)
    declared = int(offs[len(offs) // 2]) + 8            # about half of the tiles fit
    st = rad.Store(variant, dtype, B, D, f, seed=9, layer=1, step=2, relu_bits=False, capacity="worst", law=law)
    st.c.values_capacity = declared
    st.values.fill_(float("nan"))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rad.rad_linear_forward_store(to_dev(A, dtype), st, status)
    torch.cuda.synchronize()
    assert status.item() == rad.RAD_DEV_ECAPACITY
    nnz = st.nnz.cpu().numpy()
    assert nnz[0] == ref.nnz and nnz[1] == offs[-1]
    got = bits_host(st.values)
    fits = int(max(o for o in offs if o <= declared))
    assert np.array_equal(got[:fits], bits_of(vals, dtype)[:fits])
    assert torch.isnan(st.values[declared:].float()).all()
