"""rad_linear_forward_store against the oracle: masks, offsets, values and ReLU bits bit for bit."""
import numpy as np
import pytest
import torch

from oracle import rad as orc
from workloads import layer_inputs

from gpu_util import bits_host, to_dev, u32
from layout import bits_of, tile_major

pytestmark = pytest.mark.gpu

SHAPES = [
    (150, 784, "f32"),      # MNIST layer 1 (7 ragged column blocks, 3 row slabs)
    (150, 300, "f32"),      # row stride not 16-byte aligned for bf16, ragged everything
    (150, 300, "bf16"),
    (1, 1, "f32"),          # degenerate
    (7, 5, "bf16"),
    (64, 128, "bf16"),      # exactly one tile
    (328, 640, "bf16"),     # several tiles and ragged slab
    (257, 1160, "f32"),
]


@pytest.fixture
def store_kernel(request):
    """Forces one of the two different-sample store kernels for the test, then restores the automatic choice."""
    import paper_2007_10412_b200 as rad
    prev = rad.rad_set_store_kernel(request.param)
    yield request.param
    rad.rad_set_store_kernel(prev)


# both kernels through the same cases (the automatic choice would send all of these to the generic
# one); the last two shapes span several chunks of the pipelined kernel with a ragged last chunk,
# slab and column block
@pytest.mark.parametrize("store_kernel", ["generic", "pipelined"], indirect=True)
@pytest.mark.parametrize("B,D,dtype", SHAPES + [(1000, 1160, "bf16"), (449, 2200, "f32")])
# thresholds with trailing zero digits need fewer generator outputs per word: 0.5 -> one, 416/4096 -> two,
# 1.0 -> none
@pytest.mark.parametrize("p", [0.1, 0.5, 1.0, 0.01, 416 / 4096])
def test_different_sample_store_is_bit_exact(B, D, dtype, p, store_kernel):
    import paper_2007_10412_b200 as rad
    A, _ = layer_inputs(B, D, 1, dtype=dtype, seed=B + D, relu_like=True)
    seed, layer, step = (1 << 40) + 12345, 3, 7
    ref = orc.forward_store(A, dtype, "different", p, seed, layer, step)
    st = rad.Store("different", dtype, B, D, p, seed=seed, layer=layer, step=step, capacity="worst")
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


@pytest.mark.parametrize("B,D,dtype", SHAPES)
@pytest.mark.parametrize("p", [0.1, 0.5, 1.0, 0.01])
def test_same_sample_store_is_bit_exact(B, D, dtype, p):
    import paper_2007_10412_b200 as rad
    A, _ = layer_inputs(B, D, 1, dtype=dtype, seed=B + D + 1, relu_like=True)
    seed, layer, step = 99, 1, 0
    ref = orc.forward_store(A, dtype, "same", p, seed, layer, step)
    st = rad.Store("same", dtype, B, D, p, seed=seed, layer=layer, step=step, capacity="worst")
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
    assert np.array_equal(u32(st.relubits).reshape(B, -1), ref.relubits)


def test_capacity_overflow_is_reported_not_faulted():
    import paper_2007_10412_b200 as rad
    B, D, p = 200, 512, 0.5
    A, _ = layer_inputs(B, D, 1, seed=1)
    ref = orc.forward_store(A, "f32", "different", p, 0, 0, 0)
    st = rad.Store("different", "f32", B, D, p, capacity=1024)
    guard = st.values.clone()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rad.rad_linear_forward_store(to_dev(A, "f32"), st, status)
    torch.cuda.synchronize()
    assert status.item() == rad.RAD_DEV_ECAPACITY
    assert st.nnz.cpu().numpy()[0] == ref.nnz          # counts stay exact
    del guard
    st2 = rad.Store("same", "f32", B, D, p, capacity=8)
    rad.rad_linear_forward_store(to_dev(A, "f32"), st2, status.zero_())
    torch.cuda.synchronize()
    assert status.item() == rad.RAD_DEV_ECAPACITY


def test_host_argument_checks():
    import paper_2007_10412_b200 as rad
    A = torch.zeros(8, 16, device="cuda")
    st = rad.Store("different", "f32", 8, 16, 0.5)
    st.c.p = 0.0
    with pytest.raises(rad.RadError, match="invalid argument"):
        rad.rad_linear_forward_store(A, st)
    st.c.p = 0.5
    st.workspace = st.workspace[:8]
    with pytest.raises(rad.RadError, match="workspace"):
        rad.rad_linear_forward_store(A, st)


def test_mask_is_independent_of_data_and_dtype():
    import paper_2007_10412_b200 as rad
    B, D, p = 130, 264, 0.2
    outs = []
    for dtype, seed in (("f32", 1), ("bf16", 2)):
        A, _ = layer_inputs(B, D, 1, dtype=dtype, seed=seed)
        st = rad.Store("different", dtype, B, D, p, seed=5, layer=1, step=2)
        rad.rad_linear_forward_store(to_dev(A, dtype), st)
        torch.cuda.synchronize()
        outs.append((u32(st.keepbits).copy(), u32(st.offsets).copy()))
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])


@pytest.mark.parametrize("p,relu", [(0.1, False), (0.3, True)])
def test_automatic_kernel_choice_on_a_layer_of_many_tiles(p, relu):
    """2145 tiles (33 ragged slabs x 65 ragged column blocks): large enough for the automatic choice
    to take the pipelined kernel, small enough for the oracle; every output bit for bit."""
    import paper_2007_10412_b200 as rad
    B, D, dtype = 2100, 8200, "bf16"
    A, _ = layer_inputs(B, D, 1, dtype=dtype, seed=77, relu_like=True)
    ref = orc.forward_store(A, dtype, "different", p, 99, 1, 4)
    st = rad.Store("different", dtype, B, D, p, seed=99, layer=1, step=4, relu_bits=relu)
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
    if relu:
        assert np.array_equal(u32(st.relubits).reshape(B, -1), ref.relubits)


def test_pipelined_kernel_reports_a_short_values_buffer():
    """Capacity overflow in the pipelined kernel: the status word is raised, counts stay exact, no fault."""
    import paper_2007_10412_b200 as rad
    B, D, p = 700, 1160, 0.5
    A, _ = layer_inputs(B, D, 1, dtype="bf16", seed=3)
    ref = orc.forward_store(A, "bf16", "different", p, 0, 0, 0)
    prev = rad.rad_set_store_kernel("pipelined")
    try:
        st = rad.Store("different", "bf16", B, D, p, capacity=4096)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        rad.rad_linear_forward_store(to_dev(A, "bf16"), st, status)
        torch.cuda.synchronize()
    finally:
        rad.rad_set_store_kernel(prev)
    assert status.item() == 1                     # RAD_DEV_ECAPACITY
    assert st.nnz.cpu().numpy()[0] == ref.nnz
