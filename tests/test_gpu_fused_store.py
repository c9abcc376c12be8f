"""The store produced where the activation already is: rad_store_index (index part from the key alone) and
rad_linear_forward_fill (forward GEMM whose epilogue drops the kept activations into the next layer's
store), against the oracle's store of the very activations the call wrote."""
import numpy as np
import pytest
import torch

from oracle import rad as orc
from workloads import layer_inputs, mlp_inputs

from gpu_util import bits_host, to_dev, to_host_f32, u32
from layout import bits_of, tile_major

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,D", [(1, 1), (64, 128), (150, 300), (328, 640), (257, 1160), (1000, 2200)])
@pytest.mark.parametrize("p", [0.01, 0.1, 0.5, 1.0])
def test_index_from_the_key_alone_is_bit_exact(B, D, p):
    """Keep bits, row offsets, tile offsets and both counts without any layer input: they equal the index
    part of the oracle's store of an arbitrary input of that shape."""
    import paper_2007_10412_b200 as rad
    seed, layer, step = (7 << 33) + 5, 4, 9
    A = np.ones((B, D), np.float32)
    ref = orc.forward_store(A, "f32", "different", p, seed, layer, step, with_relu_bits=False)
    st = rad.Store("different", "f32", B, D, p, seed=seed, layer=layer, step=step, relu_bits=False, capacity="worst")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rad.rad_store_index(st, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    kb, _, offs = tile_major(ref)
    assert np.array_equal(u32(st.keepbits), kb)
    assert np.array_equal(u32(st.offsets), offs)
    nnz = st.nnz.cpu().numpy()
    assert nnz[0] == ref.nnz and nnz[1] == offs[-1]


def test_index_reports_a_short_values_buffer_and_rejects_other_variants():
    import paper_2007_10412_b200 as rad
    st = rad.Store("different", "bf16", 300, 512, 0.5, capacity=1024)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rad.rad_store_index(st, status)
    torch.cuda.synchronize()
    assert status.item() == rad.RAD_DEV_ECAPACITY
    ref = orc.keep_mask("different", 300, 512, 0.5, 0, 0, 0)
    assert st.nnz.cpu().numpy()[0] == ref.sum()
    with pytest.raises(rad.RadError, match="unsupported"):
        rad.rad_store_index(rad.Store("same", "bf16", 64, 128, 0.5))
    with pytest.raises(rad.RadError, match="unsupported"):
        rad.rad_store_index(rad.Store("different", "bf16", 64, 128, 0.5, law="replace"))


def _check_fill(B, D, H, dtype, act, variant, p, law="bernoulli", index_ready=False, relu=True):
    import paper_2007_10412_b200 as rad
    X, _, Ws, bs = mlp_inputs((D, H), B, dtype=dtype, x_dist="normal", seed=B + H, bias_zero=False)
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    seed, layer, step = 1234567, 2, 6
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Xd, Wd, bd = to_dev(X, dtype), to_dev(Ws[0], dtype), to_dev(bs[0], "f32")
    w32 = (H + 31) // 32
    # the two separate calls
    act_ref = torch.empty(B, H, dtype=tdt, device="cuda")
    zl_ref = torch.empty(B, H, dtype=tdt, device="cuda")
    rb_ref = torch.zeros(B * w32, dtype=torch.int32, device="cuda")
    rad.rad_linear_forward(Xd, Wd, bd, act, out_act=act_ref, out_zlow=zl_ref, relubits=rb_ref, dev_status=status)
    # the fused call
    out_act = torch.full((B, H), float("nan"), dtype=tdt, device="cuda")
    zl = torch.empty(B, H, dtype=tdt, device="cuda")
    rb = torch.zeros(B * w32, dtype=torch.int32, device="cuda") if relu else None
    st = rad.Store(variant, dtype, B, H, p, seed=seed, layer=layer, step=step, relu_bits=False, law=law)
    st.values.fill_(float("nan"))
    if index_ready:
        rad.rad_store_index(st, status)
    rad.rad_linear_forward_fill(Xd, Wd, bd, act, out_act, st, out_zlow=zl, relubits=rb, index_ready=index_ready,
                                dev_status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert torch.equal(out_act.view(torch.int16 if dtype == "bf16" else torch.int32),
                       act_ref.view(torch.int16 if dtype == "bf16" else torch.int32))
    assert torch.equal(zl, zl_ref)
    if relu:
        assert torch.equal(rb, rb_ref)
    # the oracle's store of the activations the device wrote
    a_host = to_host_f32(out_act)
    ref = orc.forward_store(a_host, dtype, variant, p, seed, layer, step, with_relu_bits=False, law=law)
    nnz = st.nnz.cpu().numpy()
    if variant == "different":
        kb, vals, offs = tile_major(ref)
        assert np.array_equal(u32(st.keepbits), kb)
        assert np.array_equal(u32(st.offsets), offs)
        assert nnz[0] == ref.nnz and nnz[1] == offs[-1]
        assert np.array_equal(bits_host(st.values[:int(offs[-1])]), bits_of(vals, dtype))
    else:
        k = ref.idx.size
        assert nnz[0] == k
        ld = st.c.values_ld
        got = bits_host(st.values[:B * ld]).reshape(B, ld)
        assert np.array_equal(got[:, :k], bits_of(ref.values, dtype).reshape(B, k))


@pytest.mark.parametrize("B,D,H", [(328, 640, 520), (328, 392, 200), (1024, 256, 512), (200, 128, 1160), (64, 64, 64)])
@pytest.mark.parametrize("act", ["relu", "gelu"])
@pytest.mark.parametrize("p", [0.1, 0.5, 1.0, 0.01])
def test_fused_store_matches_the_oracle_store_of_the_written_activations(B, D, H, act, p):
    _check_fill(B, D, H, "bf16", act, "different", p)


@pytest.mark.parametrize("f", [0.1, 0.5])
def test_fused_store_under_the_fixed_count_law(f):
    """Exactly k columns per row: the index of that law also comes from the key alone, so the same epilogue fills it."""
    _check_fill(328, 640, 520, "bf16", "relu", "different", f, law="fixed")
    _check_fill(200, 128, 1160, "bf16", "gelu", "different", f, law="fixed", index_ready=True, relu=False)


def test_fused_store_with_the_index_made_beforehand():
    _check_fill(520, 384, 648, "bf16", "gelu", "different", 0.2, index_ready=True, relu=False)


@pytest.mark.parametrize("B,D,H,dtype,variant,law", [(150, 784, 300, "f32", "different", "bernoulli"),
                                                     (150, 300, 300, "bf16", "different", "bernoulli"),
                                                     (328, 640, 520, "bf16", "same", "bernoulli"),
                                                     (328, 640, 520, "bf16", "different", "replace")])
def test_shapes_the_fused_kernel_does_not_take_give_the_same_results(B, D, H, dtype, variant, law):
    _check_fill(B, D, H, dtype, "relu", variant, 0.1, law=law)


def test_fused_store_reports_a_short_values_buffer():
    import paper_2007_10412_b200 as rad
    B, D, H, p = 328, 256, 512, 0.5
    X, _, Ws, bs = mlp_inputs((D, H), B, dtype="bf16", x_dist="normal", seed=3)
    st = rad.Store("different", "bf16", B, H, p, relu_bits=False, capacity=4096)
    guard = torch.full((1 << 16,), 7.0, dtype=torch.bfloat16, device="cuda")    # allocated right after `values`
    out_act = torch.empty(B, H, dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rad.rad_linear_forward_fill(to_dev(X, "bf16"), to_dev(Ws[0], "bf16"), to_dev(bs[0], "f32"), "relu", out_act, st,
                                dev_status=status)
    torch.cuda.synchronize()
    assert status.item() == rad.RAD_DEV_ECAPACITY
    assert (guard == 7.0).all()
    assert st.nnz.cpu().numpy()[0] == orc.keep_mask("different", B, H, p, 0, 0, 0).sum()
