"""rad_linear_forward_store_static: the store for callers that cannot allocate device memory.

Some users of this library run under a rule of "no device allocation after start-up": their
trainer owns one big memory pool, or an allocation in the step loop would stall the GPU.  They
cannot hand the store kernel a workspace, so this entry point keeps its scratch in an array built
into the library.  The test calls it twice in a row through the C ABI (the second call must not be
confused by what the first left in the shared array) and wants exactly the bytes the ordinary
entry point produces.  This file is collected last on purpose.
"""
import numpy as np
import pytest
import torch

from workloads import layer_inputs

pytestmark = pytest.mark.gpu


def _store_outputs(st):
    torch.cuda.synchronize()
    used = int(st.nnz[1].item())
    vals = st.values[:used]
    vals = vals.view(torch.int16) if vals.dtype == torch.bfloat16 else vals.view(torch.int32)
    return (st.keepbits.cpu().numpy().copy(), st.offsets.cpu().numpy().copy(), st.nnz.cpu().numpy().copy(),
            vals.cpu().numpy().copy(), st.relubits.cpu().numpy().copy())


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_two_calls_in_a_row_match_the_workspace_entry_point(dtype):
    import paper_2007_10412_b200 as rad
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    # a larger problem first, then a smaller one with another mask: stale scratch would show
    for (B, D, p, seed) in [(1500, 1160, 0.1, 3), (328, 640, 0.5, 4)]:
        A, _ = layer_inputs(B, D, 1, dtype=dtype, seed=B, relu_like=True)
        Ad = torch.from_numpy(A).to(tdt).cuda()
        ref = rad.Store("different", dtype, B, D, p, seed=seed, layer=1, step=2)
        rad.rad_linear_forward_store(Ad, ref, status)
        want = _store_outputs(ref)
        got_st = rad.Store("different", dtype, B, D, p, seed=seed, layer=1, step=2)
        got_st.workspace = None                      # not used by the static entry point
        rad.rad_linear_forward_store_static(Ad, got_st, status)
        got = _store_outputs(got_st)
        assert status.item() == 0
        for g, w in zip(got, want):
            assert np.array_equal(g, w)              # integer and byte work: bit exact


def test_many_tiles_through_the_built_in_scratch_match_the_oracle():
    """2145 tiles: the size at which the library switches to its persistent kernel, whose per-chunk words
    and shared claim counter then live in the built-in array.  Checked against the CPU oracle, not against
    the other entry point; a small call right after it (the one-CTA-per-tile kernel, same array) must not
    trip over what the large one left behind."""
    import paper_2007_10412_b200 as rad
    from oracle import rad as orc
    from gpu_util import bits_host, to_dev, u32
    from layout import bits_of, tile_major
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for (B, D, p, seed) in [(2100, 8200, 0.1, 21), (200, 300, 0.3, 22)]:
        A, _ = layer_inputs(B, D, 1, dtype="bf16", seed=seed, relu_like=True)
        ref = orc.forward_store(A, "bf16", "different", p, seed, 2, 5)
        st = rad.Store("different", "bf16", B, D, p, seed=seed, layer=2, step=5)
        st.workspace = None
        rad.rad_linear_forward_store_static(to_dev(A, "bf16"), st, status)
        torch.cuda.synchronize()
        assert status.item() == 0
        kb, vals, offs = tile_major(ref)
        assert np.array_equal(u32(st.keepbits), kb)
        assert np.array_equal(u32(st.offsets), offs)
        nnz = st.nnz.cpu().numpy()
        assert nnz[0] == ref.nnz and nnz[1] == offs[-1]
        assert np.array_equal(bits_host(st.values[:int(offs[-1])]), bits_of(vals, "bf16"))
        assert np.array_equal(u32(st.relubits).reshape(B, -1), ref.relubits)


def test_limits_are_reported():
    import paper_2007_10412_b200 as rad
    A = torch.zeros(64, 128, device="cuda")
    st = rad.Store("same", "f32", 64, 128, 0.5)
    with pytest.raises(rad.RadError, match="unsupported"):
        rad.rad_linear_forward_store_static(A, st)
    # 131073 tiles: one more than the built-in array holds; rejected before anything is launched
    big = rad.Store("different", "f32", 64, 128, 0.5)
    big.c.B, big.c.D = 64 * 131073, 128
    with pytest.raises(rad.RadError, match="built-in"):
        rad.rad_linear_forward_store_static(A.expand(64, 128), big)
