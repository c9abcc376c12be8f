"""The C-ABI library builds, loads without a GPU and exports every symbol include/rad.h declares."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "rad.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rad_[a-z_0-9]+)\s*\(", text)))


@pytest.fixture(scope="module")
def library():
    from paper_2007_10412_b200 import build
    return ctypes.CDLL(build.build())


def test_every_declared_symbol_is_exported(library):
    names = _declared()
    assert "rad_linear_forward_store" in names and "rad_linear_weight_grad" in names and "rad_mlp_step" in names
    for n in names:
        assert hasattr(library, n), n


def test_binding_covers_the_header():
    from paper_2007_10412_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()
    for n in binding.EXPORTS:
        assert hasattr(binding.lib(), n)


def test_host_only_entry_points():
    from oracle import rad as orc
    from paper_2007_10412_b200 import binding as b
    for p in (0.01, 0.05, 0.1, 0.2, 0.5, 1.0, 0.3333, 1e-7):
        assert b.rad_keep_threshold(p) == orc.keep_threshold(p)
        assert b.rad_scale(p) == float(orc.scale_factor(p))
        assert b.rad_effective_p(p) == pytest.approx(orc.effective_p(p), rel=1e-7)
    assert b.rad_keep_threshold(0.0) == 0 and b.rad_keep_threshold(1.5) == 0
    sz = b.rad_store_size_query("different", "bf16", 65536, 8192, 0.1)
    ntiles = 1024 * 64
    assert sz.keepbits_words == ntiles * 288 and sz.offsets_words == ntiles + 1
    assert sz.relubits_words == 65536 * 256
    assert sz.values_worst == 65536 * 8192 + 7 * ntiles
    assert 410 / 4096 * 65536 * 8192 < sz.values_typical < 1.01 * 410 / 4096 * 65536 * 8192
    sz = b.rad_store_size_query("same", "f32", 150, 784, 0.1)
    assert sz.values_ld_worst == 832 and sz.values_ld_typical % 64 == 0 and sz.values_ld_typical >= 128
    with pytest.raises(b.RadError):
        b.rad_store_size_query("same", "f32", 150, 784, 0.0)
    assert b.lib().rad_strerror(-4).decode() == "workspace too small"
    assert 1 <= b.rad_sm_pairs() <= 74
    # held without its keep bits: same values and offsets, no keep-bit words, the index of one layer in the workspace
    full = b.rad_store_size_query("different", "bf16", 65536, 8192, 0.1)
    held = b.rad_store_size_query("redrawn", "bf16", 65536, 8192, 0.1)
    assert held.keepbits_words == 0 and held.offsets_words == full.offsets_words
    assert held.values_typical == full.values_typical and held.values_worst == full.values_worst
    assert held.workspace_bytes >= full.workspace_bytes + ntiles * 288 * 4
    with pytest.raises(b.RadError):
        b.rad_store_size_query_law("redrawn", "bf16", "replace", 1000, 1160, 0.1)


def test_host_only_entry_points_of_the_with_replacement_law_and_the_kernel_choice():
    from oracle import rad as orc
    from paper_2007_10412_b200 import binding as b
    for f, D in [(0.1, 784), (0.1, 300), (0.5, 3), (1.0, 7), (0.05, 8192), (1e-9, 50), (0.3333, 1000)]:
        assert b.rad_draws_per_row(f, D) == orc.draws_per_row(f, D)
        assert np.float32(b.rad_replace_scale(f, D)) == orc.replace_scale(f, D)
    assert b.rad_draws_per_row(0.0, 10) == 0 and b.rad_draws_per_row(1.5, 10) == 0
    # the workspace of a different-sample store with this law holds a byte per entry on top of the status words
    plain = b.rad_store_size_query_law("different", "bf16", "bernoulli", 1000, 1160, 0.1)
    repl = b.rad_store_size_query_law("different", "bf16", "replace", 1000, 1160, 0.1)
    assert repl.workspace_bytes >= plain.workspace_bytes + 1000 * 1168
    k = orc.draws_per_row(0.1, 1160)
    mean = 1000 * 1160 * (1 - (1 - 1 / 1160) ** k)
    assert mean < repl.values_typical < 1.1 * mean + 16 * 10 * 7 + 2000
    assert b.rad_set_store_kernel("generic") == "auto"
    assert b.rad_set_store_kernel("pipelined") == "generic"
    assert b.rad_set_store_kernel("auto") == "pipelined"
    assert b.lib().rad_set_store_kernel(7) == -1


def test_held_bytes_from_the_counts_of_a_step():
    """rad_mlp_held_bytes is host arithmetic on the counts a step leaves: against the oracle's own accounting of
    the stores it builds for the same net (values only; the device pads every tile to a multiple of 8)."""
    import ctypes as C
    from oracle import rad as orc
    from workloads import mlp_inputs
    from paper_2007_10412_b200 import binding as b
    dims, B = (70, 52, 33, 10), 37
    X, y, Ws, bs = mlp_inputs(dims, B, "f32", "normal", 5)
    for variant in ("same", "different"):
        ref = orc.mlp_step(X, y, Ws, bs, dtype="f32", variant=variant, p=0.3, seed=4, step=1)
        want = orc.stored_bytes(ref.stores, (B, dims[-1]), 4)
        dims_c = (C.c_int64 * len(dims))(*dims)
        desc = b.rad_mlp_desc(len(dims) - 1, b.ACTS["relu"], b.DTYPES["f32"], b.VARIANTS[variant], dims_c, B, 0.3, 1, 4, 0)
        nnz = []
        for st in ref.stores:
            # different-sample: (kept entries, elements used with per-tile padding); same-sample: (k', B k')
            nnz += [st.nnz, st.nnz] if variant == "different" else [st.idx.size, st.nnz]
        arr = (C.c_int64 * len(nnz))(*nnz)
        stats = b.rad_step_stats()
        assert b.lib().rad_mlp_held_bytes(C.byref(desc), arr, C.byref(stats)) == 0
        assert stats.value_bytes == want["value_bytes"]
        assert stats.relu_bytes == want["relu_bytes"] and stats.unsampled_bytes == want["unsampled_bytes"]
        assert stats.full_backprop_bytes == want["full_backprop_bytes"]
        reserved = b.rad_step_stats()
        nbytes = C.c_int64(0)
        assert b.lib().rad_mlp_workspace(C.byref(desc), C.byref(nbytes), C.byref(reserved)) == 0
        assert reserved.value_bytes >= stats.value_bytes
    arr[1] = arr[0] - 1
    assert b.lib().rad_mlp_held_bytes(C.byref(desc), arr, C.byref(stats)) == -1
