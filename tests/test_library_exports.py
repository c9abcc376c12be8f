"""The C-ABI library builds, loads without a GPU and exports every symbol include/rad.h declares."""
import ctypes
import os
import re

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
    assert 26 / 256 * 65536 * 8192 < sz.values_typical < 1.01 * 26 / 256 * 65536 * 8192
    sz = b.rad_store_size_query("same", "f32", 150, 784, 0.1)
    assert sz.values_ld_worst == 832 and sz.values_ld_typical % 64 == 0 and sz.values_ld_typical >= 128
    with pytest.raises(b.RadError):
        b.rad_store_size_query("same", "f32", 150, 784, 0.0)
    assert b.lib().rad_strerror(-4).decode() == "workspace too small"
