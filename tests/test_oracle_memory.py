"""The oracle's byte accounting reproduces the figures the paper prints (App. A, Table 1)."""
import os

import pytest

from oracle import memory_model as mm

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_memory_figures.txt")


def _rows():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.split("|")[0].strip()
            if not line or line.startswith("#"):
                continue
            net, quantity, fraction, value, unit = line.split()
            rows.append((net, quantity, float(fraction), float(value), unit))
    return rows


@pytest.mark.parametrize("net,quantity,fraction,value,unit", _rows())
def test_paper_figure(net, quantity, fraction, value, unit):
    if quantity == "per_element":
        assert mm.per_element_bytes(net, fraction) == pytest.approx(value, abs=1e-9)
    else:
        # Table 1 prints two decimals; most entries are the rounded figure, the RNN row is
        # truncated and the MLP entry at 0.5 is 2.2045 printed as 2.21: accept less than one
        # unit of the last printed digit.
        assert abs(mm.table1_megabytes(net, fraction) - value) < 0.01


def test_savings_ratios_quoted_in_text():
    # "approximately 8x", "7.5x", "7.15x" savings per minibatch element (App. A)
    assert mm.per_element_bytes("mlp", 1.0) / mm.per_element_bytes("mlp", 0.1) == pytest.approx(8.18, abs=0.01)
    assert mm.per_element_bytes("cnn", 1.0) / mm.per_element_bytes("cnn", 0.1) == pytest.approx(7.75, abs=0.01)
    assert mm.per_element_bytes("rnn", 1.0) / mm.per_element_bytes("rnn", 0.1) == pytest.approx(7.15, abs=0.01)
