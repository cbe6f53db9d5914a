"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU)."""
import pytest

import pins
from oracle import OracleGraph


def make_graph(n, edges, w, m, C):
    return OracleGraph(n, edges, w, m, C)


@pytest.mark.parametrize("pin", pins.ALL_PINS, ids=lambda f: f.__name__)
def test_pin(pin):
    pin(make_graph)
