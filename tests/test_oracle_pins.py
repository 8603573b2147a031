"""The CPU oracle against what the paper, the benchmark definition and mathematics fix."""
import os

import pytest

import oracle
from tests import pins

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "table1_kv_cache.txt")


@pytest.mark.parametrize("pin", pins.ALL_SELECT_PINS + pins.ALL_COMPACT_PINS + pins.ALL_ADJACENT_PINS, ids=lambda p: p.__name__)
def test_pin(pin):
    pin(oracle.default)


def test_cache_ratio_eq14():
    pins.pin_cache_ratio(oracle.default, GOLDEN)
