"""The CPU oracle against what the paper and the mathematics fix (no GPU needed)."""
import os

import pytest

import oracle_pins as pins

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


@pytest.mark.parametrize("pin", pins.ALL_PINS, ids=lambda f: f.__name__)
def test_pin(pin):
    pin()


def test_effective_bits_match_table1():
    pins.pin_effective_bits(os.path.join(GOLDEN, "table1_effective_bits.txt"))


def test_every_bf16_pattern_as_single_nonzero_block():
    pins.pin_single_nonzero_block_truncates()
