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


def test_e4m3_bytes_match_the_hand_worked_table():
    import numpy as np
    from oracle import fb4_oracle as orc
    table = {}
    for line in open(os.path.join(GOLDEN, "e4m3_of_integers_0_to_15.txt")):
        if line.strip() and not line.startswith("#"):
            k, b = line.split()
            table[int(k)] = int(b, 16)
    assert sorted(table) == list(range(16))
    FB = pins.FB
    # one block per dialect, codes 0..7 and 8..15 (negative) in turn, scale byte 127 (scale 1)
    codes = np.tile(np.array([0x10, 0x32, 0x54, 0x76, 0x98, 0xBA, 0xDC, 0xFE], np.uint8), (32, 2))
    meta = (127 | (np.arange(32) << 8)).astype(np.uint16).reshape(32, 1)
    e, sc = orc.to_mxfp8(orc.Quantized(codes, meta), FB, 0)
    assert np.all(sc == 127)
    for d in range(32):
        for i in range(32):
            idx, neg = i % 16 % 8, (i % 16) >= 8
            assert int(e[d, i]) == (table[int(FB[d, idx])] | (0x80 if neg else 0))
