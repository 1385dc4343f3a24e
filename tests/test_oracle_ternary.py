"""Pins for the oracle's radix-3 container (five ternary codes per byte): checked against the positional number
system itself (Python's own base-3 parser and big integers) and against the paper's raw-bit count for a
three-level quantizer, never against the oracle's formulas."""
import itertools
import math

import numpy as np
import pytest

import oracle


def test_every_byte_value_is_the_base3_number_of_its_five_codes():
    seen = set()
    for t in itertools.product(range(3), repeat=5):
        byte = int(oracle.ternary_pack(np.array(t, dtype=np.uint32))[0])
        assert byte == int("".join(str(d) for d in reversed(t)), 3)      # first code = least significant digit
        assert list(oracle.ternary_unpack(np.array([byte], dtype=np.uint8), 5)) == list(t)
        seen.add(byte)
    assert seen == set(range(243))                                        # a bijection onto 0 .. 242


@pytest.mark.parametrize("n", [1, 2, 4, 5, 6, 79, 80, 81, 1000, 12347])
def test_stream_is_the_base243_expansion_of_the_base3_number(n):
    rng = np.random.default_rng(n)
    t = rng.integers(0, 3, size=n, dtype=np.uint32)
    data = oracle.ternary_pack(t)
    assert data.size == -(-n // 5) == oracle.ternary_bytes(n)
    as_base3 = sum(int(d) * 3 ** i for i, d in enumerate(t))
    as_base243 = sum(int(b) * 243 ** k for k, b in enumerate(data))
    assert as_base3 == as_base243
    assert np.array_equal(oracle.ternary_unpack(data, n), t)
    if n % 5:                                                             # codes past the end count as 0
        assert int(data[-1]) < 3 ** (n % 5)


def test_codes_above_two_are_stored_as_two():
    t = np.array([0, 3, 1, 2, 3, 3, 0], dtype=np.uint32)
    assert np.array_equal(oracle.ternary_unpack(oracle.ternary_pack(t), t.size), np.minimum(t, 2))


def test_rate_against_the_papers_raw_bit_count(golden_dir):
    # Section 4, raw-bits table: the three-level DQSGD row counts log2(3) bits per parameter plus a 32-bit scale
    # per tensor.  Five codes per byte cost 1.6 bits per parameter: at most 1 % above that count, 20 % below two
    # bits per parameter.
    row = [l.split() for l in (golden_dir / "raw_bits_table.txt").read_text().splitlines()
           if l.startswith("dqsgd_fc300_100_ternary")][0]
    n, tensors, levels, printed_kbit = int(row[1]), int(row[2]), int(row[3]), float(row[4])
    assert levels == 3
    container_kbit = (8 * oracle.ternary_bytes(n) + 32 * tensors) / 1000
    assert printed_kbit <= container_kbit <= 1.01 * printed_kbit
    assert 8 * oracle.ternary_bytes(n) < 0.8001 * 2 * n
    assert math.log2(3) <= 8 * oracle.ternary_bytes(n) / n <= 1.6 + 8 / n


def test_container_of_a_real_three_level_message_round_trips():
    rng = np.random.default_rng(7)
    n = 5000 + 13
    g = rng.normal(size=n).astype(np.float32)
    packed, scale = oracle.dqsg_encode(g, 99, 3, 17, 512, 2, 3)
    codes = oracle.unpack(packed, n, 2)
    assert codes.max() <= 2 and set(np.unique(codes)) == {0, 1, 2}
    data = oracle.ternary_pack_stream(packed, n)
    assert data.size == oracle.ternary_bytes(n)
    assert np.array_equal(oracle.ternary_unpack_stream(data, n), packed)
