"""Pins for the oracle's 16-bit dither stream (eight elements per Philox block): layout against the raw
Philox block function, the exact grid, and the same statistical laws as the 32-bit stream."""
import math

import numpy as np
import pytest
from scipy import stats

import oracle

SEED = 0x0FED_CBA9_8765_4321


def test_half_word_layout_against_the_block_function():
    seed, worker, step = SEED, 3, (7 << 32) | 11
    for i in (0, 1, 2, 7, 8, 9, 1023, 1024, (1 << 35) + 5):
        blk = oracle.philox4x32_10([(i >> 3) & 0xFFFFFFFF, worker, 11, 7], [seed & 0xFFFFFFFF, seed >> 32])
        word = blk[(i & 7) >> 1]
        want = (word >> 16) if (i & 1) else (word & 0xFFFF)
        assert oracle.dither16_half(seed, worker, step, i) == want


def test_grid_is_exact_and_symmetric():
    assert oracle.dither16_from_half(0) == -0.5 + 2.0 ** -17
    assert oracle.dither16_from_half(65535) == 0.5 - 2.0 ** -17
    for h in (0, 1, 2, 32767, 32768, 40000, 65534, 65535):
        d = oracle.dither16_from_half(h)
        assert d == (2 * h + 1) * 2.0 ** -17 - 0.5
        assert oracle.dither16_from_half(65535 - h) == -d and d != 0.0 and abs(d) < 0.5


def test_stream_statistics_and_separation():
    n = 200_000
    d = oracle.dither_vector(SEED, 1, 5, n, dither_bits=16).astype(np.float64)
    assert abs(d.mean()) < 5 * math.sqrt(1 / 12 / n)
    assert abs(d.var() - 1 / 12) < 0.01 / 12
    assert stats.kstest(d + 0.5, "uniform").pvalue > 1e-3
    assert abs(np.corrcoef(d[:-1], d[1:])[0, 1]) < 5 / math.sqrt(n)          # neighbours share a word, not a value
    assert not np.array_equal(d[:64], oracle.dither_vector(SEED, 2, 5, 64, dither_bits=16))
    assert not np.array_equal(d[:64].astype(np.float32), oracle.dither_vector(SEED, 1, 5, 64, dither_bits=32))


@pytest.mark.parametrize("bits,levels", [(1, 2), (2, 3), (3, 5), (4, 15)])
def test_dqsg_error_law_with_16_bit_dither(bits, levels):
    rng = np.random.default_rng(30 + bits)
    n, B = 1 << 17, 2048
    g = (rng.standard_normal(n) * 0.05).astype(np.float32)
    pk, sc, codes = oracle.dqsg_encode(g, SEED, 2, 9, B, bits, levels, want_codes=True, dither_bits=16)
    m = oracle.Msg(pk, sc, SEED, 2, oracle.KIND_DQSG, B, bits, levels, dither_bits=16)
    rec = oracle.decode_aggregate([m], n, 9)
    kappa = np.repeat(sc.astype(np.float64), B)
    Delta = 2.0 / (levels - 1)
    e = (rec.astype(np.float64) - g) / kappa / Delta
    assert np.abs(e).max() <= 0.5 + 1e-5
    assert abs(e.mean()) < 5 / math.sqrt(12 * n)
    assert abs(e.var() - 1 / 12) < 0.02 / 12
    assert stats.kstest(e + 0.5, "uniform").pvalue > 1e-3
    assert abs(np.corrcoef(e, g / kappa)[0, 1]) < 5 / math.sqrt(n)
    # a message decoded with the other stream is wrong by up to a whole step: the streams really differ
    wrong = oracle.decode_aggregate([oracle.Msg(pk, sc, SEED, 2, oracle.KIND_DQSG, B, bits, levels)], n, 9)
    assert np.abs((wrong.astype(np.float64) - g) / kappa / Delta).max() > 0.6


def test_ndqsg_with_16_bit_dither_recovers_in_cell_and_matches_dqsg():
    rng = np.random.default_rng(40)
    n, B, K, M1, bits = 1 << 15, 512, 4, 4.0, 2
    y = rng.uniform(-0.8, 0.8, n).astype(np.float32)
    z = rng.uniform(-0.33, 0.33, n).astype(np.float32)          # inside (K-1)/(2 M1) = 0.375
    g = (y + z).astype(np.float32)
    g[::B] = 1.0
    y[::B] = 1.0
    pk, sc, q1 = oracle.ndqsg_encode(g, SEED, 4, 2, B, bits, K, M1, 1.0, want_q1=True, dither_bits=16)
    m = oracle.Msg(pk, sc, SEED, 4, oracle.KIND_NDQSG, B, bits, coarse_K=K, fine_M=M1, dither_bits=16)
    _, rec, qhat = oracle.decode_aggregate([m], n, 2, side_info=y, want_recon=True, want_qhat=True)
    assert np.array_equal(qhat[0], q1)
    dp, ds, dk = oracle.dqsg_encode(g, SEED, 4, 2, B, 4, 9, want_codes=True, dither_bits=16)
    drec = oracle.decode_aggregate([oracle.Msg(dp, ds, SEED, 4, oracle.KIND_DQSG, B, 4, 9, dither_bits=16)], n, 2)
    same = (dk - 4) == q1
    assert same.mean() > 0.9999 and np.array_equal(rec[0][same], drec[same])


def test_oracle_rejects_unknown_stream():
    with pytest.raises(ValueError):
        oracle.dqsg_encode(np.zeros(64, np.float32), 1, 0, 0, 32, 2, dither_bits=8)
