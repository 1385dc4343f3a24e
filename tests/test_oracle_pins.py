"""Pins for the CPU oracle: everything here checks ``oracle/`` against facts the paper or the
mathematics fix, never against the oracle's own formulas and never against the CUDA path."""
import math

import numpy as np
import pytest
from scipy import stats

import oracle

SEED = 0x1234_5678_9ABC_DEF0


# ------------------------------------------------------------------ Philox
def test_philox_known_answers(golden_dir):
    rows = [l.split() for l in (golden_dir / "philox4x32_10_kat.txt").read_text().splitlines()
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        assert oracle.philox4x32_10(v[0:4], v[4:6]) == v[6:10]


def test_philox_counter_layout():
    # element i uses block i//4, word i%4; key = (lo32(seed), hi32(seed)); counter = (i//4, worker, step lo, step hi)
    seed, worker, step = SEED, 7, (5 << 32) | 9
    for i in (0, 1, 2, 3, 4, 1023, (1 << 34) + 6):
        blk = oracle.philox4x32_10([(i >> 2) & 0xFFFFFFFF, worker, 9, 5], [seed & 0xFFFFFFFF, seed >> 32])
        assert oracle.dither_bits(seed, worker, step, i) == blk[i & 3]


# ------------------------------------------------------------------ dither
def test_dither_grid_symmetry_and_extremes():
    # grid {(2j+1) 2^-23 - 1/2}: symmetric, never 0 or +-1/2
    assert oracle.dither_from_bits(0) == -0.5 + 2.0 ** -23
    assert oracle.dither_from_bits(0xFFFFFFFF) == 0.5 - 2.0 ** -23
    rng = np.random.default_rng(1)
    for x in rng.integers(0, 2 ** 32, size=2000, dtype=np.uint64):
        x = int(x)
        d = oracle.dither_from_bits(x)
        assert -0.5 < d < 0.5 and d != 0.0
        assert oracle.dither_from_bits(x ^ 0xFFFFFFFF) == -d          # complementing the bits mirrors the dither
        j = x >> 10
        assert d == (2 * j + 1) * 2.0 ** -23 - 0.5                      # exact in double


def test_dither_uniform_statistics():
    n = 200_000
    d = oracle.dither_vector(SEED, 3, 11, n).astype(np.float64)
    assert abs(d.mean()) < 5 * math.sqrt(1 / 12 / n)
    assert abs(d.var() - 1 / 12) < 0.01 * (1 / 12)
    assert stats.kstest(d + 0.5, "uniform").pvalue > 1e-3
    # different workers / steps / seeds give different streams
    assert not np.array_equal(d[:64], oracle.dither_vector(SEED, 4, 11, 64))
    assert not np.array_equal(d[:64], oracle.dither_vector(SEED, 3, 12, 64))
    assert not np.array_equal(d[:64], oracle.dither_vector(SEED + 1, 3, 11, 64))


# ------------------------------------------------------------------ worked example (Section 3.2)
def _golden_kv(path):
    kv = {}
    for l in path.read_text().splitlines():
        if l.strip() and not l.startswith("#"):
            k, *v = l.split()
            kv[k] = [float(x) for x in v]
    return kv


def test_paper_worked_nested_example(golden_dir):
    g = _golden_kv(golden_dir / "nested_example.txt")
    D1, D2, al = g["Delta1"][0], g["Delta2"][0], g["alpha"][0]
    x, u, y = g["x"][0], g["u"][0], g["y"][0]
    t = al * x + u
    assert t == pytest.approx(g["t"][0], abs=1e-12)
    assert oracle.Q(t, D1) == g["Q1_t"][0]
    assert oracle.Q(t, D2) == g["Q2_t"][0]
    s = oracle.nested_encode_scalar(x, u, D1, D2, al)
    assert s == g["s"][0]
    assert oracle.nested_decode_scalar(s, u, y, D2, al) == pytest.approx(g["x_hat"][0], abs=1e-12)
    for xa in g["alias_same_s"]:
        assert oracle.nested_encode_scalar(xa, u, D1, D2, al) == g["s"][0]
    # the printed 2.7 does not give the same s (see the fixture's header)
    assert oracle.nested_encode_scalar(g["printed_alias_inconsistent"][0], u, D1, D2, al) == 0.0
    # modulo form used on the wire: q1 = -4, K = 3 -> m = 2, which is s = -1 modulo 3
    assert (int(oracle.Q(t, D1)) % 3) == 2 == int(s) % 3


def test_scalar_dithered_quantizer_bound_and_nestedness():
    rng = np.random.default_rng(2)
    for _ in range(500):
        D = float(rng.uniform(0.05, 2))
        x = float(rng.uniform(-5, 5))
        u = float(rng.uniform(-D / 2, D / 2))
        assert abs(oracle.dithered(x, u, D) - x) <= D / 2 + 1e-12      # |x~ - x| <= Delta/2
        k = int(rng.integers(2, 9))
        assert oracle.Q(oracle.Q(x, k * D), D) == pytest.approx(oracle.Q(x, k * D), abs=1e-9)  # Q1(Q2(x)) = Q2(x)


# ------------------------------------------------------------------ helpers
def _dqsg_roundtrip(g, bucket, bits, levels=0, seed=SEED, worker=1, step=3):
    packed, scale, codes = oracle.dqsg_encode(g, seed, worker, step, bucket, bits, levels, want_codes=True)
    msg = oracle.Msg(packed, scale, seed, worker, oracle.KIND_DQSG, bucket, bits, levels)
    rec = oracle.decode_aggregate([msg], g.size, step)
    return packed, scale, codes, rec


# ------------------------------------------------------------------ DQSG error law (Schuchman; Section 3.1)
@pytest.mark.parametrize("bits,levels", [(1, 2), (2, 3), (3, 5), (3, 7), (4, 15), (8, 255), (2, 4)])
def test_dqsg_error_is_bounded_uniform_and_independent(bits, levels):
    rng = np.random.default_rng(3)
    n, B = 1 << 17, 1024
    g = (rng.standard_normal(n) * 0.01).astype(np.float32)
    _, scale, codes, rec = _dqsg_roundtrip(g, B, bits, levels)
    kappa = np.repeat(scale.astype(np.float64), B)[:n]
    assert np.array_equal(scale, np.abs(g).reshape(-1, B).max(axis=1))
    Delta = 2.0 / (levels - 1)
    e = (rec.astype(np.float64) - g.astype(np.float64)) / kappa / Delta      # error in units of Delta
    assert np.abs(e).max() <= 0.5 + 1e-5
    assert abs(e.mean()) < 5 / math.sqrt(12 * n)
    assert abs(e.var() - 1 / 12) < 0.02 * (1 / 12)
    assert stats.kstest(e + 0.5, "uniform").pvalue > 1e-3
    # independent of the signal: no correlation with g or |g|, and the conditional variance is flat
    x = g / kappa
    assert abs(np.corrcoef(e, x)[0, 1]) < 5 / math.sqrt(n)
    assert abs(np.corrcoef(e * e, np.abs(x))[0, 1]) < 5 / math.sqrt(n)
    assert codes.min() >= 0 and codes.max() <= levels - 1                      # indices in {-M..M} + M


def test_dqsg_unbiased_over_iterations():
    rng = np.random.default_rng(4)
    n, B, T = 256, 64, 4000
    g = rng.uniform(-1, 1, n).astype(np.float32)
    acc = np.zeros(n)
    for step in range(T):
        acc += _dqsg_roundtrip(g, B, 2, 3, step=step)[3]
    kappa = np.repeat(np.abs(g).reshape(-1, B).max(axis=1), B)
    z = (acc / T - g) / (kappa * 1.0 / math.sqrt(12 * T))                      # Delta = 1 for L = 3
    assert np.abs(z).max() < 5.5
    assert abs(z.mean()) < 5 / math.sqrt(n)


def test_dqsg_decoded_with_another_dither_stream_triples_the_error():
    """A message decoded with the wrong seed or step (a corrupt header): the receiver subtracts a dither u' that is
    independent of the sender's u, so the error in units of Delta is e + u - u' with e, u, u' independent and
    uniform on (-1/2, 1/2): variance 3/12 instead of 1/12, and no longer bounded by 1/2.  (Schuchman's condition,
    Section 3.1: only the SAME dither makes the error independent of the signal.)"""
    rng = np.random.default_rng(31)
    n, B, levels = 1 << 17, 1024, 15
    g = (rng.standard_normal(n) * 0.01).astype(np.float32)
    packed, scale, _ = oracle.dqsg_encode(g, SEED, 1, 3, B, 4, levels, want_codes=True)
    kappa = np.repeat(scale.astype(np.float64), B)[:n]
    Delta = 2.0 / (levels - 1)
    for seed, worker, step in ((SEED + 1, 1, 3), (SEED, 2, 3), (SEED, 1, 4)):
        msg = oracle.Msg(packed, scale, seed, worker, oracle.KIND_DQSG, B, 4, levels)
        rec = oracle.decode_aggregate([msg], n, step)
        e = (rec.astype(np.float64) - g.astype(np.float64)) / kappa / Delta
        assert abs(e.var() - 3 / 12) < 0.03 * (3 / 12), (seed, worker, step, e.var())
        assert np.abs(e).max() > 1.0                                            # up to 3/2, never above
        assert np.abs(e).max() <= 1.5 + 1e-5


# ------------------------------------------------------------------ Appendix A: selection probabilities
@pytest.mark.parametrize("M,x", [(1, 0.3), (2, 0.3), (2, -0.7), (3, 0.95)])
def test_level_selection_probabilities(M, x):
    # for l/M <= |x| < (l+1)/M and d = |x| - l/M:  P(l/M) = 1 - M d,  P((l+1)/M) = M d
    n, B = 1 << 18, 65536
    g = np.full(n, x, dtype=np.float32)
    g[::B] = 1.0                                   # kappa = 1 in every bucket
    L = 2 * M + 1
    bits = max(2, math.ceil(math.log2(L)))
    codes = oracle.dqsg_encode(g, SEED, 2, 5, B, bits, L, want_codes=True)[2]
    q = codes.astype(np.int64) - M
    keep = np.ones(n, bool)
    keep[::B] = False
    q = q[keep]
    ax = abs(float(np.float32(x)))
    l = math.floor(ax * M)
    d = ax - l / M
    sgn = 1 if x > 0 else -1
    p_hi = float(np.mean(q == sgn * (l + 1)))
    p_lo = float(np.mean(q == sgn * l))
    assert p_hi + p_lo == 1.0
    tol = 5 * math.sqrt(0.25 / q.size)
    assert abs(p_hi - M * d) < tol and abs(p_lo - (1 - M * d)) < tol
    # half-dithered (no subtraction at the receiver) variance: (|x|-l/M)((l+1)/M-|x|)
    var_half = float(np.mean((q / M - x) ** 2))
    assert var_half == pytest.approx(d * (1 / M - d), rel=0.03, abs=1e-4)


def test_half_dithered_average_variance_is_twice_dithered():
    # x ~ U[-1,1]: stochastic quantization averages 1/(6 M^2), the subtractive dither 1/(12 M^2)
    rng = np.random.default_rng(5)
    n, B, M = 1 << 18, 65536, 2
    g = rng.uniform(-1, 1, n).astype(np.float32)
    g[::B] = 1.0
    _, _, codes, rec = _dqsg_roundtrip(g, B, 3, 2 * M + 1)
    half = (codes.astype(np.float64) - M) / M
    assert np.mean((half - g) ** 2) == pytest.approx(1 / (6 * M * M), rel=0.02)
    assert np.mean((rec.astype(np.float64) - g) ** 2) == pytest.approx(1 / (12 * M * M), rel=0.02)


# ------------------------------------------------------------------ rate accounting (raw-bits table)
def test_raw_bits_table(golden_dir):
    assert 784 * 300 + 300 + 300 * 100 + 100 + 100 * 10 + 10 == 266610
    for l in (golden_dir / "raw_bits_table.txt").read_text().splitlines():
        if not l.strip() or l.startswith("#"):
            continue
        name, n, tensors, levels, printed = l.split()
        n, tensors, levels, printed = int(n), int(tensors), int(levels), float(printed)
        if levels == 2 ** 32:
            kbit = 32 * n / 1000
        else:
            kbit = oracle.raw_bits(n, levels, tensors) / 1000
        assert abs(kbit - printed) < 0.06, name
    # levels = 2M+1 and the default level count for b bits
    assert [oracle.default_levels(b) for b in range(1, 9)] == [2, 3, 7, 15, 31, 63, 127, 255]


# ------------------------------------------------------------------ bit stream
@pytest.mark.parametrize("bits", range(1, 9))
def test_pack_matches_big_integer_definition(bits):
    rng = np.random.default_rng(6 + bits)
    for n in (0, 1, 5, 31, 32, 33, 64, 1000, 1027):
        code = rng.integers(0, 1 << bits, size=n, dtype=np.uint32)
        words = oracle.pack(code, bits)
        assert words.size == (n * bits + 31) // 32 == oracle.packed_words(n, bits)
        stream = 0
        for i, c in enumerate(code.tolist()):
            stream |= c << (i * bits)
        expect = [(stream >> (32 * j)) & 0xFFFFFFFF for j in range(words.size)]
        assert words.tolist() == expect                                    # includes zero pad bits
        assert np.array_equal(oracle.unpack(words, n, bits), code)


def test_pack_known_small_vector():
    # 3-bit codes 1,2,3,4,5,6,7,0,1,2,3: written out by hand
    code = np.array([1, 2, 3, 4, 5, 6, 7, 0, 1, 2, 3], dtype=np.uint32)
    w = oracle.pack(code, 3)
    # bits (LSB first): 001 010 011 100 101 110 111 000 001 010 | 11 -> word0 ; remaining bit of the last code -> word1
    word0 = 0
    for i, c in enumerate([1, 2, 3, 4, 5, 6, 7, 0, 1, 2]):
        word0 |= c << (3 * i)
    word0 |= (3 & 0b11) << 30
    assert w.tolist() == [word0 & 0xFFFFFFFF, 3 >> 2]
    assert w[1] == 0                                   # the spilled high bit of the last code (3 = 0b011) is 0
    assert w[0] == 0b11_010_001_000_111_110_101_100_011_010_001


def test_message_sizes():
    assert oracle.num_buckets(11_689_512, 2048) == 5708
    assert oracle.num_buckets(25_557_032, 2048) == 12480
    assert oracle.num_buckets(124_439_808, 4096) == 30381
    assert oracle.packed_words(65536, 2) * 4 == 16384


# ------------------------------------------------------------------ reconstruction against the definition in double
@pytest.mark.parametrize("levels,bits", [(2, 1), (3, 2), (5, 3), (16, 4)])
def test_dqsg_reconstruction_matches_double_definition(levels, bits):
    # g~ = kappa (Delta q - u),  Delta = 2/(L-1), q = k - (L-1)/2, u = delta Delta   (Algorithm 1, server)
    rng = np.random.default_rng(7)
    n, B = 8192, 256
    g = (rng.standard_normal(n) * 3).astype(np.float32)
    seed, worker, step = SEED, 5, 77
    _, scale, codes, rec = _dqsg_roundtrip(g, B, bits, levels, seed, worker, step)
    delta = oracle.dither_vector(seed, worker, step, n).astype(np.float64)
    Delta = 2.0 / (levels - 1)
    kappa = np.repeat(scale.astype(np.float64), B)
    ref = kappa * (Delta * (codes - (levels - 1) / 2) - delta * Delta)
    err = np.abs(rec - ref)
    assert (err <= 2 * np.spacing(np.abs(ref).astype(np.float32)) + 1e-45).all()
    # and the encoder's index is the nearest integer of (g/kappa + u)/Delta in double, up to fp32 rounding ties
    tt = (g.astype(np.float64) / kappa) / Delta + delta
    assert (np.abs(tt - (codes - (levels - 1) / 2)) <= 0.5 + 1e-5).all()


def test_zero_bucket_and_single_element():
    n, B = 96, 32
    g = np.zeros(n, dtype=np.float32)
    g[40] = -2.5
    _, scale, codes, rec = _dqsg_roundtrip(g, B, 2, 3)
    assert scale.tolist() == [0.0, 2.5, 0.0]
    assert (rec[:32] == 0).all() and (rec[64:] == 0).all()
    assert abs(rec[40] + 2.5) <= 1.25 + 1e-6
    assert codes[40] == 0 or codes[40] == 1


def test_bucket_independence_offsets_and_threads():
    rng = np.random.default_rng(8)
    n, B = 5 * 512 + 100, 512
    g = rng.standard_normal(n).astype(np.float32)
    p, s = oracle.dqsg_encode(g, SEED, 1, 9, B, 3, 5)
    p2, s2 = oracle.dqsg_encode(g[2 * B:4 * B], SEED, 1, 9, B, 3, 5, i0=2 * B)
    w0 = 2 * B * 3 // 32
    assert np.array_equal(p[w0:w0 + p2.size], p2) and np.array_equal(s[2:4], s2)
    p3, s3 = oracle.dqsg_encode(g, SEED, 1, 9, B, 3, 5, threads=4)
    assert np.array_equal(p, p3) and np.array_equal(s, s3)
    q, t = oracle.ndqsg_encode(g, SEED, 1, 9, B, 3, 8, 8.0)
    q2, t2 = oracle.ndqsg_encode(g[3 * B:], SEED, 1, 9, B, 3, 8, 8.0, i0=3 * B)
    w0 = 3 * B * 3 // 32
    assert np.array_equal(q[w0:], q2) and np.array_equal(t[3:], t2)


# ------------------------------------------------------------------ NDQSG
def _in_cell_problem(rng, n, B, K, M1, frac=0.9):
    """g = y + z with |z| strictly inside the always-correct region |z| < (Delta2 - Delta1)/(2 alpha)."""
    y = rng.uniform(-0.8, 0.8, n).astype(np.float32)
    bound = frac * (K - 1) / (2.0 * M1)                      # in units of kappa = 1
    z = rng.uniform(-bound, bound, n).astype(np.float32)
    g = (y + z).astype(np.float32)
    g[::B] = 1.0                                             # kappa = 1 per bucket
    y[::B] = 1.0
    return g, y


@pytest.mark.parametrize("K,M1,bits", [(3, 3.0, 2), (4, 4.0, 2), (8, 16.0, 3), (2, 2.0, 1), (5, 7.0, 3)])
def test_ndqsg_equals_dqsg_when_side_information_in_cell(K, M1, bits):
    rng = np.random.default_rng(9)
    n, B = 1 << 16, 512
    g, y = _in_cell_problem(rng, n, B, K, M1)
    seed, worker, step = SEED, 4, 21
    pk, sc, q1 = oracle.ndqsg_encode(g, seed, worker, step, B, bits, K, M1, 1.0, want_q1=True)
    m = oracle.Msg(pk, sc, seed, worker, oracle.KIND_NDQSG, B, bits, coarse_K=K, fine_M=M1, alpha=1.0)
    avg, rec, qhat = oracle.decode_aggregate([m], n, step, side_info=y, want_recon=True, want_qhat=True)
    assert np.array_equal(qhat[0], q1)                       # p = 0 inside the cell: the fine index is recovered
    # the plain DQSG with step Delta_1 = 1/M1 (L = 2 M1 + 1 levels) and the same dither
    L = int(2 * M1 + 1)
    dbits = math.ceil(math.log2(L))
    dp, ds, dk = oracle.dqsg_encode(g, seed, worker, step, B, dbits, L, want_codes=True)
    dm = oracle.Msg(dp, ds, seed, worker, oracle.KIND_DQSG, B, dbits, L)
    drec = oracle.decode_aggregate([dm], n, step)
    same_index = (dk - int(M1)) == q1
    assert same_index.mean() > 0.9999                        # only fp32 near-ties of the extra '+ s' can differ
    assert np.array_equal(rec[0][same_index], drec[same_index])          # bit-exact
    assert np.array_equal(avg, rec[0])
    # the codes on the wire are q1 mod K
    assert np.array_equal(oracle.unpack(pk, n, bits).astype(np.int64), np.mod(q1, K))


def test_ndqsg_closed_form_equals_bruteforce_nearest_coset():
    rng = np.random.default_rng(10)
    n, B, K, M1, bits = 2048, 64, 4, 4.0, 2
    y = rng.uniform(-1, 1, n).astype(np.float32)
    g = (y + rng.normal(0, 0.25, n)).astype(np.float32)     # a good share of out-of-cell cases as well
    seed, worker, step = SEED, 6, 2
    for alpha in (1.0, 0.75):
        pk, sc = oracle.ndqsg_encode(g, seed, worker, step, B, bits, K, M1, alpha)
        m = oracle.Msg(pk, sc, seed, worker, oracle.KIND_NDQSG, B, bits, coarse_K=K, fine_M=M1, alpha=alpha)
        _, _, qhat = oracle.decode_aggregate([m], n, step, side_info=y, want_recon=True, want_qhat=True)
        codes = oracle.unpack(pk, n, bits)
        delta = oracle.dither_vector(seed, worker, step, n)
        checked = 0
        for i in range(n):
            kappa = float(sc[i // B])
            a = float(np.float32(np.float32(alpha) * np.float32(M1)) / np.float32(kappa))
            q, margin = oracle.nearest_coset_bruteforce(int(codes[i]), K, a, float(delta[i]), float(y[i]), 64)
            if margin > 1e-4:
                assert q == qhat[0, i]
                checked += 1
        assert checked > 0.99 * n


@pytest.mark.parametrize("alpha", [1.0, 0.8])
def test_ndqsg_failure_bound_and_mse(alpha):
    # p <= Delta1^2/(3 Delta2^2) + 4 alpha^2 sigma_z^2/Delta2^2 ;  MSE = alpha^2 Delta1^2/12 + (1-alpha^2)^2 sigma_z^2
    rng = np.random.default_rng(11)
    n, B, K, M1, bits = 1 << 18, 1024, 4, 4.0, 2
    D1, D2 = 1 / M1, K / M1
    sigma_z = 0.08
    y = rng.uniform(-0.55, 0.55, n).astype(np.float32)
    z = rng.normal(0, sigma_z, n).astype(np.float32)
    g = (y + z).astype(np.float32)
    g[::B] = 1.0
    y[::B] = 1.0
    seed, worker, step = SEED, 8, 5
    pk, sc, q1 = oracle.ndqsg_encode(g, seed, worker, step, B, bits, K, M1, alpha, want_q1=True)
    assert (sc == 1.0).all()
    m = oracle.Msg(pk, sc, seed, worker, oracle.KIND_NDQSG, B, bits, coarse_K=K, fine_M=M1, alpha=alpha)
    _, rec, qhat = oracle.decode_aggregate([m], n, step, side_info=y, want_recon=True, want_qhat=True)
    ok = qhat[0] == q1
    keep = np.ones(n, bool)
    keep[::B] = False
    p_fail = 1.0 - ok[keep].mean()
    bound = D1 ** 2 / (3 * D2 ** 2) + 4 * alpha ** 2 * sigma_z ** 2 / D2 ** 2
    assert p_fail <= bound
    sel = keep & ok
    zz = (g.astype(np.float64) - y)[sel]
    err = (rec[0].astype(np.float64) - g)[sel]
    mse_theory = alpha ** 2 * D1 ** 2 / 12 + (1 - alpha ** 2) ** 2 * float(np.mean(zz ** 2))
    assert np.mean(err ** 2) == pytest.approx(mse_theory, rel=0.02)
    # error form of the proof: with y = g + z',  g^ = g + (1 - alpha^2) z' - alpha e,  e uniform in the fine cell
    # (zz = g - y = -z')
    e = (-err - (1 - alpha ** 2) * zz) / alpha
    assert np.abs(e).max() <= D1 / 2 + 1e-5
    assert abs(np.corrcoef(e, zz)[0, 1]) < 0.01


def test_ndqsg_out_of_cell_errors_are_multiples_of_coarse_step():
    rng = np.random.default_rng(12)
    n, B, K, M1, bits = 1 << 14, 256, 4, 2.0, 2
    y = rng.uniform(-0.5, 0.5, n).astype(np.float32)
    g = (y + rng.normal(0, 0.6, n)).astype(np.float32)
    g[::B] = 2.0
    y[::B] = 2.0
    pk, sc, q1 = oracle.ndqsg_encode(g, SEED, 1, 1, B, bits, K, M1, 1.0, want_q1=True)
    m = oracle.Msg(pk, sc, SEED, 1, oracle.KIND_NDQSG, B, bits, coarse_K=K, fine_M=M1)
    _, _, qhat = oracle.decode_aggregate([m], n, 1, side_info=y, want_recon=True, want_qhat=True)
    diff = qhat[0].astype(np.int64) - q1
    assert (diff % K == 0).all() and (diff != 0).any()


# ------------------------------------------------------------------ aggregate
def test_aggregate_is_the_mean_in_worker_order():
    rng = np.random.default_rng(13)
    n, B, W = 4096, 128, 5
    msgs = []
    for w in range(W):
        g = rng.standard_normal(n).astype(np.float32)
        p, s = oracle.dqsg_encode(g, SEED + w, w, 3, B, 3, 7)
        msgs.append(oracle.Msg(p, s, SEED + w, w, oracle.KIND_DQSG, B, 3, 7))
    avg, rec = oracle.decode_aggregate(msgs, n, 3, want_recon=True)
    for w in range(W):
        assert np.array_equal(rec[w], oracle.decode_aggregate([msgs[w]], n, 3))     # W = 1 is the reconstruction
    acc = np.zeros(n, dtype=np.float32)
    for w in range(W):
        acc = acc + rec[w]
    assert np.array_equal(avg, acc / np.float32(W))
    ref = rec.astype(np.float64).mean(axis=0)
    assert np.abs(avg - ref).max() <= 4 * np.spacing(np.float32(np.abs(rec).max()))
    perm = oracle.decode_aggregate(msgs[::-1], n, 3)
    assert np.abs(perm - avg).max() <= 4 * np.spacing(np.float32(np.abs(rec).max()))
    avg_t = oracle.decode_aggregate(msgs, n, 3, threads=3)
    assert np.array_equal(avg, avg_t)


def test_oracle_rejects_bad_arguments():
    g = np.zeros(64, dtype=np.float32)
    with pytest.raises(ValueError):
        oracle.dqsg_encode(g, 1, 0, 0, 48, 2)            # bucket not a multiple of 32
    with pytest.raises(ValueError):
        oracle.dqsg_encode(g, 1, 0, 0, 32, 9)            # bits out of range
    with pytest.raises(ValueError):
        oracle.dqsg_encode(g, 1, 0, 0, 32, 2, 5)         # 5 levels do not fit 2 bits
    with pytest.raises(ValueError):
        oracle.ndqsg_encode(g, 1, 0, 0, 32, 2, 5, 4.0)   # K > 2^bits
    with pytest.raises(ValueError):
        oracle.ndqsg_encode(g, 1, 0, 0, 32, 2, 4, 4.0, alpha=1.5)


# ------------------------------------------------------------------ half-dithered decoding (Section 2.1, Lemma 1)
def test_half_dithered_decoder_matches_stochastic_quantization_statistics():
    # the receiver does not subtract the dither: x~_h = Q(x + u) = kappa * Delta * q.  It is unbiased and its
    # error variance is (|x| - l/M)((l+1)/M - |x|): exactly M-level stochastic quantization (Lemma 1).
    n, B, M = 1 << 18, 65536, 2
    x = 0.3
    g = np.full(n, x, dtype=np.float32)
    g[::B] = 1.0
    pk, sc, codes = oracle.dqsg_encode(g, SEED, 1, 2, B, 3, 2 * M + 1, want_codes=True)
    half = oracle.decode_aggregate([oracle.Msg(pk, sc, SEED, 1, oracle.KIND_DQSG, B, 3, 2 * M + 1, dither_bits=0)], n, 2)
    assert np.array_equal(half, ((codes - M) / M).astype(np.float32))          # kappa = 1: Delta * q
    keep = np.ones(n, bool)
    keep[::B] = False
    err = half[keep].astype(np.float64) - np.float32(x)
    d = float(np.float32(x)) - 0.0                                              # l = 0, d = x
    assert abs(err.mean()) < 5 * math.sqrt(d * (1 / M - d) / keep.sum())
    assert err.var() == pytest.approx(d * (1 / M - d), rel=0.03)
    full = oracle.decode_aggregate([oracle.Msg(pk, sc, SEED, 1, oracle.KIND_DQSG, B, 3, 2 * M + 1)], n, 2)
    assert (full[keep].astype(np.float64) - np.float32(x)).var() == pytest.approx(1 / (12 * M * M), rel=0.03)
    with pytest.raises(ValueError):                                             # the nested decoder needs the dither
        oracle.decode_aggregate([oracle.Msg(pk, sc, SEED, 1, oracle.KIND_NDQSG, B, 3, coarse_K=4, fine_M=2.0,
                                            dither_bits=0)], n, 2, side_info=g)


# ------------------------------------------------------------------ index statistics (rate after entropy coding)
def test_ternary_index_distribution_and_entropy_for_uniform_input():
    # x ~ U[-1, 1], kappa = 1, M = 1: P(q = +1) = E[max(x, 0)] = 1/4 = P(q = -1), P(q = 0) = 1/2 (Appendix A),
    # so the index stream carries 1.5 bits per element, below the raw log2(3) of the raw-bits table.
    rng = np.random.default_rng(77)
    n, B = 1 << 18, 65536
    g = rng.uniform(-1, 1, n).astype(np.float32)
    g[::B] = 1.0
    pk, sc = oracle.dqsg_encode(g, SEED, 0, 1, B, 2, 3)
    hist = np.bincount(oracle.unpack(pk, n, 2), minlength=4)
    assert hist.sum() == n and hist[3] == 0
    p = hist[:3] / n
    assert np.allclose(p, [0.25, 0.5, 0.25], atol=5 * math.sqrt(0.25 / n))
    H = -(p * np.log2(p)).sum()
    assert H == pytest.approx(1.5, abs=0.01) and H < math.log2(3)
