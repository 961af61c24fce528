"""Pins for the CPU oracle: random stream and natural compression (Def. 1, Thm. 1, Sec. 2).

Nothing here calls the CUDA library.  Each check compares the oracle with something
fixed outside it: published known-answer vectors, values the paper prints, closed
forms from the proofs, or exhaustive enumeration of all 2^23 random thresholds.
"""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
ALL_R23 = np.arange(1 << 23, dtype=np.uint32)


def _golden_lines(name):
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                yield line.split()


# ------------------------------------------------------------------ Philox
def test_philox_known_answers():
    n = 0
    for tok in _golden_lines("philox4x32_10_kat.txt"):
        v = [int(t, 16) for t in tok]
        out = oracle.philox4x32_10(v[0:4], v[4:6])
        assert [int(o) for o in out] == v[6:10]
        n += 1
    assert n == 3


def _philox_inverse(out, key):
    """Undo the 10 rounds with the modular inverses of the multipliers (a different
    computation from the forward rounds)."""
    M0, M1 = 0xD2511F53, 0xCD9E8D57
    inv0, inv1 = pow(M0, -1, 1 << 32), pow(M1, -1, 1 << 32)
    keys = [((key[0] + r * 0x9E3779B9) & 0xFFFFFFFF, (key[1] + r * 0xBB67AE85) & 0xFFFFFFFF)
            for r in range(10)]
    n0, n1, n2, n3 = [int(v) for v in out]
    for r in reversed(range(10)):
        k0, k1 = keys[r]
        c2 = (n1 * inv1) & 0xFFFFFFFF
        c0 = (n3 * inv0) & 0xFFFFFFFF
        hi1 = (M1 * c2) >> 32
        hi0 = (M0 * c0) >> 32
        c1 = n0 ^ hi1 ^ k0
        c3 = n2 ^ hi0 ^ k1
        n0, n1, n2, n3 = c0, c1, c2, c3
    return [n0, n1, n2, n3]


def test_philox_is_the_invertible_permutation():
    rng = np.random.default_rng(7)
    for _ in range(50):
        ctr = rng.integers(0, 1 << 32, 4, dtype=np.uint64).astype(np.uint32)
        key = rng.integers(0, 1 << 32, 2, dtype=np.uint64).astype(np.uint32)
        out = oracle.philox4x32_10(ctr, key)
        assert _philox_inverse(out, [int(k) for k in key]) == [int(c) for c in ctr]


def test_stream_mapping_counter_key_word():
    # element j uses word j mod 4 of the block with counter (lo(j/4), hi(j/4), worker, domain)
    seed, worker, domain = 0x0123456789ABCDEF, 5, 2
    j0 = (1 << 34) + 8          # exercises the high counter word
    words = oracle.stream_words(seed, worker, domain, j0, 8)
    for blk in range(2):
        q = j0 // 4 + blk
        ref = oracle.philox4x32_10([q & 0xFFFFFFFF, q >> 32, worker, domain],
                                   [seed & 0xFFFFFFFF, seed >> 32])
        assert list(words[4 * blk:4 * blk + 4]) == list(ref)
    # different worker / domain / seed give different streams
    base = oracle.stream_words(1, 0, 0, 0, 64)
    assert not np.array_equal(base, oracle.stream_words(1, 1, 0, 0, 64))
    assert not np.array_equal(base, oracle.stream_words(1, 0, 1, 0, 64))
    assert not np.array_equal(base, oracle.stream_words(2, 0, 0, 0, 64))


def test_stream_low_23_bits_are_uniform():
    r = oracle.stream_words(0, 0, 0, 0, 1 << 20) & 0x7FFFFF
    hist = np.bincount(r >> 15, minlength=256).astype(np.float64)   # 256 cells
    expected = r.size / 256
    chi2 = ((hist - expected) ** 2 / expected).sum()
    assert chi2 < 255 + 6 * np.sqrt(2 * 255)
    assert abs(r.mean() / (1 << 23) - 0.5) < 4 * np.sqrt(1 / 12 / r.size)


# ------------------------------------------------------- natural compression
def test_cnat_paper_worked_examples():
    seen = 0
    for tok in _golden_lines("paper_worked_examples.txt"):
        if tok[0] != "cnat":
            continue
        t, lower, upper, p_up = (float(v) for v in tok[1:5])
        vals = oracle.cnat_values(np.full(ALL_R23.size, t, np.float32), ALL_R23)
        n_up = int((vals == upper).sum()) if upper != lower else 0
        assert set(np.unique(vals)) <= {lower, upper}
        assert n_up == int(round(p_up * (1 << 23)))          # exact probability
        seen += 1
    assert seen == 5


@pytest.mark.parametrize("t", [2.5, -2.75, 0.75, 1e-3, -3.1415927e-5, 1.9999999, 1.0000001,
                               6.02e23, -1.17549435e-38])
def test_cnat_unbiased_and_second_moment_by_enumeration(t):
    t32 = np.float32(t)
    vals = oracle.cnat_values(np.full(ALL_R23.size, t32, np.float32), ALL_R23)
    # E C(t) = t exactly (Def. 1's probabilities; binary32 mantissa has 23 bits)
    assert vals.sum() / ALL_R23.size == float(t32)
    # proof of Thm. 1: E C(t)^2 = 2^a (3|t| - 2^(a+1)),  a = floor(log2 |t|)
    a = np.floor(np.log2(abs(float(t32))))
    closed = 2.0 ** a * (3 * abs(float(t32)) - 2.0 ** (a + 1))
    second = (vals * vals).sum() / ALL_R23.size
    assert second == pytest.approx(closed, rel=1e-12)
    assert second <= 9.0 / 8.0 * float(t32) ** 2 * (1 + 1e-12)


def test_cnat_second_moment_ratio_peaks_at_four_thirds():
    # Thm. 1: sup over 1 < theta < 2 of (3 theta - 2) / theta^2 = 9/8 at theta = 4/3.
    thetas = np.float32([1.25, 4.0 / 3.0, 1.4, 1.75])
    ratios = []
    for th in thetas:
        v = oracle.cnat_values(np.full(ALL_R23.size, th * 8.0, np.float32), ALL_R23)
        ratios.append((v * v).mean() / (float(th) * 8.0) ** 2)
    assert int(np.argmax(ratios)) == 1
    assert ratios[1] == pytest.approx(9.0 / 8.0, abs=1e-6)
    assert all(r <= 9.0 / 8.0 + 1e-12 for r in ratios)


def test_cnat_monte_carlo_with_the_philox_stream():
    # unbiasedness within 4 sigma over 10^6 stream draws, for several inputs
    n = 1_000_000
    r23 = oracle.stream_words(0, 3, 0, 0, n) & 0x7FFFFF
    for t in [2.5, -0.3, 1.7e-4, -7.7e5]:
        t32 = float(np.float32(t))
        vals = oracle.cnat_values(np.full(n, t32, np.float32), r23)
        a = np.floor(np.log2(abs(t32)))
        lo, hi = 2.0 ** a, 2.0 ** (a + 1)
        sigma = np.sqrt((hi - abs(t32)) * (abs(t32) - lo))
        assert abs(vals.mean() - t32) <= 4 * sigma / np.sqrt(n)
        assert (vals * vals).mean() <= 9 / 8 * t32 ** 2 * 1.01


def test_cnat_brute_force_outcome_probabilities_tiny_mantissas():
    # inputs 2^k (1 + i/8): exactly i/8 of the thresholds round up
    for k in (-20, 0, 7):
        for i in range(8):
            t = np.float32(2.0 ** k * (1 + i / 8))
            vals = oracle.cnat_values(np.full(ALL_R23.size, -t, np.float32), ALL_R23)
            assert int((vals == -2.0 ** (k + 1)).sum()) == i * (1 << 20)
            assert int((vals == -2.0 ** k).sum()) == (8 - i) * (1 << 20)


def test_cnat_threshold_rule_uses_low_23_bits_strictly_below():
    # m = 5 * 2^-23: thresholds 0..4 round up, 5.. do not; bits above 23 are ignored
    t = np.float32(1.0) + np.float32(5 * 2.0 ** -23)
    r = np.uint32([0, 4, 5, 6, (1 << 23) + 4, (0xFF << 23) | 5])
    vals = oracle.cnat_values(np.full(r.size, t, np.float32), r)
    assert list(vals) == [2.0, 2.0, 1.0, 1.0, 2.0, 1.0]


def test_cnat_edge_policy_table():
    f32 = np.float32
    tiny = f32(2.0 ** -126)
    sub = f32(3 * 2.0 ** -149)                       # subnormal, field M = 3
    big = np.frombuffer(np.uint32(0x7F7FFFFF).tobytes(), f32)[0]   # largest finite
    cases = [
        # (t, r23, expected value)
        (f32(0.0), 0, 0.0), (f32(-0.0), 0, -0.0),
        (sub, 2, float(tiny)), (sub, 3, 0.0), (-sub, 0, -float(tiny)), (-sub, 5, -0.0),
        (tiny, 0, float(tiny)),                       # 2^-126 is a power of two
        (big, 0, 2.0 ** 127), (-big, 0, -(2.0 ** 127)),           # never up at the top
        (f32(np.inf), 0, np.inf), (f32(-np.inf), 0, -np.inf),
        (f32(np.nan), 0, np.inf),
    ]
    t = np.array([c[0] for c in cases], f32)
    r = np.array([c[1] for c in cases], np.uint32)
    vals = oracle.cnat_values(t, r)
    for v, (_, _, want) in zip(vals, cases):
        assert v == want and np.signbit(v) == np.signbit(want)
    # the same through the 9-bit code
    e, s = oracle.cnat_codes(t, r)
    assert list(e) == [0, 0, 1, 0, 1, 0, 1, 254, 254, 255, 255, 255]
    assert list(s[:11]) == [0, 1, 0, 0, 1, 1, 0, 0, 1, 0, 1]
    neg_nan = np.frombuffer(np.uint32(0xFFC00001).tobytes(), f32)
    e2, s2 = oracle.cnat_codes(neg_nan, np.uint32([7]))
    assert (int(e2[0]), int(s2[0])) == (255, 1)


def test_subnormal_policy_is_unbiased_but_breaks_nine_eighths():
    sub = np.float32(2.0 ** -140)
    vals = oracle.cnat_values(np.full(ALL_R23.size, sub, np.float32), ALL_R23)
    assert vals.sum() / ALL_R23.size == float(sub)
    assert (vals * vals).mean() > 9 / 8 * float(sub) ** 2      # same mechanism as Thm. 2


def test_code_round_trip_for_every_representable_output():
    # every +-2^k (biased exponent 1..254), +-0 and +-inf survives encode -> decode
    e_all = np.arange(256, dtype=np.uint8)
    for sbit in (0, 1):
        dec = oracle.cnat_decode(e_all, np.full(256, sbit, np.uint8))
        want = np.ldexp(1.0, e_all.astype(np.int64) - 127)
        want[0], want[255] = 0.0, np.inf
        want = (-want if sbit else want).astype(np.float32)
        assert np.array_equal(dec.view(np.uint32), want.view(np.uint32))
        e2, s2 = oracle.cnat_codes(dec, np.zeros(256, np.uint32))
        assert np.array_equal(e2, e_all) and np.all(s2 == sbit)


def test_cnat_agrees_with_ieee_field_rule_on_random_bit_patterns():
    # Sec. 2: keep sign and exponent, drop the mantissa, add one to the exponent with
    # probability m.  Checked on random bit patterns of normal numbers with numpy.
    rng = np.random.default_rng(11)
    u = rng.integers(0, 1 << 32, 200_000, dtype=np.uint64).astype(np.uint32)
    ex = (u >> 23) & 0xFF
    u = u[(ex >= 1) & (ex <= 253)]
    r = rng.integers(0, 1 << 23, u.size, dtype=np.uint64).astype(np.uint32)
    t = u.view(np.float32)
    e, s = oracle.cnat_codes(t, r)
    want_e = ((u >> 23) & 0xFF) + (r < (u & 0x7FFFFF))
    assert np.array_equal(e.astype(np.uint32), want_e)
    assert np.array_equal(s.astype(np.uint32), u >> 31)


def test_nc_compress_packed_layout_and_tail():
    rng = np.random.default_rng(3)
    d = 1000                                   # 31 full sign words + 8 bits
    x = (rng.standard_normal(d) * 1e-3).astype(np.float32)
    x[5] = 0.0
    x[6] = -0.0
    e, sg = oracle.nc_compress(x, seed=9, worker=2)
    r23 = oracle.stream_words(9, 2, 0, 0, d) & 0x7FFFFF
    e_ref, s_ref = oracle.cnat_codes(x, r23)
    assert np.array_equal(e, e_ref)
    bits = (sg[np.arange(d) // 32] >> (np.arange(d) % 32)) & 1
    assert np.array_equal(bits.astype(np.uint8), s_ref)
    assert sg[-1] >> 8 == 0                     # padding bits are zero
    # a slice starting at element j0 reproduces the same codes
    e2, sg2 = oracle.nc_compress(x[64:], seed=9, worker=2, j0=64)
    assert np.array_equal(e2, e[64:]) and np.array_equal(sg2, sg[2:])
    # the thread count does not change the output (counter-based stream)
    full = oracle.max_threads()
    oracle.set_threads(1)
    e3, sg3 = oracle.nc_compress(x, seed=9, worker=2)
    oracle.set_threads(full)
    assert np.array_equal(e3, e) and np.array_equal(sg3, sg)
