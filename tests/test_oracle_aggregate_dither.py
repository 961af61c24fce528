"""Pins for the CPU oracle: aggregation (Algorithm 1), norms and natural dithering
(Def. 3, Thm. 4, the identity in the proof of Thm. 5) and the sparsifier composition.

Nothing here calls the CUDA library.
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


def _pack_signs(bits):
    d = bits.size
    words = np.zeros((d + 31) // 32, np.uint32)
    for j in range(d):
        words[j // 32] |= np.uint32(int(bits[j]) << (j % 32))
    return words


def _codes_of(values):
    """9-bit codes of exact powers of two / zeros / infinities (threshold irrelevant)."""
    v = np.asarray(values, np.float32)
    e, s = oracle.cnat_codes(v, np.zeros(v.size, np.uint32))
    return e, _pack_signs(s)


# ------------------------------------------------------------- aggregation
def test_aggregate_hand_cases_fix_order_and_start_value():
    cols = [
        [2.0, 2.0, -4.0, 2.0 ** -30],      # (((0+2)+2)-4)+2^-30 = 2^-30; other orders lose it
        [2.0 ** -30, 2.0, 2.0, -4.0],      # same terms, other order: 2^-30 is absorbed -> 0
        [-0.0, -0.0, -0.0, -0.0],          # starts from +0: result +0
        [np.inf, 1.0, -np.inf, 1.0],       # inf - inf = NaN, stays NaN
        [2.0 ** 127, 2.0 ** 127, -2.0 ** 127, 0.0],   # overflow to inf is not undone
        [2.0 ** -126, -2.0 ** -126, 2.0 ** -126, 2.0 ** -126],
    ]
    n, d = 4, len(cols)
    exps, signs = [], []
    for i in range(n):
        e, s = _codes_of([c[i] for c in cols])
        exps.append(e)
        signs.append(s)
    out = oracle.nc_aggregate(exps, signs, d)
    assert out[0] == np.float32(2.0 ** -30)
    assert out[1] == 0.0
    assert out[2] == 0.0 and not np.signbit(out[2])
    assert np.isnan(out[3])
    assert np.isinf(out[4]) and out[4] > 0
    assert out[5] == np.float32(2.0 ** -125)


def test_aggregate_equals_numpy_sequential_float32_sum_and_decode_accumulate():
    rng = np.random.default_rng(5)
    n, d = 7, 4099
    exps = [rng.integers(90, 140, d).astype(np.uint8) for _ in range(n)]
    for e in exps:
        e[rng.random(d) < 0.05] = 0
    signs = [rng.integers(0, 1 << 32, (d + 31) // 32, dtype=np.uint64).astype(np.uint32)
             for _ in range(n)]
    out = oracle.nc_aggregate(exps, signs, d)
    acc = np.zeros(d, np.float32)
    acc2 = np.zeros(d, np.float32)
    j = np.arange(d)
    for e, s in zip(exps, signs):
        bits = ((s[j // 32] >> (j % 32)) & 1).astype(np.uint8)
        v = oracle.cnat_decode(e, bits)
        acc = (acc + v).astype(np.float32)          # numpy binary32 add, worker order
        oracle.nc_decode_accumulate(e, s, acc2)
    assert np.array_equal(out.view(np.uint32), acc.view(np.uint32))
    assert np.array_equal(out.view(np.uint32), acc2.view(np.uint32))
    # n = 1 is a plain decode
    one = oracle.nc_aggregate(exps[:1], signs[:1], d)
    bits0 = ((signs[0][j // 32] >> (j % 32)) & 1).astype(np.uint8)
    assert np.array_equal(one.view(np.uint32),
                          (np.float32(0) + oracle.cnat_decode(exps[0], bits0)).view(np.uint32))


def test_sum_fp32_equals_numpy_sequential_sum():
    rng = np.random.default_rng(6)
    xs = [(rng.standard_normal(1001) * 10.0 ** rng.integers(-6, 3)).astype(np.float32)
          for _ in range(5)]
    acc = np.zeros(1001, np.float32)
    for x in xs:
        acc = (acc + x).astype(np.float32)
    assert np.array_equal(oracle.sum_fp32(xs).view(np.uint32), acc.view(np.uint32))


# -------------------------------------------------------------------- norms
def test_norm_closed_forms():
    d = 1000
    const = np.full(d, -0.5, np.float32)
    onehot = np.zeros(d, np.float32)
    onehot[123] = -3.25e-7
    ramp = np.arange(1, d + 1, dtype=np.float32)
    off = [0, d]
    assert oracle.norms(const, off, 1)[0] == np.float32(0.5 * d)
    assert oracle.norms(const, off, 2)[0] == np.float32(0.5 * np.sqrt(d))
    assert oracle.norms(const, off, oracle.P_INF)[0] == np.float32(0.5)
    for p in (1, 2, oracle.P_INF):                 # a single non-zero: every norm is |x|
        assert oracle.norms(onehot, off, p)[0] == np.float32(3.25e-7)
    assert oracle.norms(ramp, off, 1)[0] == np.float32(d * (d + 1) / 2)
    assert oracle.norms(ramp, off, 2)[0] == np.float32(np.sqrt(d * (d + 1) * (2 * d + 1) / 6))
    assert oracle.norms(ramp, off, oracle.P_INF)[0] == np.float32(d)
    # per-bucket, including an empty bucket; against numpy in float64
    rng = np.random.default_rng(0)
    x = rng.standard_normal(5000).astype(np.float32)
    off = [0, 7, 7, 100, 4096, 5000]
    for p, f in ((1, lambda v: np.abs(v).sum()), (2, lambda v: np.sqrt((v * v).sum())),
                 (oracle.P_INF, lambda v: np.abs(v).max() if v.size else 0.0)):
        got = oracle.norms(x, off, p)
        for b in range(5):
            seg = x[off[b]:off[b + 1]].astype(np.float64)
            assert got[b] == pytest.approx(f(seg), rel=2e-7)
    assert oracle.norms(x, off, 2)[1] == 0.0
    xn = x.copy()
    xn[50] = np.nan
    assert np.isnan(oracle.norms(xn, off, oracle.P_INF)[2])


# ------------------------------------------------------- natural dithering
def test_dnat_paper_worked_examples():
    seen = 0
    for tok in _golden_lines("paper_worked_examples.txt"):
        if tok[0] == "dnat":
            y, s, lower, upper, p_up = float(tok[1]), int(tok[2]), *map(float, tok[3:6])
            codes = oracle.nd_level_codes(np.full(ALL_R23.size, y), ALL_R23, s)
            vals = np.where(codes == 0, 0.0, np.ldexp(1.0, codes - s))
            assert set(np.unique(vals)) == {lower, upper}
            assert int((vals == upper).sum()) == int(p_up * (1 << 23))
            seen += 1
        elif tok[0] == "levels":
            s = int(tok[1])
            want = [float(v) for v in tok[2:]]
            assert len(want) == s + 1
            ys = np.linspace(0, 1, 4097)
            reach = set()
            for r in (0, (1 << 23) - 1):
                c = oracle.nd_level_codes(ys, np.full(ys.size, r, np.uint32), s)
                reach |= set(np.where(c == 0, 0.0, np.ldexp(1.0, c - s)))
            assert sorted(reach) == want
            seen += 1
    assert seen == 3


@pytest.mark.parametrize("s", [1, 3, 8])
def test_dnat_rounding_is_unbiased_and_meets_the_second_moment_bound(s):
    # Def. 3: E xi(y) = y.  Proof of Thm. 4: E xi^2 <= 9/8 y^2 for y >= 2^(1-s), and
    # E xi^2 = y 2^(1-s) below.  The draw has resolution 2^-23 (floor), hence the slack.
    bottom = 2.0 ** (1 - s)
    for y in [0.0, bottom / 7, bottom * 0.999, bottom, 0.3, 0.5, 2 / 3, 0.9999, 1.0]:
        if y > 1:
            continue
        codes = oracle.nd_level_codes(np.full(ALL_R23.size, y), ALL_R23, s)
        xi = np.where(codes == 0, 0.0, np.ldexp(1.0, codes - s))
        width = bottom if y < bottom else 2.0 ** np.floor(np.log2(y))
        assert abs(xi.mean() - y) <= width * 2.0 ** -23
        second = (xi * xi).mean()
        if y < bottom:
            assert second == pytest.approx(y * bottom, abs=bottom * bottom * 2.0 ** -23)
        else:
            assert second <= 9 / 8 * y * y * (1 + 1e-6)


def test_dnat_bracket_ties_and_clamp():
    s = 4
    for k in range(s):                            # y exactly a level: both brackets agree
        y = 2.0 ** -k
        for r in (0, 12345, (1 << 23) - 1):
            assert oracle.nd_level_codes([y], [r], s)[0] == s - k
    assert oracle.nd_level_codes([1.0000001], [0], s)[0] == s      # rounding excess clamps
    assert oracle.nd_level_codes([0.0], [0], s)[0] == 0


def test_dnat_equals_cnat_of_standard_dithering_in_distribution():
    # Identity in the proof of Thm. 5: D_nat(x) =_D ||x|| sign(x) C_nat(xi_sta(x)) with
    # standard levels k / 2^(s-1).  Outcome probabilities of both sides, per level.
    s = 4
    u = 2 ** (s - 1)
    for y in [0.03, 0.1, 0.125, 0.2, 0.33, 0.6, 0.77, 0.95]:
        codes = oracle.nd_level_codes(np.full(ALL_R23.size, y), ALL_R23, s)
        p_nat = np.bincount(codes, minlength=s + 1) / ALL_R23.size
        # right-hand side: standard dithering (closed form), then C_nat (oracle, enumerated)
        k = int(np.floor(y * u))
        p_hi = y * u - k
        p_rhs = np.zeros(s + 1)
        for lvl, pr in ((k, 1 - p_hi), (k + 1, p_hi)):
            if pr == 0:
                continue
            if lvl == 0:
                p_rhs[0] += pr
                continue
            v = oracle.cnat_values(np.full(ALL_R23.size, lvl / u, np.float32), ALL_R23)
            c = (np.log2(v) + s).astype(np.int64)          # value 2^(c-s)
            p_rhs += pr * np.bincount(c, minlength=s + 1) / ALL_R23.size
        assert np.allclose(p_nat, p_rhs, atol=2.0 ** -22)


def test_dnat_empirical_variance_within_theorem_4():
    # Appendix A.2 set-up: x ~ N(0, I), d = 10^5, omega(x) = ||C(x) - x||^2 / ||x||^2.
    d = 100_000
    rng = np.random.default_rng(42)
    x = rng.standard_normal(d).astype(np.float32)
    off = [0, d]
    x2 = float((x.astype(np.float64) ** 2).sum())
    for p in (1, 2, oracle.P_INF):
        r = 1 if p == 1 else 2
        for s in (4, 8, 12):
            nrm, level, sign = oracle.nd_compress(x, off, p, s, seed=1, worker=0)
            dec = np.zeros(d, np.float32)
            oracle.nd_decode_accumulate(nrm, level, sign, off, s, dec)
            omega = float(((dec.astype(np.float64) - x) ** 2).sum()) / x2
            a = d ** (1.0 / r) * 2.0 ** (1 - s)
            bound = 1 / 8 + a * min(1.0, a)
            assert omega <= bound * 1.05
            # E omega is the variance: it cannot be far below the C_nat part for large s
            if s == 12 and p != 1:
                assert omega > 0.05


def test_dnat_with_power_of_two_norm_reduces_to_cnat():
    # D_nat is C_nat on the normalised entries with the bottom interval not subdivided;
    # with ||x||_inf = 2^k and every |y| >= 2^(1-s) the two coincide draw for draw when
    # they read the same random stream.
    rng = np.random.default_rng(8)
    d, s = 4096, 12
    x = (rng.uniform(2.0 ** -9, 1.0, d) * rng.choice([-1, 1], d)).astype(np.float32) * 4.0
    x[17] = -4.0                                   # the norm: 2^2
    off = [0, d]
    nrm, level, sign = oracle.nd_compress(x, off, oracle.P_INF, s, seed=77, worker=3, domain=0)
    assert nrm[0] == 4.0
    dec = np.zeros(d, np.float32)
    oracle.nd_decode_accumulate(nrm, level, sign, off, s, dec)
    e, sg = oracle.nc_compress(x, seed=77, worker=3)
    ref = np.zeros(d, np.float32)
    oracle.nc_decode_accumulate(e, sg, ref)
    assert np.array_equal(dec.view(np.uint32), ref.view(np.uint32))
    assert np.array_equal(sign, sg)


def test_dnat_given_norm_mode_matches_definition_mode_closely():
    rng = np.random.default_rng(9)
    d = 50_000
    x = (rng.standard_normal(d) * 3e-4).astype(np.float32)
    off = [0, 10, 11, 5000, d]
    for p in (1, 2, oracle.P_INF):
        n0, l0, s0 = oracle.nd_compress(x, off, p, 8, seed=4, worker=1)
        n1, l1, s1 = oracle.nd_compress(x, off, p, 8, seed=4, worker=1, given_norms=n0)
        assert np.array_equal(s0, s1) and np.array_equal(n0, n1)
        c0 = np.stack([l0 & 0xF, l0 >> 4], 1).ravel()[:d].astype(np.int64)
        c1 = np.stack([l1 & 0xF, l1 >> 4], 1).ravel()[:d].astype(np.int64)
        diff = c0 != c1
        assert diff.mean() <= 1e-5 * 3 + 3 / d      # reciprocal-multiply vs true division
        assert np.all(np.abs(c0 - c1)[diff] == 1)


def test_dnat_degenerate_norms_give_zero_codes():
    x = np.float32([1.0, -2.0, 3.0, 0.0, 0.0, np.nan, -1.0, np.inf, 1.0, 2.0])
    off = [0, 3, 5, 7, 10]
    nrm, level, sign = oracle.nd_compress(x, off, 2, 4, seed=0, worker=0)
    c = np.stack([level & 0xF, level >> 4], 1).ravel()[:10]
    assert nrm[1] == 0.0 and np.all(c[3:5] == 0)           # x = 0 -> D(x) = 0 (Def. 3)
    assert np.isnan(nrm[2]) and np.all(c[5:7] == 0)        # NaN norm: no ratio to round
    assert np.isinf(nrm[3]) and np.all(c[7:10] == 0)       # infinite norm: the same
    assert np.any(c[0:3] > 0)
    dec = np.zeros(10, np.float32)
    oracle.nd_decode_accumulate(nrm, level, sign, off, 4, dec)
    # level code 0 stands for the value 0 whatever the norm: the compressed bucket adds zeros,
    # and its stored norm is what tells the receiver that the bucket was not finite
    assert np.all(dec[3:] == 0) and not np.any(np.isnan(dec))
    assert (sign[0] >> 6) & 1 == 1 and (sign[0] >> 5) & 1 == 0   # sign plane keeps sign(x)


def test_dnat_decode_under_a_norm_that_is_not_finite():
    """Def. 3: the decoded entry is norm * sign * 2^(c-s) for c > 0 and 0 for c = 0.  With an
    infinite norm every non-zero level therefore decodes to an infinity of the entry's sign, with
    a NaN norm to NaN; level 0 stays a zero.  Expected values written out by hand."""
    s = 3
    codes = np.uint8([0, 1, 2, 3, 0, 1, 2, 3])
    level = (codes[0::2] | (codes[1::2] << 4)).astype(np.uint8)
    sign = np.uint32([0b10100110])                # entries 1, 2, 5, 7 negative
    inf = np.float32(np.inf)
    acc = np.zeros(8, np.float32)
    oracle.nd_decode_accumulate(np.float32([np.inf]), level, sign, [0, 8], s, acc)
    want = np.float32([0.0, -inf, -inf, inf, 0.0, -inf, inf, -inf])
    assert np.array_equal(acc, want)
    acc = np.full(8, 5.0, np.float32)
    oracle.nd_decode_accumulate(np.float32([np.nan]), level, sign, [0, 8], s, acc)
    assert np.array_equal(np.isnan(acc), codes > 0)
    assert np.all(acc[codes == 0] == 5.0)
    # two workers, one with an infinite norm: the column sums show it (inf, or inf - inf = NaN)
    out = oracle.nd_aggregate([np.float32([np.inf]), np.float32([2.0])], [level, level],
                              [sign, sign], [0, 8], s, 8)
    assert np.array_equal(out, np.float32([0.0, -inf, -inf, inf, 0.0, -inf, inf, -inf]))
    out = oracle.nd_aggregate([np.float32([np.inf]), np.float32([np.inf])], [level, level],
                              [sign, ~sign], [0, 8], s, 8)
    assert np.array_equal(np.isnan(out), codes > 0) and np.all(out[codes == 0] == 0)
    # the sparse decoders follow the same rule
    idx = np.uint32([1, 4, 6])
    sp = np.uint8([0x0 | (0xB << 4), 0x2])        # codes (sign<<3 | level): 0, 8|3, 2
    acc = np.zeros(8, np.float32)
    oracle.sparse_decode_accumulate(idx, sp, 3, np.float32(np.inf), 4, acc)
    assert np.array_equal(acc, np.float32([0, 0, 0, 0, -inf, 0, inf, 0]))


def test_dnat_ratios_outside_the_unit_interval_take_the_top_level():
    """xi(y) is defined for y in [0, 1] (Def. 3).  With norms given by the caller a ratio can
    exceed 1 or be NaN (a NaN entry against a finite norm); both are read as the top level s,
    whatever the draw.  Values written out by hand."""
    r = np.uint32([0, 1, (1 << 23) - 1, 12345])
    for s in (1, 4, 8, 15):
        for y in (1.0, 1.5, 1e30, np.inf, np.nan):
            assert np.array_equal(oracle.nd_level_codes(np.full(4, y), r, s), np.full(4, s))
    x = np.float32([0.5, -3.0, np.nan, 0.25, 8.0, -0.125, 0.0, 1.0])
    nrm, level, sign = oracle.nd_compress(x, [0, 8], 2, 3, seed=1, worker=0,
                                          given_norms=np.float32([1.0]))
    c = np.stack([level & 0xF, level >> 4], 1).ravel()[:8]
    assert c[1] == 3 and c[2] == 3 and c[4] == 3 and c[7] == 3 and c[6] == 0
    assert c[0] in (2, 3) and c[3] in (1, 2) and c[5] in (0, 1)
    assert sign[0] == 0b00100010 | (int(np.signbit(x[2])) << 2)


def test_dnat_bucket_with_a_subnormal_norm_is_an_ordinary_bucket():
    """y = |x| / norm does not change when a bucket is multiplied by a power of two (Def. 3), so
    neither do the level codes: a bucket of tiny entries, subnormal norm included, must get the
    codes of the same bucket scaled up by 2^100, in both arithmetic modes, and stays unbiased."""
    rng = np.random.default_rng(11)
    big = (rng.standard_normal(4000) * 0.3).astype(np.float32)
    big = np.ldexp(np.round(np.ldexp(big, 20)), -20).astype(np.float32)   # 21 significant bits
    tiny = np.ldexp(big, -128).astype(np.float32)                        # exact: multiples of 2^-148
    assert np.array_equal(np.ldexp(tiny.astype(np.float64), 128), big.astype(np.float64))
    off = [0, 1000, 4000]
    for p in (1, 2, oracle.P_INF):
        nb, lb, sb = oracle.nd_compress(big, off, p, 8, seed=3, worker=2)
        if p == oracle.P_INF:
            nt, lt, st = oracle.nd_compress(tiny, off, p, 8, seed=3, worker=2)
            assert np.all(nt < 2.0 ** -126) and np.all(nt > 0)
            assert np.array_equal(np.ldexp(nt.astype(np.float64), 128), nb.astype(np.float64))
            assert np.array_equal(lt, lb) and np.array_equal(st, sb)
        # given-norm arithmetic (binary32 reciprocal and multiply), norms scaled exactly
        g_big = oracle.nd_compress(big, off, p, 8, seed=3, worker=2, given_norms=nb)
        g_norm = np.ldexp(nb.astype(np.float64), -128).astype(np.float32)
        if np.array_equal(np.ldexp(g_norm.astype(np.float64), 128), nb.astype(np.float64)):
            g_tiny = oracle.nd_compress(tiny, off, p, 8, seed=3, worker=2, given_norms=g_norm)
            assert np.array_equal(g_tiny[1], g_big[1]) and np.array_equal(g_tiny[2], g_big[2])
    # unbiased: the mean decoded value over many seeds approaches x (max-norm, s = 4)
    x = np.ldexp(np.float32([1.0, -0.75, 0.3125, 0.046875]), -140).astype(np.float32)
    tot = np.zeros(4, np.float64)
    reps = 4000
    for seed in range(reps):
        nrm, lv, sg = oracle.nd_compress(x, [0, 4], oracle.P_INF, 4, seed=seed, worker=0)
        acc = np.zeros(4, np.float32)
        oracle.nd_decode_accumulate(nrm, lv, sg, [0, 4], 4, acc)
        tot += np.ldexp(acc.astype(np.float64), 140)
    mean = tot / reps
    want = np.float64([1.0, -0.75, 0.3125, 0.046875])
    # standard error of one entry is at most (gap between its levels) / 2 / sqrt(reps)
    assert np.all(np.abs(mean - want) <= 4 * 0.25 / np.sqrt(reps))
    assert mean[0] == 1.0


def test_dnat_decode_is_norm_times_power_of_two_in_binary32():
    s = 8
    nrm = np.float32([3.0e-3, 2.0 ** -120])
    off = [0, 9, 18]
    codes = np.array(list(range(9)) * 2, np.uint8)
    level = (codes[0::2] | (codes[1::2] << 4)).astype(np.uint8)
    sign = np.uint32([0b101010101010101010])
    acc = np.zeros(18, np.float32)
    oracle.nd_decode_accumulate(nrm, level, sign, off, s, acc)
    j = np.arange(18)
    want = np.where(codes == 0, np.float32(0),
                    (nrm[j // 9].astype(np.float64) * np.ldexp(1.0, codes.astype(int) - s))
                    .astype(np.float32))     # exact scaling, one rounding (subnormal results)
    want = np.where((j % 2) == 1, -want, want).astype(np.float32)
    assert np.array_equal(acc.view(np.uint32), (np.float32(0) + want).view(np.uint32))
    # n-way aggregate equals repeated decode-accumulate in worker order
    out = oracle.nd_aggregate([nrm, nrm * 3], [level, level], [sign, ~sign], off, s, 18)
    acc2 = np.zeros(18, np.float32)
    oracle.nd_decode_accumulate(nrm, level, sign, off, s, acc2)
    oracle.nd_decode_accumulate(nrm * 3, level, ~sign, off, s, acc2)
    assert np.array_equal(out.view(np.uint32), acc2.view(np.uint32))


# ------------------------------------------------- sparsifier composition
def _unpack4(codes, count):
    return np.stack([codes & 0xF, codes >> 4], 1).ravel()[:count]


def test_sparse_keep_everything_is_dense_dithering():
    # S^q with q = d is the identity, so the composition is plain D_nat (given-norm arithmetic)
    rng = np.random.default_rng(12)
    d, s = 3001, 4
    x = rng.standard_normal(d).astype(np.float32)
    for p in (oracle.P_INF, 2):
        idx, codes, count, nrm = oracle.sparse_compress(x, 1 << 32, 1.0, p, s, seed=5, worker=2)
        assert count == d and np.array_equal(idx, np.arange(d))
        assert nrm == oracle.norms(x, [0, d], p)[0]
        n1, l1, s1 = oracle.nd_compress(x, [0, d], p, s, seed=5, worker=2, given_norms=[nrm])
        c = _unpack4(codes, d)
        assert np.array_equal(c & 7, _unpack4(l1, d))
        j = np.arange(d)
        assert np.array_equal(c >> 3, (s1[j // 32] >> (j % 32)) & 1)


def test_sparse_selection_scaling_and_scatter():
    rng = np.random.default_rng(13)
    d, s = 200_000, 4
    x = rng.standard_normal(d).astype(np.float32)
    thr, scale = 42_949_673, 100.0
    idx, codes, count, nrm = oracle.sparse_compress(x, thr, scale, oracle.P_INF, s, seed=0,
                                                    worker=6)
    # selection is the domain-2 stream word compared with the threshold
    keep = oracle.stream_words(0, 6, 2, 0, d) < thr
    assert np.array_equal(idx, np.nonzero(keep)[0])
    assert count == int(keep.sum())
    assert abs(count - 0.01 * d) <= 5 * np.sqrt(d * 0.01 * 0.99)
    assert np.all(np.diff(idx.astype(np.int64)) > 0)
    # the dense vector S(x) put through the dense dithering path gives the same entries
    dense = np.where(keep, np.float32(scale) * x, np.float32(0)).astype(np.float32)
    assert nrm == np.abs(dense).max()
    n1, l1, s1 = oracle.nd_compress(dense, [0, d], oracle.P_INF, s, seed=0, worker=6,
                                    given_norms=[nrm])
    c = _unpack4(codes, count)
    assert np.array_equal(c & 7, _unpack4(l1, d)[idx])
    assert np.array_equal(c >> 3, ((s1[idx // 32] >> (idx % 32)) & 1))
    acc = np.zeros(d, np.float32)
    oracle.sparse_decode_accumulate(idx, codes, count, nrm, s, acc)
    ref = np.zeros(d, np.float32)
    oracle.nd_decode_accumulate(n1, l1, s1, [0, d], s, ref)
    assert np.array_equal(acc[idx].view(np.uint32), ref[idx].view(np.uint32))
    assert np.all(acc[~keep] == 0)
    # cap: entries beyond it are counted but not stored
    idx2, codes2, count2, _ = oracle.sparse_compress(x, thr, scale, oracle.P_INF, s, seed=0,
                                                     worker=6, cap=100)
    assert count2 == count and np.array_equal(idx2, idx[:100])
    assert np.array_equal(codes2, codes[:50])


def test_sparse_composition_is_unbiased_with_bounded_second_moment():
    # Thm. 3: omega_12 = omega_1 omega_2 + omega_1 + omega_2 with omega_S = 1/prob - 1
    # and omega_D from Thm. 4; checked by Monte Carlo over seeds on a small vector.
    rng = np.random.default_rng(14)
    d, s, trials = 64, 4, 4000
    x = rng.standard_normal(d).astype(np.float32)
    thr, scale = 1 << 30, 4.0                      # keep probability 1/4
    mean = np.zeros(d)
    second = 0.0
    for t in range(trials):
        idx, codes, count, nrm = oracle.sparse_compress(x, thr, scale, oracle.P_INF, s, seed=t,
                                                        worker=0)
        acc = np.zeros(d, np.float32)
        oracle.sparse_decode_accumulate(idx, codes, count, nrm, s, acc)
        mean += acc
        second += float((acc.astype(np.float64) ** 2).sum())
    mean /= trials
    second /= trials
    x2 = float((x.astype(np.float64) ** 2).sum())
    a = d ** 0.5 * 2.0 ** (1 - s)
    omega_d = 1 / 8 + a * min(1.0, a)
    bound = (omega_d + 1) * 4.0 * x2
    assert second <= bound * 1.05
    # per-coordinate standard error <= sqrt(bound_j / trials); use a global 5-sigma envelope
    err = np.abs(mean - x)
    assert np.all(err <= 5 * np.sqrt((omega_d + 1) * 4.0 * 16.0 * np.maximum(x * x, 0.05)
                                     / trials))
