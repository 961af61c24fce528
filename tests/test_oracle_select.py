"""Oracle pins for the exact-count sparsifier S^q (exactly q coordinates kept, chosen uniformly)
and for TopK followed by C_nat.  CPU only."""
import itertools
import math

import numpy as np

import oracle


def test_select_smallest_against_numpy_sort_with_ties():
    rng = np.random.default_rng(0)
    for d, q, hi in [(1, 1, 4), (10, 3, 3), (1000, 17, 8), (1000, 999, 1 << 32), (257, 0, 5),
                     (64, 64, 2)]:
        keys = rng.integers(0, hi, d, dtype=np.uint64).astype(np.uint32)
        mask = oracle.select_smallest(keys, q)
        order = np.lexsort((np.arange(d), keys))              # by key, then by index
        want = np.zeros(d, np.uint8)
        want[order[:q]] = 1
        assert np.array_equal(mask, want)
        assert mask.sum() == q
    # all keys equal: the first q indices
    assert np.array_equal(oracle.select_smallest(np.zeros(9, np.uint32), 4),
                          np.uint8([1, 1, 1, 1, 0, 0, 0, 0, 0]))


def test_exact_sparsifier_keeps_exactly_q_and_subsets_are_uniform():
    # d = 6, q = 2: 15 subsets, each with probability 1/15 over seeds
    d, q, trials = 6, 2, 15_000
    counts = {}
    incl = np.zeros(d)
    for seed in range(trials):
        keys = oracle.stream_words(seed, 9, 2, 0, d)
        mask = oracle.select_smallest(keys, q)
        assert mask.sum() == q
        counts[tuple(np.nonzero(mask)[0])] = counts.get(tuple(np.nonzero(mask)[0]), 0) + 1
        incl += mask
    assert set(counts) == set(itertools.combinations(range(d), q))
    expect = trials / math.comb(d, q)
    for c in counts.values():
        assert abs(c - expect) < 5 * math.sqrt(expect)
    assert np.all(np.abs(incl / trials - q / d) < 5 * math.sqrt((q / d) * (1 - q / d) / trials))


def test_exact_sparse_compress_structure_and_special_cases():
    rng = np.random.default_rng(1)
    d, s = 5000, 4
    x = rng.standard_normal(d).astype(np.float32)
    # q = d with scale 1: no sparsification, so it equals dithering of x itself (compact listing
    # of the non-zero levels of the dense operator)
    idx, planes, count, norm = oracle.sparse_exact_compress(x, d, 1.0, 0, s, 5, 3)
    nrm, level, sign = oracle.nd_compress(x, [0, d], 0, s, 5, 3)
    lv = np.zeros(d, np.uint8)
    lv[0::2] = level[:(d + 1) // 2] & 0xF
    lv[1::2] = (level[:d // 2] >> 4)
    nz = np.nonzero(lv)[0]
    assert norm == nrm[0] and count == nz.size and np.array_equal(idx, nz.astype(np.uint32))
    nb = oracle.code_bits(s) - 1
    k = np.arange(count)
    code = np.zeros(count, np.int64)
    for b in range(nb + 1):
        code |= ((planes[(k // 32) * (nb + 1) + b].astype(np.int64) >> (k % 32)) & 1) << b
    assert np.array_equal(code & ((1 << nb) - 1), lv[nz] - 1)
    sg = (sign[nz // 32] >> (nz % 32)) & 1
    assert np.array_equal(code >> nb, sg)
    # general q: listed indices are a subset of the selected set, the norm is that of the scaled
    # kept entries, and the selection is the q smallest domain-2 words
    q = 500
    scale = np.float32(d / q)
    idx, planes, count, norm = oracle.sparse_exact_compress(x, q, scale, 2, s, 5, 3)
    mask = oracle.select_smallest(oracle.stream_words(5, 3, 2, 0, d), q)
    assert mask.sum() == q and np.all(mask[idx] == 1) and count <= q
    kept = (scale * x[mask == 1]).astype(np.float64)
    assert norm == np.float32(np.sqrt((kept ** 2).sum()))
    # decoding through the compact decoder gives values 2^(c - s) * norm with the right sign
    acc = np.zeros(d, np.float32)
    oracle.sparse_compact_decode_accumulate(idx, planes, count, norm, s, acc)
    assert np.all(acc[mask == 0] == 0)
    nzv = acc[idx]
    assert np.all(np.sign(nzv) == np.sign(x[idx]))
    ratio = np.abs(nzv.astype(np.float64)) / float(norm)
    assert np.all(np.isin(np.log2(ratio), np.arange(1 - s, 1)))


def test_exact_sparse_compress_is_unbiased():
    # E[D_nat(S^q(x))] = x (composition of unbiased operators); average over seeds
    rng = np.random.default_rng(2)
    d, q, s, trials = 40, 10, 6, 6000
    x = rng.standard_normal(d).astype(np.float32)
    mean = np.zeros(d)
    for seed in range(trials):
        idx, planes, count, norm = oracle.sparse_exact_compress(x, q, np.float32(d / q), 2, s,
                                                                seed, 0)
        acc = np.zeros(d, np.float32)
        oracle.sparse_compact_decode_accumulate(idx, planes, count, norm, s, acc)
        mean += acc
    mean /= trials
    # per-coordinate std is at most about ||x'|| ~ (d/q) ||x||; generous 5 sigma bound
    sigma = (d / q) * np.linalg.norm(x) / math.sqrt(trials)
    assert np.all(np.abs(mean - x) < 5 * sigma)
    assert abs(np.mean(mean - x)) < 5 * sigma / math.sqrt(d)


def test_topk_against_numpy_and_cnat_on_the_selected_entries():
    rng = np.random.default_rng(3)
    d, K = 3000, 100
    x = rng.standard_normal(d).astype(np.float32)
    x[rng.choice(d, 200, replace=False)] = np.float32(1.5)       # many ties near the cut
    x[5] = -np.inf
    x[6] = np.float32(-0.0)
    idx, exp, sign = oracle.topk_compress(x, K, 7, 2)
    order = np.lexsort((np.arange(d), -np.abs(x).astype(np.float64)))
    want = np.sort(order[:K])
    assert np.array_equal(idx, want.astype(np.uint32))
    assert 5 in idx
    # the codes are those of dense C_nat at the selected coordinates (same stream position j)
    e_all, s_all = oracle.nc_compress(x, 7, 2)
    assert np.array_equal(exp, e_all[idx])
    k = np.arange(K)
    assert np.array_equal((sign[k // 32] >> (k % 32)) & 1, (s_all[idx // 32] >> (idx % 32)) & 1)
    # K >= d lists everything; K = 0 nothing
    idx, exp, sign = oracle.topk_compress(x, d + 5, 7, 2)
    assert np.array_equal(idx, np.arange(d, dtype=np.uint32)) and np.array_equal(exp, e_all)
    idx, exp, sign = oracle.topk_compress(x, 0, 7, 2)
    assert idx.size == 0
    # decode-accumulate scatters the decoded powers of two
    idx, exp, sign = oracle.topk_compress(x, K, 7, 2)
    acc = np.ones(d, np.float32)
    oracle.topk_decode_accumulate(idx, exp, sign, acc)
    dense = np.zeros(d, np.float32)
    oracle.nc_decode_accumulate(e_all, s_all, dense)
    ref = np.ones(d, np.float32)
    ref[idx] = np.float32(1) + dense[idx]
    assert np.array_equal(acc.view(np.uint32), ref.view(np.uint32))
