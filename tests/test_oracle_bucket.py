"""Pins for the oracle's bucket scope (the quantizer applied to buckets of 128 coordinates, Section 7.1): what the
definition fixes independently of the oracle's own code path."""
import numpy as np


def _model(orc, sizes, bits, K, q, seed=7):
    m = orc.OracleModel(sizes, bits, q, K, seed)
    m.norm_scope = "bucket"
    return m


def test_bucket_norms_are_the_norms_of_the_128_chunks(orc):
    rng = np.random.default_rng(0)
    sizes = [300, 128, 1000]
    g = rng.standard_normal((2, sum(sizes))).astype(np.float32)
    for q, ordv in [(2, 2), (1, 1), (0, np.inf), (3, 3)]:
        ref = _model(orc, sizes, [3, 3, 3], 2, q).quantize(g, 1)
        off = 0
        for m, d in enumerate(sizes):
            for k in range(2):
                v = g[k, off:off + d].astype(np.float64)
                want = [np.linalg.norm(v[i:i + 128], ord=ordv) for i in range(0, d, 128)]
                assert np.allclose(ref["bucket_norms"][k][m], want, rtol=1e-6)
            off += d
        if q == 2:      # the fit weight of a layer is its Euclidean norm: sum of squared bucket norms = ||v||^2
            want = np.array([[np.linalg.norm(g[k, a:b].astype(np.float64)) for a, b in [(0, 300), (300, 428), (428, 1428)]]
                             for k in range(2)])
            assert np.allclose(ref["norms"], want, rtol=1e-6)


def test_a_layer_of_one_bucket_equals_layer_scope(orc):
    rng = np.random.default_rng(1)
    sizes = [128, 77, 1]
    g = (rng.standard_normal((3, sum(sizes))) * 0.3).astype(np.float32)
    a = _model(orc, sizes, [4, 2, 3], 3, 2); b = orc.OracleModel(sizes, [4, 2, 3], 2, 3, 7)
    ra, rb = a.quantize(g, 5, want_hist=True), b.quantize(g, 5, want_hist=True)
    for key in ["idx", "sign", "decoded", "hist", "status"]:
        assert np.array_equal(ra[key], rb[key]), key
    assert np.array_equal(ra["norms"], rb["norms"])       # one bucket: sqrt(N^2) = N exactly


def test_decoded_values_bracket_the_input_within_the_bucket_and_are_unbiased(orc):
    rng = np.random.default_rng(2)
    sizes = [512]
    g = (rng.standard_normal((1, 512)) * np.repeat([1e-3, 1.0, 30.0, 0.1], 128)).astype(np.float32)
    m = _model(orc, sizes, [3], 1, 2)
    lv = np.asarray(m.levels[0], np.float64)
    acc = np.zeros(512)
    T = 400
    for t in range(1, T + 1):
        ref = m.quantize(g, t)
        acc += ref["decoded"][0]
        if t == 1:
            bn = ref["bucket_norms"][0][0]
            u = np.abs(g[0].astype(np.float64)) / np.repeat(bn.astype(np.float64), 128)
            lo = lv[np.searchsorted(lv, u, side="right") - 1]
            hi = lv[np.minimum(np.searchsorted(lv, u, side="right"), len(lv) - 1)]
            dec_u = np.abs(ref["decoded"][0]) / np.repeat(bn, 128)
            assert np.all((np.abs(dec_u - lo) < 1e-6) | (np.abs(dec_u - hi) < 1e-6))
            assert np.all(np.sign(ref["decoded"][0]) * np.sign(g[0]) >= 0)
    # E[Q(v)] = v (Section 3.1): the mean of T draws is within 5 standard errors, where the per-draw standard
    # deviation of a coordinate is at most half its bucket's norm times the level gap
    err = np.abs(acc / T - g[0])
    bound = 5.0 * 0.5 * np.repeat(bn, 128) * np.max(np.diff(lv)) / np.sqrt(T) + 1e-7
    assert np.all(err <= bound)


def test_flags_and_zeroed_buckets(orc):
    sizes = [384, 256]
    g = np.ones((1, 640), np.float32)
    g[0, 0:128] = 0.0                       # zero bucket
    g[0, 130] = np.nan                      # bad bucket
    g[0, 384:640] = 0.0                     # a layer of zero buckets only
    ref = _model(orc, sizes, [2, 2], 1, 2).quantize(g, 1, want_hist=True)
    assert list(ref["bucket_norms"][0][0]) == [0.0, 0.0, np.float32(np.sqrt(128.0))]
    assert list(ref["status"][0]) == [2, 1]
    assert not ref["idx"][0, :256].any() and not ref["sign"][0, :256].any() and not ref["decoded"][0, :256].any()
    assert ref["hist"][0, 0].sum() == 128 and ref["hist"][0, 1].sum() == 0      # zeroed buckets add no counts
