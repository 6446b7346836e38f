"""Pins of the CPU oracle's random numbers, norm, quantizer, packing and histogram.

Every check here compares the oracle with something the paper or the mathematics fixes
(published known-answer vectors, closed forms, brute-force enumeration, library
routines), never with the CUDA path.
"""
import itertools
import math
import os

import numpy as np
import pytest

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
SEED = 0x5EED0DA


# ------------------------------------------------------------------------------- Philox
def test_philox_known_answers(orc):
    rows = 0
    for line in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        assert orc.philox4x32_10(w[:4], w[4:6]) == w[6:10]
        rows += 1
    assert rows == 3


def test_uniform_keying_and_range(orc):
    # coordinate i takes word i%4 of the block with counter (i/4, layer, worker, step)
    seed = 0x0123456789ABCDEF
    for (step, worker, layer, i) in [(0, 0, 0, 0), (7, 3, 2, 5), (2 ** 32 - 1, 15, 224, 2 ** 33 + 3)]:
        out = orc.philox4x32_10([(i >> 2) & 0xFFFFFFFF, layer, worker, step],
                                [seed & 0xFFFFFFFF, seed >> 32])
        assert orc.uniform(seed, step, worker, layer, i) == (out[i & 3] >> 9) / 2.0 ** 23
    u = np.array([orc.uniform(SEED, 1, 0, 0, i) for i in range(20000)])
    assert u.min() >= 0.0 and u.max() < 1.0
    # mean and variance of U(0,1), lag-1 correlation
    assert abs(u.mean() - 0.5) < 5 * math.sqrt(1 / 12 / u.size)
    assert abs(u.var() - 1 / 12) < 0.005
    assert abs(np.corrcoef(u[:-1], u[1:])[0, 1]) < 0.03
    # different workers / layers / steps give different streams
    a = [orc.uniform(SEED, 1, 0, 0, i) for i in range(64)]
    for other in [(2, 0, 0), (1, 1, 0), (1, 0, 1)]:
        b = [orc.uniform(SEED, other[0], other[1], other[2], i) for i in range(64)]
        assert a != b


# --------------------------------------------------------------------------------- norm
@pytest.mark.parametrize("q", [0, 1, 2, 3, 5])
def test_layer_norm_matches_library(orc, q):
    rng = np.random.default_rng(q)
    v = (rng.standard_normal(10007) * 1e-3).astype(np.float32)
    ref = np.linalg.norm(v.astype(np.float64), ord=np.inf if q == 0 else q)
    n, st = orc.layer_norm(v, q)
    assert st == 0
    assert n == np.float32(ref) or abs(float(n) - ref) <= 1e-7 * ref


def test_layer_norm_flags(orc):
    assert orc.layer_norm(np.zeros(5, np.float32), 2) == (0.0, 1)
    assert orc.layer_norm(np.array([], np.float32), 2) == (0.0, 1)
    assert orc.layer_norm(np.array([1.0, np.nan], np.float32), 2) == (0.0, 2)
    assert orc.layer_norm(np.array([1.0, np.inf], np.float32), 0) == (0.0, 2)
    assert orc.layer_norm(np.array([np.nan, 1.0], np.float32), 0) == (0.0, 2)
    assert orc.layer_norm(np.array([3e38, 3e38], np.float32), 2) == (0.0, 2)   # overflows fp32
    n, st = orc.layer_norm(np.array([3.0, -4.0], np.float32), 2)
    assert (n, st) == (5.0, 0)


# ---------------------------------------------------------------------------- quantizer
def _xi_reference(v, levels, q):
    """tau and xi from the definition in Section 3.1, in float64 numpy (written independently)."""
    norm = np.linalg.norm(v.astype(np.float64), ord=np.inf if q == 0 else q)
    u = np.abs(v.astype(np.float64)) / norm
    lv = levels.astype(np.float64)
    tau = np.clip(np.searchsorted(lv, u, side="right") - 1, 0, len(lv) - 2)
    xi = (u - lv[tau]) / (lv[tau + 1] - lv[tau])
    return norm, u, tau, xi


def _sample(orc, v, levels, q, steps):
    norm, st = orc.layer_norm(v, q)
    assert st == 0
    outs = np.zeros((len(steps), v.size), np.float64)
    idxs = np.zeros((len(steps), v.size), np.int64)
    for r, s in enumerate(steps):
        idx, sg, _ = orc.quantize_layer(v, norm, levels, SEED, s, 0, 0)
        outs[r] = orc.decode_layer(idx, sg, norm, levels)
        idxs[r] = idx
    return norm, outs, idxs


def test_bruteforce_enumeration_small_vector(orc):
    """d = 6: enumerate all 2^d up/down outcomes with their probabilities; the exact mean is v
    and the exact variance is Eq. (Var); sampled outcomes follow those probabilities."""
    v = np.array([0.31, -0.07, 0.52, 0.0, -0.9, 0.23], np.float32)
    levels = np.array([0.0, 0.1, 0.25, 0.45, 0.6, 0.8, 0.9, 1.0], np.float32)
    norm, u, tau, xi = _xi_reference(v, levels, 2)
    lv = levels.astype(np.float64)
    mean = np.zeros(6); second = 0.0; probs = {}
    for ups in itertools.product([0, 1], repeat=6):
        p = np.prod([xi[i] if ups[i] else 1 - xi[i] for i in range(6)])
        qv = norm * np.sign(v) * lv[tau + np.array(ups)]
        mean += p * qv
        second += p * np.sum((qv - v) ** 2)
        probs[ups] = p
    assert np.allclose(mean, v, atol=1e-12)                                   # unbiased
    closed = norm ** 2 * np.sum((lv[tau + 1] - u) * (u - lv[tau]))            # Eq. (Var)
    assert abs(second - closed) < 1e-12

    R = 40000
    _, outs, idxs = _sample(orc, v, levels, 2, range(R))
    ups = idxs - tau[None, :]
    assert ups.min() >= 0 and ups.max() <= 1                                   # feasible set only
    # per-coordinate frequencies against xi
    freq = ups.mean(axis=0)
    sd = np.sqrt(np.maximum(xi * (1 - xi), 1e-12) / R)
    assert np.all(np.abs(freq - xi) < 5 * sd + 1e-9)
    # joint outcome chi-square over outcomes with non-negligible probability
    codes = (ups * (1 << np.arange(6))).sum(axis=1)
    chi = 0.0; dof = 0
    for o, p in probs.items():
        if p * R < 5:
            continue
        c = np.count_nonzero(codes == sum(b << i for i, b in enumerate(o)))
        chi += (c - p * R) ** 2 / (p * R); dof += 1
    assert chi < dof + 6 * math.sqrt(2 * dof)
    # empirical mean / variance
    assert np.all(np.abs(outs.mean(axis=0) - v) < 5 * np.sqrt(
        norm ** 2 * (lv[tau + 1] - u) * (u - lv[tau]) / R) + 1e-9)
    emp = np.mean(np.sum((outs - v) ** 2, axis=1))
    assert abs(emp - closed) < 0.03 * closed


@pytest.mark.parametrize("q", [2, 0, 1])
def test_unbiased_and_variance_bound(orc, q):
    """E[Q(v)] = v; E||Q(v)-v||^2 equals Eq. (Var) and stays below eps_Q ||v||_2^2 (Theorem 5.1,
    one layer: M = 1, d = d_m, maxima over j >= 1 as in the theorem's proof)."""
    rng = np.random.default_rng(11 + q)
    d = 300
    v = (rng.standard_normal(d) * 0.02).astype(np.float32)
    levels = np.array([0, 0.02, 0.05, 0.1, 0.18, 0.3, 0.55, 1.0], np.float32)
    norm, u, tau, xi = _xi_reference(v, levels, q)
    lv = levels.astype(np.float64)
    R = 3000
    _, outs, _ = _sample(orc, v, levels, q, range(100, 100 + R))
    var_i = norm ** 2 * (lv[tau + 1] - u) * (u - lv[tau])
    z = (outs.mean(axis=0) - v) / np.sqrt(np.maximum(var_i, 1e-30) / R)
    assert np.all(np.abs(z[var_i > 0]) < 5.0)
    closed = var_i.sum()
    emp = np.mean(np.sum((outs - v) ** 2, axis=1))
    assert abs(emp - closed) < 0.05 * closed
    lbar = np.max(lv[2:] / lv[1:-1]); l1 = lv[1]; qq = min(q if q else 2, 2)
    dth = (2 / l1) ** qq
    eps = (lbar - 1) ** 2 / (4 * lbar) + ((l1 * d ** (1 / qq) - 1) if d >= dth
                                          else (l1 ** 2 / 4) * d ** (2 / qq))
    assert closed <= eps * np.sum(v.astype(np.float64) ** 2) * (1 + 1e-9)
    # per-interval constant of the proof: (l_{j+1}-u)(u-l_j) <= k_j u^2, k_j = (r-1)^2/(4r)
    j = tau >= 1
    r = lv[tau[j] + 1] / lv[tau[j]]
    assert np.all((lv[tau[j] + 1] - u[j]) * (u[j] - lv[tau[j]]) <= (r - 1) ** 2 / (4 * r) * u[j] ** 2 + 1e-15)


def test_values_on_levels_are_deterministic(orc):
    levels = np.array([0, 0.25, 0.5, 1.0], np.float32)
    v = np.array([1.0, 0.5, -0.25, 0.0, -1.0], np.float32)      # q = inf: norm 1, u on levels
    for s in range(200):
        idx, sg, _ = orc.quantize_layer(v, 1.0, levels, SEED, s, 1, 2)
        assert idx.tolist() == [3, 2, 1, 0, 3] and sg.tolist() == [0, 0, 1, 0, 1]


def test_one_bit_inf_norm_is_bernoulli(orc):
    """b = 1 (levels {0,1}) with the max norm: Q(v_i) = N sign(v_i) Bernoulli(|v_i|/N)."""
    v = np.array([0.8, -0.2, 0.4, -0.8, 0.05], np.float32)
    levels = np.array([0.0, 1.0], np.float32)
    norm, outs, idxs = _sample(orc, v, levels, 0, range(20000))
    assert norm == np.float32(0.8)
    p = np.abs(v.astype(np.float64)) / 0.8
    f = idxs.mean(axis=0)
    assert np.all(np.abs(f - p) < 5 * np.sqrt(np.maximum(p * (1 - p), 1e-9) / 20000) + 1e-9)
    assert set(np.unique(np.abs(outs))) <= {0.0, float(np.float32(0.8))}


def test_uniform_levels_reduce_to_floor_plus_bernoulli(orc):
    """Uniform levels j/s: idx is floor(u s) or floor(u s)+1 (QSGD-style rounding)."""
    rng = np.random.default_rng(5)
    v = rng.standard_normal(5000).astype(np.float32)
    levels = orc.uniform_levels(3)
    norm, _ = orc.layer_norm(v, 2)
    idx, sg, _ = orc.quantize_layer(v, norm, levels, SEED, 3, 0, 0)
    u = np.abs(v.astype(np.float64)) / float(norm)
    fl = np.floor(u * 7 + 1e-9).astype(int)
    inside = np.abs(u * 7 - np.round(u * 7)) > 1e-5
    d = idx.astype(int) - fl
    assert np.all((d[inside] == 0) | (d[inside] == 1))
    assert np.array_equal(sg, (v < 0).astype(np.uint8))
    # expected index equals u*s
    R = 400
    acc = np.zeros(v.size)
    for s in range(R):
        acc += orc.quantize_layer(v, norm, levels, SEED, 1000 + s, 0, 0)[0]
    assert abs((acc / R - u * 7).mean()) < 0.01


def test_negative_zero_has_sign_zero(orc):
    levels = orc.uniform_levels(2)
    v = np.array([-0.0, 0.0, -1e-30, 1.0, -1.0], np.float32)
    idx, sg, _ = orc.quantize_layer(v, 1.0, levels, SEED, 0, 0, 0)
    assert sg.tolist() == [0, 0, 1, 0, 1] and idx[:2].tolist() == [0, 0]


def test_zero_norm_gives_zero_message(orc):
    levels = orc.uniform_levels(4)
    idx, sg, near = orc.quantize_layer(np.array([1.0, -2.0], np.float32), 0.0, levels, SEED, 0, 0, 0)
    assert idx.tolist() == [0, 0] and sg.tolist() == [0, 0] and near == 0


def test_near_threshold_fraction_is_tiny(orc):
    rng = np.random.default_rng(8)
    v = rng.standard_normal(200000).astype(np.float32)
    norm, _ = orc.layer_norm(v, 2)
    *_, near = orc.quantize_layer(v, norm, orc.uniform_levels(4), SEED, 0, 0, 0)
    # |rho*den - num| <= 1e-6 den happens with probability about 2e-6 per coordinate
    assert near <= 6


# --------------------------------------------------------------------------------- pack
def test_pack_roundtrip_all_widths_and_tails(orc):
    rng = np.random.default_rng(1)
    for b in range(1, 9):
        for d in list(range(0, 35)) + [127, 128, 129, 1023, 1024, 1025, 2500]:
            idx = rng.integers(0, 1 << b, d).astype(np.uint8)
            sg = rng.integers(0, 2, d).astype(np.uint8)
            w = orc.pack_layer(idx, sg, b)
            assert w.size == ((d + 1023) // 1024) * 32 * (b + 1)
            i2, s2 = orc.unpack_layer(w, d, b)
            assert np.array_equal(i2, idx) and np.array_equal(s2, sg)


def test_pack_layout_hand_worked_positions(orc):
    """Positions worked out by hand from the layout text: block of 1024 coordinates, lane
    (c/4)%32, position p = 4*(c/128) + c%4, symbol = 2*idx + sign of b+1 bits at bit offset
    p*(b+1) of the lane's string, bit t in word (t/32)*32 + lane."""
    b = 3                                      # 4-bit symbols, 4 planes of 32 words per block
    d = 1200
    for (i, code, expect) in [
        # i = 0: block 0, lane 0, p 0 -> symbol 101|1 = 1011 in bits 0..3 of word 0
        (0, 0b101, {0: 0b1011}),
        # i = 129: c = 129, lane 32%32 = 0, p = 4*1+1 = 5 -> bits 20..23 of word 0
        (129, 0b111, {0: 0b1111 << 20}),
        # i = 7: lane 1, p = 3 -> bits 12..15 of word 1; symbol 010|1 = 0101
        (7, 0b010, {1: 0b0101 << 12}),
        # i = 1023: lane 31, p = 31 -> bits 124..127 -> plane 3 (word 96+31) bits 28..31; symbol 110|1
        (1023, 0b110, {96 + 31: 0b1101 << 28}),
        # i = 427: lane 106%32 = 10, p = 4*3+3 = 15 -> bits 60..63 -> plane 1 (word 32+10) bits 28..31; 011|1
        (427, 0b011, {32 + 10: 0b0111 << 28}),
        # second block: i = 1028 -> block base 128 words, lane 1, p 0; symbol 001|1
        (1028, 0b001, {128 + 1: 0b0011}),
    ]:
        idx = np.zeros(d, np.uint8); sg = np.zeros(d, np.uint8)
        idx[i] = code; sg[i] = 1
        w = orc.pack_layer(idx, sg, b)
        got = {int(j): int(w[j]) for j in np.flatnonzero(w)}
        assert got == expect, (i, got, expect)
    # a positive coordinate leaves bit 0 of its symbol clear: i = 4 (lane 1, p 0), idx 6 -> 1100
    idx = np.zeros(d, np.uint8); sg = np.zeros(d, np.uint8); idx[4] = 6
    w = orc.pack_layer(idx, sg, b)
    assert {int(j): int(w[j]) for j in np.flatnonzero(w)} == {1: 0b1100}
    # b = 4: 5-bit symbols straddle words; p = 6 (i = 128 + 4*lane + 2, lane 3 -> i = 142) sits at
    # bits 30..34: two bits in plane 0 and three in plane 1
    idx = np.zeros(200, np.uint8); sg = np.zeros(200, np.uint8)
    idx[142] = 0b1011; sg[142] = 1                  # symbol 1011|1 = 10111
    w = orc.pack_layer(idx, sg, 4)
    got = {int(j): int(w[j]) for j in np.flatnonzero(w)}
    assert got == {3: 0b11 << 30, 32 + 3: 0b101}


# ---------------------------------------------------------------------------- histogram
def test_histogram_bins(orc):
    rng = np.random.default_rng(3)
    v = (rng.standard_normal(50000) * np.exp(rng.uniform(-12, 0, 50000))).astype(np.float32)
    v[:7] = [0.0, 1e-30, -5.0, 5.0, 2.0 ** -24 * 5.0, 2.0 ** -25 * 5.0, 0.3]
    norm, _ = orc.layer_norm(v, 0)                                   # max norm -> some u = 1
    h = orc.histogram_layer(v, norm)
    assert h.sum() == v.size and h[386:].sum() == 0
    r = np.float32(1.0) / norm
    u = np.minimum(np.abs(v) * r, np.float32(1.0)).astype(np.float32)
    # edges from their definition: 0, then 2^(e-24) (1 + m/16), last bin = {1}
    edges = np.array([0.0] + [math.ldexp(1 + m / 16, -24 + o) for o in range(24) for m in range(16)] + [1.0])
    assert len(edges) == 386
    assert np.allclose([orc.bin_edge(i) for i in range(386)], edges, rtol=0, atol=0)
    ref = np.bincount(np.searchsorted(edges, u.astype(np.float64), side="right") - 1, minlength=386)
    assert np.array_equal(h[:386], ref)
    # the same bins from the bit pattern of u
    bits = u.view(np.uint32).astype(np.int64)
    trick = np.where(bits < 0x33800000, 0, 1 + ((bits - 0x33800000) >> 19))
    assert np.array_equal(np.bincount(trick, minlength=386), ref)
    assert h[385] == 2                                               # the two entries with |v| = max


# --------------------------------------------------------------------- decode / aggregate
def test_decode_and_aggregate(orc):
    rng = np.random.default_rng(9)
    levels = np.sort(np.concatenate([[0, 1], rng.uniform(0, 1, 14)])).astype(np.float32)
    idx = rng.integers(0, 16, 1000).astype(np.uint8); sg = rng.integers(0, 2, 1000).astype(np.uint8)
    norm = np.float32(3.7)
    out = orc.decode_layer(idx, sg, norm, levels)
    assert np.array_equal(out, np.where(sg == 1, -1, 1).astype(np.float32) * (norm * levels[idx]))
    assert np.array_equal(orc.aggregate(out[None, :]), out)           # K = 1 is the identity
    dec = rng.standard_normal((5, 1000)).astype(np.float32)
    g = orc.aggregate(dec)
    assert np.allclose(g, dec.astype(np.float64).mean(axis=0), rtol=1e-5, atol=1e-7)


def test_global_norm_scope_is_the_formal_definition(orc):
    """Section 3.1 defines Q with the norm of the whole vector and a level sequence per type.  With the global
    scope every layer is normalised by ||v||_q of the concatenation; quantizing layer by layer with that norm is
    the same as quantizing the concatenation when all layers share one sequence; and it stays unbiased."""
    rng = np.random.default_rng(31)
    sizes = [40, 7, 100]
    v = (rng.standard_normal((1, sum(sizes))) * np.repeat([1.0, 0.01, 0.1], sizes)).astype(np.float32)
    model = orc.OracleModel(sizes, [3, 3, 3], 2, 1, SEED)
    model.norm_scope = "global"
    out = model.quantize(v, 4)
    gn = np.float32(np.linalg.norm(v[0].astype(np.float64)))
    assert np.all(out["norms"] == gn)
    # one shared sequence: identical to a single layer of 147 coordinates except for the Philox keying by layer;
    # check through the probabilities instead: the decoded values are N * l_idx with idx a neighbour of u's interval
    lv = orc.uniform_levels(3).astype(np.float64)
    u = np.abs(v[0].astype(np.float64)) / float(gn)
    tau = np.clip(np.searchsorted(lv, u, side="right") - 1, 0, 6)
    assert np.all((out["idx"][0] == tau) | (out["idx"][0] == tau + 1))
    # unbiased with the shared norm: mean of many draws
    acc = np.zeros(v.shape[1]); R = 4000
    for s in range(R):
        acc += model.quantize(v, 100 + s)["decoded"][0]
    var = float(gn) ** 2 * (lv[tau + 1] - u) * (u - lv[tau])
    z = (acc / R - v[0]) / np.sqrt(np.maximum(var, 1e-30) / R)
    assert np.all(np.abs(z[var > 0]) < 5.0)
