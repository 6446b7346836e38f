"""Parity of the CUDA library (through its C ABI) with the CPU oracle on seeded inputs.

Tolerances: packed signs and level indices bit-exact except coordinates within 1e-6 of a
rounding threshold (fewer than 1e-6 of all coordinates); layer norms relative 1e-6; decoded
and aggregated values relative 1e-6 (against the layer's largest magnitude); QODA iterates
relative 1e-5.
"""
import math

import numpy as np
import pytest
import torch

from helpers import compare_messages, oracle_model, to_padded, to_unpadded

pytestmark = pytest.mark.gpu
SEED = 0x5EED0DA
RAGGED = [0, 1, 31, 32, 33, 127, 128, 129, 1023, 1024, 1025, 8191, 8192, 8193, 20000, 3, 70001]


@pytest.fixture(scope="module")
def lqm():
    import paper_2505_14371_b200 as pkg
    pkg.load_library()
    return pkg


def _grads(plan, seed, scale=1.0):
    g = torch.Generator(device="cuda").manual_seed(seed)
    x = torch.randn((plan.num_workers, plan.padded_elems), generator=g, device="cuda") * scale
    return x.contiguous()


def _random_levels(rng, n):
    inner = np.sort(rng.uniform(0.0, 1.0, n - 2) ** 3)
    lv = np.concatenate([[0.0], inner, [1.0]]).astype(np.float32)
    for j in range(1, n):                       # strictly increasing in fp32
        if lv[j] <= lv[j - 1]:
            lv[j] = np.nextafter(lv[j - 1], np.float32(2.0))
    lv[-1] = 1.0
    return lv


def _close(a, b, rel, scale=None):
    a = np.asarray(a, np.float64); b = np.asarray(b, np.float64)
    s = np.max(np.abs(b)) if scale is None else scale
    return np.max(np.abs(a - b), initial=0.0) <= rel * max(s, 1e-300)


@pytest.mark.parametrize("q", [2, 0, 1, 3])
def test_layer_norms(lqm, orc, q):
    plan = lqm.Plan(RAGGED, 4, q, 3, SEED)
    grads = _grads(plan, 1, 0.01)
    norms = plan.empty_norms()
    plan.lq_layer_norms(grads, norms)
    g = to_unpadded(plan, grads)
    off = np.concatenate([[0], np.cumsum(RAGGED)])
    got = norms.cpu().numpy()
    for k in range(3):
        for m in range(len(RAGGED)):
            ref, st = orc.layer_norm(g[k, off[m]:off[m + 1]], q)
            assert abs(float(got[k, m]) - float(ref)) <= 1e-6 * float(ref), (k, m)
    _, flags = plan.lq_get_statistics()
    assert flags[:, 0].tolist() == [lqm.STATUS_ZERO_NORM] * 3 and int(flags[:, 1:].sum()) == 0


@pytest.mark.parametrize("bits", [1, 2, 3, 4, 5, 6, 7, 8])
def test_quantize_pack_all_widths_ragged(lqm, orc, bits):
    rng = np.random.default_rng(bits)
    plan = lqm.Plan(RAGGED, bits, 2, 2, SEED + bits)
    if bits > 1:
        for m in range(plan.num_layers):
            if m % 2:
                plan.lq_set_levels(m, _random_levels(rng, 1 << bits))
    grads = _grads(plan, 10 + bits)
    packed = plan.empty_packed(); norms = plan.empty_norms(); hist = plan.zero_hist()
    plan.lq_quantize_pack(grads, 5, packed, norms, hist=hist)
    model = oracle_model(orc, plan)
    ref = model.quantize(to_unpadded(plan, grads), 5, want_hist=True)
    assert np.array_equal(norms.cpu().numpy()[:, :plan.num_layers], ref["norms"])
    bad, stray = compare_messages(orc, plan, packed, ref)
    assert bad == 0 and stray == 0
    assert np.array_equal(hist.cpu().numpy().view(np.uint32), ref["hist"])
    sq, _ = plan.lq_get_statistics()
    assert _close(sq.numpy(), ref["sq_diff"], 1e-12)


def test_config1_mlp_single_step(lqm, orc):
    """4-layer MLP gradient set, K=4, 3-bit uniform levels: quantize -> decode-aggregate -> QODA."""
    from paper_2505_14371_b200 import workloads as W
    w = W.mlp_workload()
    plan = lqm.Plan(w.layer_sizes, w.bits, w.q, w.num_workers, W.PHILOX_SEED)
    grads = W.make_gradients(w, plan.elem_offsets, plan.padded_elems, "cuda")
    packed = plan.empty_packed(); norms = plan.empty_norms()
    gbar = torch.zeros(plan.padded_elems, device="cuda")
    X1 = _grads(plan, 77)[0].contiguous(); Y = torch.empty_like(X1); Xh = torch.empty_like(X1)
    X = torch.empty_like(X1); g2 = torch.empty_like(X1)
    plan.qoda_init(X1, Y, Xh)
    plan.lq_quantize_pack(grads, 1, packed, norms)
    plan.lq_decode_aggregate(packed, norms, gbar)
    plan.qoda_step(packed, norms, X1, Y, Xh, X, g2)

    model = oracle_model(orc, plan)
    model.qoda_init(to_unpadded(plan, X1))
    ref = model.quantize(to_unpadded(plan, grads), 1)
    bad, stray = compare_messages(orc, plan, packed, ref)
    total = w.num_coords * w.num_workers
    assert stray == 0 and bad <= max(1, int(1e-6 * total)) and ref["near"] < 1e-5 * total
    assert _close(norms.cpu().numpy(), ref["norms"], 1e-6)
    gref = model.qoda_step()
    off = np.concatenate([[0], np.cumsum(w.layer_sizes)])
    if bad == 0:
        for name, got, want in [("gbar", gbar, gref), ("gbar2", g2, gref), ("Y", Y, model.Y),
                                ("X", X, model.X), ("Xhalf", Xh, model.Xhalf)]:
            gg = to_unpadded(plan, got)
            for m in range(plan.num_layers):
                assert _close(gg[off[m]:off[m + 1]], want[off[m]:off[m + 1]], 1e-6), (name, m)
    t, S, eta = plan.qoda_get_scalars()
    assert t == 2 and abs(S - model.S) <= 1e-12 * model.S and eta == float(model.eta)


def test_statistic_with_previous_message_and_level_change(lqm, orc):
    rng = np.random.default_rng(4)
    sizes = [5000, 33, 12345]
    plan = lqm.Plan(sizes, [4, 3, 2], 2, 3, SEED)
    model = oracle_model(orc, plan)
    pk = [plan.empty_packed(), plan.empty_packed()]; nm = [plan.empty_norms(), plan.empty_norms()]
    for step in range(1, 5):
        if step == 3:                            # levels change between two messages
            for m, b in enumerate(plan.bits):
                lv = _random_levels(rng, 1 << b)
                plan.lq_set_levels(m, lv); model.levels[m] = lv
        grads = _grads(plan, 100 + step, 0.1)
        cur, prv = pk[step % 2], pk[(step + 1) % 2]
        plan.lq_quantize_pack(grads, step, cur, nm[step % 2],
                              prev_packed=None if step == 1 else prv,
                              prev_norms=None if step == 1 else nm[(step + 1) % 2])
        ref = model.quantize(to_unpadded(plan, grads), step)
        model.prev_decoded = ref["decoded"]
        bad, stray = compare_messages(orc, plan, cur, ref)
        assert bad == 0 and stray == 0
        sq, _ = plan.lq_get_statistics()
        assert _close(sq.numpy(), ref["sq_diff"], 1e-12), step


def test_zero_rows_and_negative_zero(lqm, orc):
    """Long runs of +0 and -0 (rows nobody touched): symbols 0, sign 0, and the statistic still sees
    the previous message where the current one is zero."""
    sizes = [9000, 70001, 300]
    plan = lqm.Plan(sizes, [4, 3, 4], 2, 2, SEED)
    model = oracle_model(orc, plan)
    pk = [plan.empty_packed(), plan.empty_packed()]; nm = [plan.empty_norms(), plan.empty_norms()]
    o = plan.elem_offsets
    for step in range(1, 4):
        grads = _grads(plan, 40 + step, 0.3)
        a = 1024 * step
        grads[:, o[0] + a: o[0] + a + 3000] = 0.0
        grads[0, o[1] + 100: o[1] + 60000] *= 0.0          # leaves -0.0 where the value was negative
        grads[1, o[1] + 30000 + 128 * step: o[1] + 30000 + 128 * step + 4096] = -0.0
        if step == 3:
            grads[:, o[2]: o[2] + 300] = -0.0               # a whole layer of -0: zero norm
        c, p = step % 2, (step + 1) % 2
        plan.lq_quantize_pack(grads, step, pk[c], nm[c], prev_packed=None if step == 1 else pk[p],
                              prev_norms=None if step == 1 else nm[p])
        ref = model.quantize(to_unpadded(plan, grads), step)
        model.prev_decoded = ref["decoded"]
        assert compare_messages(orc, plan, pk[c], ref) == (0, 0)
        sq, _ = plan.lq_get_statistics()
        assert _close(sq.numpy(), ref["sq_diff"], 1e-12), step


@pytest.mark.parametrize("K", [1, 4, 11, 16, 33, 40])
def test_decode_aggregate_worker_counts(lqm, orc, K):
    sizes = [4100, 7, 1024, 2049]
    plan = lqm.Plan(sizes, [4, 8, 1, 3], 0, K, SEED)
    grads = _grads(plan, K)
    packed = plan.empty_packed(); norms = plan.empty_norms()
    gbar = torch.full((plan.padded_elems,), 7.0, device="cuda")
    plan.lq_quantize_pack(grads, 9, packed, norms)
    plan.lq_decode_aggregate(packed, norms, gbar)
    model = oracle_model(orc, plan)
    ref = model.quantize(to_unpadded(plan, grads), 9)
    assert compare_messages(orc, plan, packed, ref) == (0, 0)
    want = model.mean_decoded(ref["decoded"])
    got = to_unpadded(plan, gbar)
    assert np.array_equal(got, want)             # fixed summation order: bit-exact


def test_nonfinite_and_zero_layers(lqm, orc):
    sizes = [1500, 1500, 1500, 64]
    plan = lqm.Plan(sizes, 4, 2, 2, SEED)
    grads = _grads(plan, 3)
    o = plan.elem_offsets
    grads[0, o[1] + 5] = float("nan")
    grads[1, o[2] + 1400] = float("inf")
    grads[:, o[3]: o[3] + 64] = 0.0
    packed = plan.empty_packed(); norms = plan.empty_norms(); gbar = torch.empty(plan.padded_elems, device="cuda")
    plan.lq_quantize_pack(grads, 2, packed, norms)
    plan.lq_decode_aggregate(packed, norms, gbar)
    torch.cuda.synchronize()
    _, flags = plan.lq_get_statistics()
    assert flags.tolist() == [[0, lqm.STATUS_NONFINITE, 0, lqm.STATUS_ZERO_NORM],
                              [0, 0, lqm.STATUS_NONFINITE, lqm.STATUS_ZERO_NORM]]
    model = oracle_model(orc, plan)
    ref = model.quantize(to_unpadded(plan, grads), 2)
    assert ref["status"].tolist() == [[0, 2, 0, 1], [0, 0, 2, 1]]
    assert compare_messages(orc, plan, packed, ref) == (0, 0)
    assert np.array_equal(norms.cpu().numpy(), ref["norms"])
    assert np.array_equal(to_unpadded(plan, gbar), model.mean_decoded(ref["decoded"]))
    assert torch.isfinite(gbar[: o[3] + 64]).all()


def test_fit_levels_parity(lqm, orc):
    from paper_2505_14371_b200 import workloads as W
    w = W.wgan_workload()
    sizes = [s // 16 for s in w.layer_sizes]
    w.layer_sizes = sizes
    plan = lqm.Plan(sizes, [3, 4, 2, 8, 3, 4, 5, 3, 1], 2, 4, SEED)
    grads = W.make_gradients(w, plan.elem_offsets, plan.padded_elems, "cuda", workers=4)
    packed = plan.empty_packed(); norms = plan.empty_norms(); hist = plan.zero_hist()
    model = oracle_model(orc, plan)               # holds the levels before the fit
    plan.lq_quantize_pack(grads, 1, packed, norms, hist=hist)
    plan.lq_fit_levels(hist, norms, 4)
    h = hist.cpu().numpy().view(np.uint32); n = norms.cpu().numpy()
    for m, b in enumerate(plan.bits):
        got = np.array(plan.lq_get_levels(m))
        want = orc.fit_levels(h[:, m, :], n[:, m], sizes[m], 1 << b)
        if want is None:
            want = model.levels[m]
        assert np.allclose(got, want, rtol=1e-6, atol=0), m
        assert got[0] == 0 and got[-1] == 1 and np.all(np.diff(got) > 0)
    # the fitted levels are used by the next message, and the previous one still decodes with the old ones
    packed2 = plan.empty_packed(); norms2 = plan.empty_norms()
    plan.lq_quantize_pack(grads, 2, packed2, norms2, prev_packed=packed, prev_norms=norms)
    ref1 = model.quantize(to_unpadded(plan, grads), 1)
    model.prev_decoded = ref1["decoded"]
    for m in range(plan.num_layers):
        model.levels[m] = np.array(plan.lq_get_levels(m), np.float32)
    ref2 = model.quantize(to_unpadded(plan, grads), 2)
    assert compare_messages(orc, plan, packed2, ref2) == (0, 0)
    sq, _ = plan.lq_get_statistics()
    assert _close(sq.numpy(), ref2["sq_diff"], 1e-12)


def test_fitted_levels_minimise_the_variance_on_the_samples(lqm):
    """The GPU's fitted levels checked against the paper's objective directly, without the oracle's solver: the
    weighted variance per unit norm (Eq. Var with the weights of Eq. cdf_weight), evaluated on the samples in numpy,
    is smaller at the fitted levels than at perturbed, uniform or exponential levels, and every interior level
    satisfies the first-order condition int_a^b (u - a) dF~ = int_b^c (c - u) dF~ on the samples."""
    K, d = 3, 300000
    rng = np.random.default_rng(2024)
    plan = lqm.Plan([d, d], [4, 3], 2, K, SEED)
    grads = torch.zeros((K, plan.padded_elems), device="cuda")
    draws = [[rng.laplace(size=d) * s for s in (1.0, 3.0, 0.2)], [rng.standard_t(3, size=d) * s for s in (0.5, 1.0, 2.0)]]
    for m in range(2):
        for k in range(K):
            grads[k, plan.elem_offsets[m]: plan.elem_offsets[m] + d] = torch.from_numpy(draws[m][k].astype(np.float32)).cuda()
    packed, norms, hist = plan.empty_packed(), plan.empty_norms(), plan.zero_hist()
    plan.lq_quantize_pack(grads, 1, packed, norms, hist=hist)
    plan.lq_fit_levels(hist, norms, K)
    torch.cuda.synchronize()
    N = norms.cpu().numpy().astype(np.float64)
    for m, n in ((0, 16), (1, 8)):
        lv = np.array(plan.lq_get_levels(m), np.float64)
        assert lv[0] == 0 and lv[-1] == 1 and np.all(np.diff(lv) > 0)
        v = grads[:, plan.elem_offsets[m]: plan.elem_offsets[m] + d].cpu().numpy().astype(np.float64)
        u = np.minimum(np.abs(v) / N[:, m: m + 1], 1.0)
        lam = N[:, m] ** 2 / np.sum(N[:, m] ** 2)

        def variance(levels):
            tau = np.clip(np.searchsorted(levels, u.ravel(), side="right") - 1, 0, len(levels) - 2).reshape(u.shape)
            return float(np.sum(lam * np.mean((levels[tau + 1] - u) * (u - levels[tau]), axis=1)))
        f_fit = variance(lv)
        assert f_fit < variance(np.arange(n) / (n - 1.0))
        assert f_fit < variance(np.concatenate([[0.0], 2.0 ** -np.arange(n - 2, -1, -1.0)]))
        # (the fit sees the samples through 16 bins per octave: perturbations smaller than a bin can win by a hair)
        for _ in range(60):
            pert = lv.copy()
            j = int(rng.integers(1, n - 1))
            pert[j] += rng.choice([-1, 1]) * rng.uniform(0.1, 0.4) * min(pert[j] - pert[j - 1], pert[j + 1] - pert[j])
            assert variance(pert) >= f_fit * (1 - 2e-3), (m, j)
        for j in range(1, n - 1):
            a, b, c = lv[j - 1], lv[j], lv[j + 1]
            left = float(np.sum(lam * np.mean(np.where((u >= a) & (u < b), u - a, 0.0), axis=1)))
            right = float(np.sum(lam * np.mean(np.where((u >= b) & (u < c), c - u, 0.0), axis=1)))
            if min(((u >= a) & (u < b)).sum(), ((u >= b) & (u < c)).sum()) < 20000:      # too few samples to compare
                continue
            assert abs(left - right) <= 0.04 * max(left, right), (m, j, left, right)


def test_fit_ends_in_the_lower_of_two_minima(lqm, orc):
    """A density constant on [0, 3/11] and 4/125 as high above has, with four levels, two local minima of the fit's
    objective; (1/5, 1/2) satisfies both first-order conditions and is the lower one (the CPU suite finds it by brute
    force), the quantile start alone ends near (0.136, 0.272).  Max norm, so that u is the value itself."""
    s, r = 3.0 / 11.0, 4.0 / 125.0
    mass1 = s / (s + r * (1.0 - s))
    N = 1 << 22
    q = (np.arange(N) + 0.5) / N
    u = np.where(q < mass1, q / mass1 * s, s + (q - mass1) / (1.0 - mass1) * (1.0 - s)).astype(np.float32)
    v = np.concatenate([u, np.float32([1.0])])
    v[1::2] *= -1
    plan = lqm.Plan([v.size], [2], 0, 1, SEED)
    grads = torch.zeros((1, plan.padded_elems), device="cuda")
    grads[0, : v.size] = torch.from_numpy(v).cuda()
    packed, norms, hist = plan.empty_packed(), plan.empty_norms(), plan.zero_hist()
    plan.lq_quantize_pack(grads, 1, packed, norms, hist=hist)
    plan.lq_fit_levels(hist, norms, 1)
    got = np.array(plan.lq_get_levels(0))
    assert norms.cpu().numpy().ravel()[0] == 1.0
    # (the step at 3/11 is smeared over the histogram bin [17/64, 18/64]: a few 1e-3 of slack)
    assert abs(got[1] - 0.2) < 2e-3 and abs(got[2] - 0.5) < 4e-3, got
    h = hist.cpu().numpy().view(np.uint32)
    want = orc.fit_levels(h[:, 0, :], norms.cpu().numpy()[:, 0], v.size, 4)
    assert np.allclose(got, want, rtol=1e-6, atol=0)


def test_statistic_with_a_copy_of_the_previous_message(lqm, orc):
    """prev_packed at another address than the buffer the last call wrote (a copy, a message that travelled), and
    the same buffer after lq_message_modified: the plan may not skip words by what it remembers, and the statistic
    and the update stay those of the oracle."""
    sizes, K = [9000, 3000], 3
    outs = []
    for mode in ("same", "copy", "modified"):
        plan = lqm.Plan(sizes, [4, 3], 2, K, SEED)
        model = oracle_model(orc, plan)
        X1 = _grads(plan, 5)[0].contiguous(); Y = torch.empty_like(X1); Xh = torch.empty_like(X1)
        plan.qoda_init(X1, Y, Xh); model.qoda_init(to_unpadded(plan, X1))
        pk = [plan.empty_packed(), plan.empty_packed()]; nm = [plan.empty_norms(), plan.empty_norms()]
        for t in (1, 2, 3):
            grads = _grads(plan, 300 + t)
            grads[0, 1024:5000] = 0.0                                   # rows and blocks of zeros in one worker
            if t == 2:
                grads[1, :] = 0.0
            c, p = t % 2, (t + 1) % 2
            prev = pk[p]
            if t > 1 and mode == "copy":
                prev = pk[p].clone()
            if t > 1 and mode == "modified":
                pk[p].copy_(pk[p].clone())                              # rewritten in place (here: with the same words)
                plan.lq_message_modified()
            plan.lq_quantize_pack(grads, t, pk[c], nm[c], prev_packed=None if t == 1 else prev,
                                  prev_norms=None if t == 1 else nm[p])
            ref = model.quantize(to_unpadded(plan, grads), t)
            assert compare_messages(orc, plan, pk[c], ref) == (0, 0)
            sq, _ = plan.lq_get_statistics()
            assert _close(sq.numpy(), ref["sq_diff"], 1e-12), (mode, t)
            msg = pk[c]
            if mode == "modified":
                plan.lq_message_modified()
            plan.qoda_step(msg, nm[c], X1, Y, Xh)
            model.qoda_step()
            assert _close(to_unpadded(plan, Y), model.Y, 1e-6) and _close(to_unpadded(plan, Xh), model.Xhalf, 1e-6)
        outs.append((Y.cpu().numpy().copy(), Xh.cpu().numpy().copy()))
    for a, b in zip(outs[0], outs[1]):
        assert np.array_equal(a, b)
    for a, b in zip(outs[0], outs[2]):
        assert np.array_equal(a, b)


def test_qoda_multi_step_small(lqm, orc):
    """20 iterations with random 'gradients' that depend on nothing: state parity every step."""
    sizes = [3000, 100, 2048]
    plan = lqm.Plan(sizes, 4, 2, 4, SEED)
    model = oracle_model(orc, plan)
    X1 = _grads(plan, 5)[0].contiguous(); Y = torch.empty_like(X1); Xh = torch.empty_like(X1)
    plan.qoda_init(X1, Y, Xh)
    model.qoda_init(to_unpadded(plan, X1))
    pk = [plan.empty_packed(), plan.empty_packed()]; nm = [plan.empty_norms(), plan.empty_norms()]
    for t in range(1, 21):
        grads = _grads(plan, 1000 + t, 1.0 / t)
        c, p = t % 2, (t + 1) % 2
        plan.lq_quantize_pack(grads, t, pk[c], nm[c], prev_packed=None if t == 1 else pk[p],
                              prev_norms=None if t == 1 else nm[p])
        plan.qoda_step(pk[c], nm[c], X1, Y, Xh)
        ref = model.quantize(to_unpadded(plan, grads), t)
        assert compare_messages(orc, plan, pk[c], ref) == (0, 0)
        model.qoda_step()
        tt, S, eta = plan.qoda_get_scalars()
        assert tt == t + 1 and abs(S - model.S) <= 1e-12 * model.S and eta == float(model.eta)
        assert _close(to_unpadded(plan, Y), model.Y, 1e-6) and _close(to_unpadded(plan, Xh), model.Xhalf, 1e-6)


def test_qoda_step_more_than_32_workers(lqm, orc):
    """K = 37: the decoder's per-block worker bitmask covers 32 workers, so every word must be read; three
    iterations of encode + fused update against the oracle, with blocks that only some workers fill."""
    sizes, K = [5000, 33, 2048], 37
    plan = lqm.Plan(sizes, [3, 5, 4], 2, K, SEED)
    model = oracle_model(orc, plan)
    X1 = _grads(plan, 5)[0].contiguous(); Y = torch.empty_like(X1); Xh = torch.empty_like(X1)
    plan.qoda_init(X1, Y, Xh)
    model.qoda_init(to_unpadded(plan, X1))
    pk = [plan.empty_packed(), plan.empty_packed()]; nm = [plan.empty_norms(), plan.empty_norms()]
    for t in range(1, 4):
        grads = _grads(plan, 2000 + t)
        grads[:30, 1024:3072] = 0.0                     # blocks that only workers 30..36 fill
        grads[34:, :1024] = 0.0
        c, p = t % 2, (t + 1) % 2
        plan.lq_quantize_pack(grads, t, pk[c], nm[c], prev_packed=None if t == 1 else pk[p],
                              prev_norms=None if t == 1 else nm[p])
        plan.qoda_step(pk[c], nm[c], X1, Y, Xh)
        ref = model.quantize(to_unpadded(plan, grads), t)
        assert compare_messages(orc, plan, pk[c], ref) == (0, 0)
        model.qoda_step()
        assert _close(to_unpadded(plan, Y), model.Y, 1e-6) and _close(to_unpadded(plan, Xh), model.Xhalf, 1e-6)


@pytest.mark.parametrize("bits", [5, 6, 8])
def test_levels_crowded_into_one_search_bin(lqm, orc, bits):
    """Level sets too dense for the one-lookup search (it takes at most one level per 1/32 of an octave): most
    interior levels a few ulps apart just above 0.75, the rest spread out, with the max norm so that the normalised
    values cover [0, 1] and many land between the crowded levels; then uniform 2^b levels, dense near 1 only.
    Words, histogram and statistic against the oracle."""
    n = 1 << bits
    crowd = n - 2 - 6
    lv = np.concatenate([[0.0], np.float32([1e-3, 0.02, 0.3, 0.74]),
                         np.float32(0.75) + np.arange(1, crowd + 1, dtype=np.float32) * np.float32(2.0 ** -22),
                         np.float32([0.9, 0.99]), [1.0]]).astype(np.float32)
    assert lv.size == n and np.all(np.diff(lv) > 0)
    sizes = [5000, 70001]
    plan = lqm.Plan(sizes, bits, 0, 2, SEED + bits)
    plan.lq_set_levels(0, lv)                                  # layer 1 keeps the uniform levels
    g = torch.Generator(device="cuda").manual_seed(bits)
    grads = torch.rand((2, plan.padded_elems), generator=g, device="cuda") * 2 - 1
    near = np.float32(0.75) + np.float32(2.0 ** -22) * torch.rand(2000, generator=g, device="cuda") * crowd
    grads[:, 100:2100] = near                                  # values between the crowded levels
    grads[:, 0] = 1.0                                          # the max norm is exactly 1
    packed = plan.empty_packed(); norms = plan.empty_norms(); hist = plan.zero_hist()
    plan.lq_quantize_pack(grads, 3, packed, norms, hist=hist)
    model = oracle_model(orc, plan)
    model.levels[0] = lv
    ref = model.quantize(to_unpadded(plan, grads), 3, want_hist=True)
    assert np.array_equal(norms.cpu().numpy()[:, :plan.num_layers], ref["norms"])
    assert compare_messages(orc, plan, packed, ref) == (0, 0)
    assert np.array_equal(hist.cpu().numpy().view(np.uint32), ref["hist"])
    packed2 = plan.empty_packed(); norms2 = plan.empty_norms()
    plan.lq_quantize_pack(grads, 4, packed2, norms2, prev_packed=packed, prev_norms=norms)
    model.prev_decoded = ref["decoded"]
    ref2 = model.quantize(to_unpadded(plan, grads), 4)
    assert compare_messages(orc, plan, packed2, ref2) == (0, 0)
    sq, _ = plan.lq_get_statistics()
    assert _close(sq.numpy(), ref2["sq_diff"], 1e-12)


def test_argument_errors(lqm):
    with pytest.raises(lqm.LqError):
        lqm.Plan([10], 9, 2, 1, 0)
    with pytest.raises(lqm.LqError):
        lqm.Plan([10], 4, 17, 1, 0)
    with pytest.raises(lqm.LqError):
        lqm.Plan([10], 4, 2, 0, 0)
    plan = lqm.Plan([10], 2, 2, 1, 0)
    with pytest.raises(lqm.LqError):
        plan.lq_set_levels(0, [0.0, 0.5, 0.5, 1.0])
    with pytest.raises(lqm.LqError):
        plan.lq_set_levels(0, [0.0, 0.5, 1.0])
    with pytest.raises(lqm.LqError):
        plan.lq_set_levels(0, [0.1, 0.5, 0.7, 1.0])
    X = torch.zeros(plan.padded_elems, device="cuda")
    with pytest.raises(lqm.LqError):              # qoda_step before qoda_init
        plan.qoda_step(plan.empty_packed(), plan.empty_norms(), X, X.clone(), X.clone())
    empty = lqm.Plan([], 4, 2, 2, 0)
    assert empty.packed_words == 0
    # misaligned rows are refused before any kernel could fault on them
    big = torch.zeros(2 * plan.padded_elems + 8, device="cuda")
    packed, norms = plan.empty_packed(), plan.empty_norms()
    with pytest.raises(lqm.LqError, match="aligned"):
        plan.lq_quantize_pack(big[1: 1 + plan.padded_elems].view(1, -1), 1, packed, norms)
    with pytest.raises(lqm.LqError, match="aligned"):
        plan.qoda_init(big[: plan.padded_elems], big[plan.padded_elems + 1: 2 * plan.padded_elems + 1], X.clone())


def test_qoda_alternative_rates_multi_step(lqm, orc):
    """Eq. (Alt): eta and gamma from the running sums lambda (||gbar||^2) and mu (||X_s - X_{s+1}||^2), no
    previous message needed.  30 iterations on ragged layers against the oracle, state compared every step."""
    sizes = [3000, 100, 2049, 7]
    plan = lqm.Plan(sizes, [4, 3, 4, 2], 2, 5, SEED)
    plan.qoda_set_alt_rates(0.25)
    model = oracle_model(orc, plan)
    model.alt_qhat = 0.25
    X1 = _grads(plan, 6)[0].contiguous(); Y = torch.empty_like(X1); Xh = torch.empty_like(X1); X = torch.empty_like(X1)
    plan.qoda_init(X1, Y, Xh)
    model.qoda_init(to_unpadded(plan, X1))
    packed = plan.empty_packed(); norms = plan.empty_norms()
    for t in range(1, 31):
        grads = _grads(plan, 2000 + t, 0.3 / math.sqrt(t))
        plan.lq_quantize_pack(grads, t, packed, norms)
        plan.qoda_step(packed, norms, X1, Y, Xh, X)
        ref = model.quantize(to_unpadded(plan, grads), t)
        assert compare_messages(orc, plan, packed, ref) == (0, 0)
        model.qoda_step()
        tt, _, eta = plan.qoda_get_scalars()
        lam, mu, gamma = plan.qoda_get_alt_scalars()
        assert tt == t + 1 and eta == float(model.eta) and gamma == float(model.gamma)
        assert abs(lam - model.lam) <= 1e-12 * model.lam and abs(mu - model.mu) <= 1e-12 * max(model.mu, 1e-300)
        for got, want in [(Y, model.Y), (Xh, model.Xhalf), (X, model.X)]:
            assert _close(to_unpadded(plan, got), want, 1e-6)
    assert 0 < eta < gamma < 1
    with pytest.raises(lqm.LqError):
        plan.qoda_set_alt_rates(0.3)
    # back to the default schedule: a fresh init gives eta = gamma again
    plan.qoda_set_alt_rates(0.0)
    plan.qoda_init(X1, Y, Xh)
    plan.lq_quantize_pack(grads, 1, packed, norms)
    plan.qoda_step(packed, norms, X1, Y, Xh)
    _, _, eta = plan.qoda_get_scalars(); _, _, gamma = plan.qoda_get_alt_scalars()
    assert eta == gamma < 1


def test_code_length_accounting(lqm, orc):
    """Level-occurrence probabilities from the histograms and the counts of emitted level indices, against
    the oracle; and the two against each other: the emitted frequencies follow the probabilities."""
    from paper_2505_14371_b200 import workloads as W
    w = W.wgan_workload()
    sizes = [s // 8 for s in w.layer_sizes] + [0, 5]
    w.layer_sizes = sizes; w.scales = w.scales + [1.0, 1.0]
    bits = [3, 4, 2, 8, 3, 4, 5, 3, 1, 4, 4]
    K = 3
    plan = lqm.Plan(sizes, bits, 2, K, SEED)
    grads = W.make_gradients(w, plan.elem_offsets, plan.padded_elems, "cuda", workers=K)
    packed = plan.empty_packed(); norms = plan.empty_norms(); hist = plan.zero_hist()
    plan.lq_quantize_pack(grads, 1, packed, norms, hist=hist)
    plan.lq_fit_levels(hist, norms, K)                                        # fitted levels for the second message
    hist.zero_()
    plan.lq_quantize_pack(grads, 2, packed, norms, hist=hist)
    probs = torch.full((plan.num_layers, 256), -1.0, dtype=torch.float64, device="cuda")
    counts = torch.zeros((K, plan.num_layers, 256), dtype=torch.int32, device="cuda")
    plan.lq_level_probabilities(hist, norms, K, probs)
    plan.lq_symbol_counts(packed, counts)
    torch.cuda.synchronize()
    model = oracle_model(orc, plan)
    ref = model.quantize(to_unpadded(plan, grads), 2, want_hist=True)
    assert compare_messages(orc, plan, packed, ref) == (0, 0)
    off = np.concatenate([[0], np.cumsum(sizes)])
    P = probs.cpu().numpy(); Cn = counts.cpu().numpy()
    for m, (d, b) in enumerate(zip(sizes, bits)):
        n = 1 << b
        want = orc.level_probabilities(ref["hist"][:, m, :], ref["norms"][:, m], d, model.levels[m])
        assert np.allclose(P[m, :n], want, rtol=1e-12, atol=1e-15), m
        assert np.all(P[m, n:] == 0)
        for k in range(K):
            assert np.array_equal(Cn[k, m, :n], np.bincount(ref["idx"][k, off[m]:off[m + 1]], minlength=n)), (k, m)
        if d > 50000 and b <= 4:
            # frequencies of one message against the probabilities (weights differ per worker, so loosely)
            freq = Cn[:, m, :n].sum(axis=0) / (K * d)
            assert abs(want.sum() - 1.0) < 1e-9
            assert np.all(np.abs(freq - want) < 0.05 * want + 2e-3), m


@pytest.mark.parametrize("q", [2, 0, 1])
def test_global_norm_scope(lqm, orc, q):
    """One norm over the worker's whole vector (Section 3.1) with per-layer levels: norms, messages, statistic,
    aggregate and update against the oracle over three steps; a NaN zeroes that worker's whole message."""
    rng = np.random.default_rng(40 + q)
    sizes = [5000, 33, 12345, 0, 2048]
    bits = [4, 3, 2, 4, 3]
    plan = lqm.Plan(sizes, bits, q, 3, SEED)
    plan.lq_set_norm_scope("global")
    for m, b in enumerate(bits):
        if m % 2 == 0 and b > 1:
            plan.lq_set_levels(m, _random_levels(rng, 1 << b))
    model = oracle_model(orc, plan)
    model.norm_scope = "global"
    X1 = _grads(plan, 8)[0].contiguous(); Y = torch.empty_like(X1); Xh = torch.empty_like(X1)
    plan.qoda_init(X1, Y, Xh); model.qoda_init(to_unpadded(plan, X1))
    pk = [plan.empty_packed(), plan.empty_packed()]; nm = [plan.empty_norms(), plan.empty_norms()]
    scale = torch.tensor(np.repeat([1.0, 0.01, 0.1, 1.0, 3.0], [5024, 64, 12352, 0, 2048]), device="cuda", dtype=torch.float32)
    for t in range(1, 4):
        grads = _grads(plan, 300 + t, 0.1) * scale[None, : plan.padded_elems]
        c, p = t % 2, (t + 1) % 2
        plan.lq_quantize_pack(grads, t, pk[c], nm[c], prev_packed=None if t == 1 else pk[p],
                              prev_norms=None if t == 1 else nm[p])
        plan.qoda_step(pk[c], nm[c], X1, Y, Xh)
        ref = model.quantize(to_unpadded(plan, grads), t)
        got = nm[c].cpu().numpy()
        assert np.array_equal(got, ref["norms"]) and np.all(got == got[:, :1])
        assert compare_messages(orc, plan, pk[c], ref) == (0, 0)
        sq, _ = plan.lq_get_statistics()
        assert _close(sq.numpy(), ref["sq_diff"], 1e-12)
        model.qoda_step()
        assert _close(to_unpadded(plan, Xh), model.Xhalf, 1e-6)
    grads[1, plan.elem_offsets[2] + 17] = float("nan")
    plan.lq_quantize_pack(grads, 9, pk[0], nm[0])
    torch.cuda.synchronize()
    _, flags = plan.lq_get_statistics()
    assert flags[1].tolist() == [lqm.STATUS_NONFINITE] * 5 and int(flags[0].sum()) == 0 and int(flags[2].sum()) == 0
    assert bool((pk[0][1] == 0).all()) and bool((nm[0][1] == 0).all()) and bool((pk[0][0] != 0).any())


def test_fit_levels_shared_by_type(lqm, orc):
    """One sequence per type: layers 0, 2, 5 (4 bits) form one type, 1 and 3 (3 bits) another, 4 is alone.
    Levels against the oracle's shared fit, every member receives the same sequence, and a type whose members
    disagree on the code width is refused."""
    from paper_2505_14371_b200 import workloads as W
    sizes = [30000, 7000, 12345, 4096, 9000, 100]
    bits = [4, 3, 4, 3, 5, 4]
    types = [7, 2, 7, 2, 9, 7]
    K = 4
    w = W.Workload("typed", sizes, bits=4, q=2, num_workers=K, dist="student3",
                   scales=[1e-2, 1e-3, 3e-2, 1e-4, 1e-1, 1e-3], config_id=6)
    plan = lqm.Plan(sizes, bits, 2, K, SEED)
    grads = W.make_gradients(w, plan.elem_offsets, plan.padded_elems, "cuda")
    packed = plan.empty_packed(); norms = plan.empty_norms(); hist = plan.zero_hist()
    plan.lq_quantize_pack(grads, 1, packed, norms, hist=hist)
    plan.lq_fit_levels_shared(hist, norms, K, types)
    h = hist.cpu().numpy().view(np.uint32); n = norms.cpu().numpy()
    got = [np.array(plan.lq_get_levels(m), np.float32) for m in range(len(sizes))]
    for tid in sorted(set(types)):
        members = [m for m, t in enumerate(types) if t == tid]
        hs = np.stack([h[z, m] for z in range(K) for m in members])
        ns = np.float32([n[z, m] for z in range(K) for m in members])
        ds = [sizes[m] for z in range(K) for m in members]
        want = orc.fit_levels_shared(hs, ns, ds, 1 << bits[members[0]])
        for m in members:
            assert np.allclose(got[m], want, rtol=1e-6, atol=0), (tid, m)
            assert np.array_equal(got[m], got[members[0]])
    # the shared sequences are what the next message is encoded with
    model = oracle_model(orc, plan)
    plan.lq_quantize_pack(grads, 2, packed, norms)
    ref = model.quantize(to_unpadded(plan, grads), 2)
    assert compare_messages(orc, plan, packed, ref) == (0, 0)
    with pytest.raises(lqm.LqError):
        plan.lq_fit_levels_shared(hist, norms, K, [1, 1, 1, 1, 1, 1])


def test_update_with_and_without_the_zero_block_masks_agree():
    """qoda_step on the buffer the encoder wrote (all-zero blocks are skipped from the masks) against qoda_step on a
    copy of the message at another address (everything is read): identical iterates, also where no worker sent
    anything."""
    import paper_2505_14371_b200 as lqm
    lqm.load_library()
    sizes, K = [70000, 3000, 9000], 5
    outs = []
    for use_copy in (False, True):
        plan = lqm.Plan(sizes, [4, 2, 6], 2, K, 5)
        g = torch.Generator(device="cuda").manual_seed(8)
        X1 = torch.randn(plan.padded_elems, generator=g, device="cuda")
        Y = torch.empty_like(X1); Xh = torch.empty_like(X1); X = torch.zeros_like(X1); gbar = torch.zeros_like(X1)
        plan.qoda_init(X1, Y, Xh)
        pk = [plan.empty_packed(), plan.empty_packed()]; nm = [plan.empty_norms(), plan.empty_norms()]
        for t in (1, 2, 3):
            grads = torch.randn((K, plan.padded_elems), generator=g, device="cuda")
            grads[:, 2048:30000] = 0.0                      # blocks that are zero for every worker
            grads[1:, 30000:50000] = 0.0                    # blocks that only worker 0 fills
            grads[2, :] = 0.0                               # a worker that sends nothing at all
            c, p = t % 2, (t + 1) % 2
            plan.lq_quantize_pack(grads, t, pk[c], nm[c], prev_packed=pk[p] if t > 1 else None,
                                  prev_norms=nm[p] if t > 1 else None)
            msg = pk[c].clone() if use_copy else pk[c]
            plan.qoda_step(msg, nm[c], X1, Y, Xh, X, gbar)
        torch.cuda.synchronize()
        outs.append([x.cpu().numpy().copy() for x in (Y, Xh, X, gbar)])
    for a, b in zip(*outs):
        assert np.array_equal(a, b)
    assert not outs[0][3][2048:30000].any()                 # gbar is zero where nobody sent anything
