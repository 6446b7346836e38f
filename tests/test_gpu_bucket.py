"""Bucket scope (one norm per 128 consecutive coordinates of a layer, the setting of Section 7.1) against the
oracle applied bucket by bucket: bucket norms, messages, flags, histogram, statistic, aggregate, state, refit."""
import numpy as np
import pytest
import torch

from helpers import bucket_norms_by_layer, compare_messages, oracle_model, to_unpadded

pytestmark = pytest.mark.gpu


def _close(a, b, rel):
    a = np.asarray(a, np.float64); b = np.asarray(b, np.float64)
    return np.max(np.abs(a - b), initial=0.0) <= rel * max(np.max(np.abs(b), initial=0.0), 1e-300)


def _random_levels(rng, n):
    inner = np.sort(1.0 - rng.uniform(0, 0.02, n - 2)) if rng.random() < 0.5 else np.sort(rng.uniform(0, 1, n - 2) ** 3)
    lv = np.concatenate([[0.0], inner, [1.0]]).astype(np.float32)
    for j in range(1, n - 1):
        if lv[j] <= lv[j - 1]:
            lv[j] = np.nextafter(lv[j - 1], np.float32(2.0))
    for j in range(n - 2, 0, -1):
        if lv[j] >= lv[j + 1]:
            lv[j] = np.nextafter(lv[j + 1], np.float32(-1.0))
    return lv


def _run(orc, sizes, bits, K, q, seed, steps=3, alt=0.0, hist_steps=(1,), special=True, random_levels=False):
    import paper_2505_14371_b200 as lqm
    lqm.load_library()
    rng = np.random.default_rng(seed)
    plan = lqm.Plan(sizes, bits, q, K, 1234 + seed)
    L = plan.num_layers
    plan.lq_set_norm_scope("bucket")
    assert plan.lq_plan_norm_count() == 8 * sum((d + 1023) // 1024 for d in sizes)
    if alt:
        plan.qoda_set_alt_rates(alt)
    model = oracle_model(orc, plan)
    model.norm_scope = "bucket"; model.alt_qhat = alt
    g = torch.Generator(device="cuda").manual_seed(seed)
    X1 = (torch.randn(plan.padded_elems, generator=g, device="cuda") * 0.1).contiguous()
    Y = torch.empty_like(X1); Xh = torch.empty_like(X1); X = torch.empty_like(X1); gbar = torch.empty_like(X1)
    plan.qoda_init(X1, Y, Xh); model.qoda_init(to_unpadded(plan, X1))
    pk = [plan.empty_packed(), plan.empty_packed()]; nm = [plan.empty_norms(), plan.empty_norms()]
    off = plan.elem_offsets
    for t in range(1, steps + 1):
        grads = torch.randn((K, plan.padded_elems), generator=g, device="cuda") * float(10.0 ** rng.uniform(-4, 1))
        grads = grads * (1.0 + 5.0 * torch.rand((K, plan.padded_elems), generator=g, device="cuda") ** 8)
        if special:
            for _ in range(3):                                   # runs of zeros: whole buckets and parts of buckets
                k = int(rng.integers(0, K)); a = int(rng.integers(0, plan.padded_elems)); n = int(rng.integers(1, 3000))
                grads[k, a: a + n] *= 0.0 if rng.random() < 0.5 else -0.0
            if t == 2 and sizes[0] > 300:                        # one bucket with NaN, one with Inf, one denormal-only
                grads[0, off[0] + 130] = float("nan")
                grads[K - 1, off[0] + 260] = float("-inf")
                grads[0, off[0]: off[0] + 128] = 1e-42
        if random_levels and t >= 2:                             # also level sets denser than the search bins
            for m in range(L):
                if plan.bits[m] > 1:
                    lv = _random_levels(rng, 1 << plan.bits[m])
                    plan.lq_set_levels(m, lv); model.levels[m] = lv
        use_hist = t in hist_steps
        hist = plan.zero_hist() if use_hist else None
        c, p = t % 2, (t + 1) % 2
        plan.lq_quantize_pack(grads, t, pk[c], nm[c], hist=hist, prev_packed=pk[p] if t > 1 else None,
                              prev_norms=nm[p] if t > 1 else None)
        plan.qoda_step(pk[c], nm[c], X1, Y, Xh, X, gbar)
        ref = model.quantize(to_unpadded(plan, grads), t, want_hist=use_hist)
        tag = (seed, t)
        got_bn, stray = bucket_norms_by_layer(plan, nm[c])
        assert stray == 0.0, tag
        for m in range(L):
            want = np.stack([ref["bucket_norms"][k][m] for k in range(K)]) if sizes[m] else np.zeros((K, 0), np.float32)
            assert np.array_equal(got_bn[m], want), (tag, m)
        assert compare_messages(orc, plan, pk[c], ref) == (0, 0), tag
        sq, flags = plan.lq_get_statistics()
        assert np.array_equal(flags.numpy(), ref["status"]), tag
        assert _close(plan.lq_layer_weights().numpy(), ref["norms"], 1e-6), tag
        if use_hist:
            assert np.array_equal(hist.cpu().numpy().view(np.uint32)[:, :L], ref["hist"]), tag
        if not alt:
            assert _close(sq.numpy(), ref["sq_diff"], max(1e-12, 2.0 * K * sum(sizes) * 2.0 ** -53)), tag
        gref = model.qoda_step()
        assert np.array_equal(to_unpadded(plan, gbar), gref), tag
        tt, S, eta = plan.qoda_get_scalars()
        assert tt == t + 1 and eta == float(model.eta), tag
        for got, want in [(Y, model.Y), (Xh, model.Xhalf), (X, model.X)]:
            assert _close(to_unpadded(plan, got), want, 1e-6), tag
        dec = torch.empty_like(X1)
        plan.lq_decode_aggregate(pk[c], nm[c], dec)
        assert np.array_equal(to_unpadded(plan, dec), gref), tag
        if use_hist:                                             # refit with the layers' energies as weights
            plan.lq_fit_levels(hist, nm[c], K)
            for m in range(L):
                n_lv = 1 << plan.bits[m]
                if n_lv >= 3 and sizes[m]:
                    want = orc.fit_levels(ref["hist"][:, m, :], ref["norms"][:, m], sizes[m], n_lv)
                    got = np.array(plan.lq_get_levels(m), np.float32)
                    if want is not None:
                        assert np.allclose(got, want, rtol=1e-6, atol=0), (tag, m)
                    model.levels[m] = got
    return plan


@pytest.mark.parametrize("q", [2, 0, 1, 3])
def test_bucket_scope_small_layers(orc, q):
    _run(orc, [5000, 127, 128, 129, 1, 0, 2049, 40000], [4, 3, 2, 1, 5, 3, 8, 4], K=3, q=q, seed=10 + q)


def test_bucket_scope_many_workers_and_tiles(orc):
    _run(orc, [300000, 70000], [4, 2], K=9, q=2, seed=21, steps=2)


def test_bucket_scope_random_level_tables(orc):
    _run(orc, [20000, 3000, 1500], [5, 3, 8], K=2, q=2, seed=31, steps=4, hist_steps=(), random_levels=True)


def test_bucket_scope_alt_rates(orc):
    _run(orc, [33000, 1000], [3, 4], K=4, q=2, seed=22, alt=0.25)


def test_bucket_scope_rules(orc):
    import paper_2505_14371_b200 as lqm
    plan = _run(orc, [4096], [4], K=2, q=2, seed=23, steps=1, special=False)
    with pytest.raises(lqm.LqError):
        plan.lq_set_norm_scope("layer")                          # a message exists: the scope is fixed
    with pytest.raises(lqm.LqError):
        plan.lq_layer_norms(torch.zeros((2, plan.padded_elems), device="cuda"), plan.empty_norms())
    other = lqm.Plan([4096], 4, 2, 2, 1)
    with pytest.raises(lqm.LqError):
        other.lq_layer_weights()
