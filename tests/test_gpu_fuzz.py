"""Randomised differential test: random plans and inputs, several QODA iterations each, every output of the
CUDA path compared with the oracle (messages and norms bit-exact, statistic, aggregate and state within the
tolerances of test_gpu_parity.py).  Seeds are fixed: a failure names the case that reproduces it."""
import os

import numpy as np
import pytest
import torch

from helpers import compare_messages, oracle_model, to_unpadded

pytestmark = pytest.mark.gpu


def _close(a, b, rel):
    a = np.asarray(a, np.float64); b = np.asarray(b, np.float64)
    return np.max(np.abs(a - b), initial=0.0) <= rel * max(np.max(np.abs(b), initial=0.0), 1e-300)


def _levels(rng, n):
    if rng.random() < 0.3:                                       # sometimes denser than the search bins: slow path
        inner = np.sort(1.0 - rng.uniform(0, 0.02, n - 2))
    else:
        inner = np.sort(rng.uniform(0.0, 1.0, n - 2) ** rng.integers(1, 6))
    lv = np.concatenate([[0.0], inner, [1.0]]).astype(np.float32)
    for j in range(1, n - 1):
        if lv[j] <= lv[j - 1]:
            lv[j] = np.nextafter(lv[j - 1], np.float32(2.0))
    for j in range(n - 2, 0, -1):
        if lv[j] >= lv[j + 1]:
            lv[j] = np.nextafter(lv[j + 1], np.float32(-1.0))
    return lv


# LQ_FUZZ_CASES=n in the environment runs the first n random plans instead of 24
@pytest.mark.parametrize("case", range(int(os.environ.get("LQ_FUZZ_CASES", "24"))))
def test_random_plan_against_the_oracle(orc, case):
    import paper_2505_14371_b200 as lqm
    lqm.load_library()
    rng = np.random.default_rng(1000 + case)
    L = int(rng.integers(1, 7))
    sizes = [int(x) for x in rng.choice([0, 1, 5, 31, 32, 127, 128, 129, 1000, 1024, 1025, 3000, 5000, 9000, 33000], L)]
    if sum(sizes) == 0:
        sizes[0] = 777
    bits = [int(b) for b in rng.integers(1, 9, L)]
    K = int(rng.choice([1, 2, 3, 8, 9]))
    q = int(rng.choice([2, 2, 0, 1, 3]))
    scope = "global" if rng.random() < 0.3 else "layer"
    alt = float(rng.choice([0.0, 0.0, 0.25, 0.1]))
    plan = lqm.Plan(sizes, bits, q, K, int(rng.integers(0, 2 ** 63)))
    plan.lq_set_norm_scope(scope)
    if alt:
        plan.qoda_set_alt_rates(alt)
    model = oracle_model(orc, plan)
    model.norm_scope = scope; model.alt_qhat = alt
    g = torch.Generator(device="cuda").manual_seed(case)
    X1 = (torch.randn(plan.padded_elems, generator=g, device="cuda") * 0.1).contiguous()
    Y = torch.empty_like(X1); Xh = torch.empty_like(X1); X = torch.empty_like(X1); gbar = torch.empty_like(X1)
    xsum = torch.full((plan.padded_elems,), 7.0, dtype=torch.float64, device="cuda")
    plan.qoda_set_average(xsum)                                  # zeroed here and again by qoda_init
    plan.qoda_init(X1, Y, Xh); model.qoda_init(to_unpadded(plan, X1))
    pk = [plan.empty_packed(), plan.empty_packed()]; nm = [plan.empty_norms(), plan.empty_norms()]
    off = plan.elem_offsets
    # fp64 sums of up to D * K non-negative terms in two different orders: the oracle adds them one after the other,
    # which can lose up to one rounding of the running total per term
    sum_tol = max(1e-12, 2.0 * K * sum(sizes) * 2.0 ** -53)
    for t in range(1, 6):
        if rng.random() < 0.4:                                   # new level tables for some layers
            for m in range(L):
                if bits[m] > 1 and rng.random() < 0.5:
                    lv = _levels(rng, 1 << bits[m])
                    plan.lq_set_levels(m, lv); model.levels[m] = lv
        scale = float(10.0 ** rng.uniform(-6, 2))
        grads = torch.randn((K, plan.padded_elems), generator=g, device="cuda") * scale
        if rng.random() < 0.5:
            grads = grads ** 3
        for _ in range(int(rng.integers(0, 4))):                 # runs of zeros of either sign, any alignment
            k = int(rng.integers(0, K)); a = int(rng.integers(0, plan.padded_elems)); n = int(rng.integers(1, 6000))
            grads[k, a: a + n] *= 0.0 if rng.random() < 0.5 else -0.0
        if rng.random() < 0.15 and L > 1:                        # a NaN or Inf somewhere
            k = int(rng.integers(0, K)); m = int(rng.integers(0, L))
            if sizes[m]:
                grads[k, off[m] + int(rng.integers(0, sizes[m]))] = float(rng.choice([np.nan, np.inf, -np.inf]))
        use_hist = rng.random() < 0.4
        hist = plan.zero_hist() if use_hist else None
        c, p = t % 2, (t + 1) % 2
        use_prev = t > 1 and (alt == 0.0 or rng.random() < 0.5)
        plan.lq_quantize_pack(grads, t, pk[c], nm[c], hist=hist, prev_packed=pk[p] if use_prev else None,
                              prev_norms=nm[p] if use_prev else None)
        plan.qoda_step(pk[c], nm[c], X1, Y, Xh, X, gbar)
        if not use_prev:
            model.prev_decoded = None
        ref = model.quantize(to_unpadded(plan, grads), t, want_hist=use_hist)
        tag = (case, t)
        assert np.array_equal(nm[c].cpu().numpy()[:, :L], ref["norms"]), tag
        assert compare_messages(orc, plan, pk[c], ref) == (0, 0), tag
        _, flags = plan.lq_get_statistics()
        assert np.array_equal(flags.numpy(), ref["status"]), tag
        if use_hist:
            assert np.array_equal(hist.cpu().numpy().view(np.uint32)[:, :L], ref["hist"]), tag
        if alt == 0.0:
            sq, _ = plan.lq_get_statistics()
            assert _close(sq.numpy(), ref["sq_diff"], sum_tol), tag
        gref = model.qoda_step()
        assert np.array_equal(to_unpadded(plan, gbar), gref), tag
        tt, S, eta = plan.qoda_get_scalars()
        assert tt == t + 1 and eta == float(model.eta), tag
        if alt:
            lam, mu, gamma = plan.qoda_get_alt_scalars()
            assert gamma == float(model.gamma) and abs(lam - model.lam) <= sum_tol * max(model.lam, 1e-300), tag
        else:
            assert abs(S - model.S) <= sum_tol * max(model.S, 1e-300), tag
        for got, want in [(Y, model.Y), (Xh, model.Xhalf), (X, model.X)]:
            assert _close(to_unpadded(plan, got), want, 1e-6), tag
        assert _close(to_unpadded(plan, xsum), model.xsum, 1e-6), tag      # running sum of X_{s+1/2}, s <= t
        if use_hist and rng.random() < 0.7:                      # refit from this step's histograms
            plan.lq_fit_levels(hist, nm[c], K)
            h = ref["hist"]
            for m in range(L):
                n_lv = 1 << bits[m]
                want = orc.fit_levels(h[:, m, :], ref["norms"][:, m], sizes[m], n_lv) if n_lv >= 3 and sizes[m] else None
                got = np.array(plan.lq_get_levels(m), np.float32)
                if want is not None:
                    assert np.allclose(got, want, rtol=1e-6, atol=0), (tag, m)
                model.levels[m] = got
