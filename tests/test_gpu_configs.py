"""GPU parity on the benchmark configurations themselves: the bilinear game tracked over 2000 QODA
iterations, the WGAN-shaped set element by element, the Transformer-XL-shaped set at full size on
sampled outputs (in the launch configuration the benchmark times), and points of the bandwidth sweep.

Tolerances as in test_gpu_parity.py: message words bit-exact apart from coordinates within 1e-6 of a
rounding threshold (fewer than 1e-6 of all coordinates), norms relative 1e-6, decoded / aggregated
values relative 1e-6, QODA iterates relative 1e-5.
"""
import math
import os

import numpy as np
import pytest
import torch

from helpers import compare_messages, oracle_model, to_unpadded

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lqm():
    import paper_2505_14371_b200 as pkg
    pkg.load_library()
    return pkg


def _rel(a, b):
    a = np.asarray(a, np.float64); b = np.asarray(b, np.float64)
    return float(np.max(np.abs(a - b), initial=0.0) / max(float(np.max(np.abs(b), initial=0.0)), 1e-300))


# ------------------------------------------------------------------------------ config 2
def test_config2_bilinear_game_2000_iterations(lqm, orc):
    """min_x max_y x'Ay, x, y in R^4096, 8 layers of 1024, K = 8 workers with N(0, 0.1^2) noise, 4-bit levels
    refitted every 100 steps.  Both sides evaluate the operator with the same routine (fp64 on the device,
    rounded to fp32) on their own iterate and add the same host-drawn noise, so the two trajectories can be
    compared step by step; the duality gap of the ergodic average must fall."""
    from paper_2505_14371_b200 import workloads as W
    w = W.bilinear_workload()
    n = 4096; D = 2 * n; K = w.num_workers; T = 2000
    A, z1 = W.bilinear_game(n)
    A64 = A.double().cuda()

    def operator(z32_dev):                     # F(z) = (A y, -A' x), fp64 arithmetic, fp32 result
        z = z32_dev.double()
        return torch.cat([A64 @ z[n:], -(A64.t() @ z[:n])]).float()

    plan = lqm.Plan(w.layer_sizes, w.bits, w.q, K, W.PHILOX_SEED)
    assert plan.padded_elems == D
    model = oracle_model(orc, plan)
    X1 = z1.cuda().contiguous(); Y = torch.empty_like(X1); Xh = torch.empty_like(X1)
    avg_gpu = torch.ones(D, dtype=torch.float64, device="cuda")          # the library's running sum of X_{t+1/2}
    plan.qoda_set_average(avg_gpu)
    plan.qoda_init(X1, Y, Xh)
    model.qoda_init(z1.numpy())
    pk = [plan.empty_packed(), plan.empty_packed()]; nm = [plan.empty_norms(), plan.empty_norms()]
    R = float(np.linalg.norm(z1.numpy().astype(np.float64)))
    avg_orc = np.zeros(D)
    gaps = {}; near = 0; first_bad = None
    for t in range(1, T + 1):
        noise = W.bilinear_noise(t, K, D)                                   # host-drawn, shared by both sides
        avg_orc += model.Xhalf
        V_gpu = (operator(Xh)[None, :] + noise.cuda()).contiguous()
        F_orc = operator(torch.from_numpy(model.Xhalf).cuda()).cpu().numpy()
        V_orc = F_orc[None, :] + noise.numpy()
        c, p = t % 2, (t + 1) % 2
        fit_now = t % 100 == 0
        hist = plan.zero_hist() if fit_now else None
        plan.lq_quantize_pack(V_gpu, t, pk[c], nm[c], hist=hist, prev_packed=None if t == 1 else pk[p],
                              prev_norms=None if t == 1 else nm[p])
        plan.qoda_step(pk[c], nm[c], X1, Y, Xh)
        ref = model.quantize(V_orc, t, want_hist=fit_now)
        near += ref["near"]
        bad, stray = compare_messages(orc, plan, pk[c], ref)
        if (bad or stray) and first_bad is None:
            first_bad = (t, bad, stray)
        model.qoda_step()
        if fit_now:                                                          # Algorithm 1 lines 2-7
            plan.lq_fit_levels(hist, nm[c], K)
            h = hist.cpu().numpy().view(np.uint32)
            assert np.array_equal(h, ref["hist"])
            for m in range(plan.num_layers):
                got = np.array(plan.lq_get_levels(m), np.float32)
                want = orc.fit_levels(h[:, m, :], ref["norms"][:, m], w.layer_sizes[m], 1 << w.bits)
                assert np.allclose(got, want, rtol=1e-6, atol=0), (t, m)
                model.levels[m] = got                                        # both sides continue with one table
        if t in (10, 100, 1000, 2000):
            gaps[t] = R * float(torch.linalg.norm(operator((avg_gpu / t).float()).double()))
        if t % 250 == 0 or t == T:
            tt, S, eta = plan.qoda_get_scalars()
            assert tt == t + 1 and abs(S - model.S) <= 1e-9 * model.S and abs(eta - float(model.eta)) <= 1e-6 * eta
            assert _rel(Xh.cpu().numpy(), model.Xhalf) <= 1e-5, t
            assert _rel(Y.cpu().numpy(), model.Y) <= 1e-5, t
    assert first_bad is None, f"first differing message at (step, coords, words) = {first_bad}"
    assert near < 1e-5 * K * D * T
    assert _rel((avg_gpu / T).cpu().numpy(), avg_orc / T) <= 1e-5
    assert np.array_equal(avg_orc, model.xsum)
    assert gaps[2000] < 0.5 * gaps[100] and gaps[100] < gaps[10]


# ------------------------------------------------------------------------------ config 3
def test_config3_wgan_full_size_element_by_element(lqm, orc):
    """All 6 320 128 coordinates x K = 8 of the WGAN-shaped set with fitted 3-bit levels: messages, norms,
    statistic, aggregate and one QODA update against the oracle, element by element."""
    from paper_2505_14371_b200 import workloads as W
    w = W.wgan_workload()
    K = w.num_workers
    plan = lqm.Plan(w.layer_sizes, w.bits, w.q, K, W.PHILOX_SEED)
    grads = W.make_gradients(w, plan.elem_offsets, plan.padded_elems, "cuda")
    pk = [plan.empty_packed(), plan.empty_packed()]; nm = [plan.empty_norms(), plan.empty_norms()]
    hist = plan.zero_hist()
    g = torch.Generator(device="cuda").manual_seed(5)
    X1 = torch.randn(plan.padded_elems, generator=g, device="cuda") * 0.01
    Y = torch.empty_like(X1); Xh = torch.empty_like(X1); gbar = torch.empty_like(X1)
    plan.qoda_init(X1, Y, Xh)
    plan.lq_quantize_pack(grads, 1, pk[1], nm[1], hist=hist)                 # step 1: uniform levels + histogram
    plan.lq_fit_levels(hist, nm[1], K)
    plan.qoda_step(pk[1], nm[1], X1, Y, Xh)
    grads2 = grads * 0.5 + torch.roll(grads, 1, dims=0) * 0.5                # step 2: another input, fitted levels
    plan.lq_quantize_pack(grads2, 2, pk[0], nm[0], prev_packed=pk[1], prev_norms=nm[1])
    plan.qoda_step(pk[0], nm[0], X1, Y, Xh, None, gbar)
    torch.cuda.synchronize()

    model = oracle_model(orc, plan)                                          # holds the fitted levels
    fitted = [lv.copy() for lv in model.levels]
    for m in range(plan.num_layers):
        model.levels[m] = orc.uniform_levels(w.bits)
    model.qoda_init(to_unpadded(plan, X1))
    ref1 = model.quantize(to_unpadded(plan, grads), 1, want_hist=True)
    assert compare_messages(orc, plan, pk[1], ref1) == (0, 0)
    assert np.array_equal(hist.cpu().numpy().view(np.uint32), ref1["hist"])
    model.qoda_step()
    for m in range(plan.num_layers):
        want = orc.fit_levels(ref1["hist"][:, m, :], ref1["norms"][:, m], w.layer_sizes[m], 1 << w.bits)
        assert np.allclose(fitted[m], want, rtol=1e-6, atol=0), m
        model.levels[m] = fitted[m]
    ref2 = model.quantize(to_unpadded(plan, grads2), 2)
    total = K * w.num_coords
    bad, stray = compare_messages(orc, plan, pk[0], ref2)
    assert stray == 0 and bad <= 1e-6 * total and ref2["near"] < 1e-5 * total
    assert _rel(nm[0].cpu().numpy(), ref2["norms"]) <= 1e-6
    sq, _ = plan.lq_get_statistics()
    assert _rel(sq.numpy(), ref2["sq_diff"]) <= 1e-9
    gref = model.qoda_step()
    if bad == 0:
        off = np.concatenate([[0], np.cumsum(w.layer_sizes)])
        for name, got, want in [("gbar", gbar, gref), ("Y", Y, model.Y), ("Xhalf", Xh, model.Xhalf)]:
            gg = to_unpadded(plan, got)
            for m in range(plan.num_layers):
                assert _rel(gg[off[m]:off[m + 1]], want[off[m]:off[m + 1]]) <= 1e-6, (name, m)
    t, S, eta = plan.qoda_get_scalars()
    assert t == 3 and abs(S - model.S) <= 1e-9 * model.S and abs(eta - float(model.eta)) <= 1e-6 * eta


def test_low_rank_factor_shapes_two_iterations(lqm, orc):
    """The rank-16 factor shapes of the Section 7.2 model (2 blocks, 8192-row embedding: 37 layers from 410 to
    131 072 coordinates, zero rows 16 values long): two iterations against the oracle, everything bit-exact."""
    from paper_2505_14371_b200 import workloads as W
    w = W.powersgd_factor_workload(rank=16, num_blocks=2, vocab=8192)
    K = w.num_workers
    plan = lqm.Plan(w.layer_sizes, w.bits, w.q, K, W.PHILOX_SEED)
    grads = W.make_gradients(w, plan.elem_offsets, plan.padded_elems, "cuda")
    model = oracle_model(orc, plan)
    X1 = torch.zeros(plan.padded_elems, device="cuda"); Y = torch.empty_like(X1); Xh = torch.empty_like(X1)
    gbar = torch.empty_like(X1)
    plan.qoda_init(X1, Y, Xh); model.qoda_init(to_unpadded(plan, X1))
    pk = [plan.empty_packed(), plan.empty_packed()]; nm = [plan.empty_norms(), plan.empty_norms()]
    for t in (1, 2):
        c, p = t % 2, (t + 1) % 2
        gt = grads if t == 1 else torch.roll(grads, 1, dims=0) * 0.7
        plan.lq_quantize_pack(gt, t, pk[c], nm[c], prev_packed=pk[p] if t > 1 else None,
                              prev_norms=nm[p] if t > 1 else None)
        plan.qoda_step(pk[c], nm[c], X1, Y, Xh, None, gbar)
        ref = model.quantize(to_unpadded(plan, gt), t)
        assert compare_messages(orc, plan, pk[c], ref) == (0, 0)
        assert np.array_equal(nm[c].cpu().numpy()[:, :plan.num_layers], ref["norms"])
        assert np.array_equal(to_unpadded(plan, gbar), model.qoda_step())
        assert _rel(to_unpadded(plan, Y), model.Y) <= 1e-6 and _rel(to_unpadded(plan, Xh), model.Xhalf) <= 1e-6


# ------------------------------------------------------------------------------ config 4
def test_config4_transformer_xl_full_size_sampled(lqm, orc):
    """The benchmark's workload and launch configuration (150 870 550 coordinates x K = 8, 4 bits): sampled
    layers' norms and statistic, and sampled blocks' symbols, aggregate and update, each computed by the oracle
    one by one; plus properties that hold at any size."""
    from paper_2505_14371_b200 import workloads as W
    if torch.cuda.mem_get_info()[0] < 20e9:
        pytest.skip("needs about 12 GB of free device memory")
    w = W.transformer_xl_workload()
    K, Lr = w.num_workers, w.num_layers
    plan = lqm.Plan(w.layer_sizes, w.bits, w.q, K, W.PHILOX_SEED)
    grads = W.make_gradients(w, plan.elem_offsets, plan.padded_elems, "cuda")
    pk = [plan.empty_packed(), plan.empty_packed()]; nm = [plan.empty_norms(), plan.empty_norms()]
    g = torch.Generator(device="cuda").manual_seed(W.SEED_BASE + 99)
    X1 = torch.randn(plan.padded_elems, generator=g, device="cuda")
    Y = torch.empty_like(X1); Xh = torch.empty_like(X1); gbar = torch.empty_like(X1)
    plan.qoda_init(X1, Y, Xh)
    hist = plan.zero_hist()
    plan.lq_quantize_pack(grads, 1, pk[1], nm[1], hist=hist)                 # as bench.py: fit once, then steady steps
    plan.lq_fit_levels(hist, nm[1], K)
    plan.qoda_step(pk[1], nm[1], X1, Y, Xh)
    del hist
    Y_before = Y.clone()
    plan.lq_quantize_pack(grads, 2, pk[0], nm[0], prev_packed=pk[1], prev_norms=nm[1])
    plan.qoda_step(pk[0], nm[0], X1, Y, Xh, None, gbar)
    torch.cuda.synchronize()
    t, S, eta = plan.qoda_get_scalars()
    sq, flags = plan.lq_get_statistics()
    assert t == 3 and int(flags.sum()) == 0 and 0 < eta <= 1
    levels = [np.array(plan.lq_get_levels(m), np.float32) for m in range(Lr)]
    norms = nm[0].cpu().numpy(); norms_prev = nm[1].cpu().numpy()
    uniform = orc.uniform_levels(w.bits)
    C = w.bits + 1
    rng = np.random.default_rng(7)

    # sampled (worker, layer): norms of whole layers, the embedding included
    for (k, m) in [(0, 0), (5, 0), (1, 1), (2, 7), (3, 8), (7, Lr - 1), (4, 100), (6, 213)]:
        v = grads[k, plan.elem_offsets[m]: plan.elem_offsets[m] + w.layer_sizes[m]].cpu().numpy()
        ref, st = orc.layer_norm(v, w.q)
        assert st == 0 and abs(float(norms[k, m]) - float(ref)) <= 1e-6 * float(ref), (k, m)

    # the oracle's own norm of every (worker, layer) whose blocks are sampled below: the GPU's must equal it, and
    # the oracle quantizes with its own (the input is the same in both iterations, hence so is the norm)
    oracle_norms = {}

    def oracle_norm(k, m):
        if (k, m) not in oracle_norms:
            v = grads[k, plan.elem_offsets[m]: plan.elem_offsets[m] + w.layer_sizes[m]].cpu().numpy()
            ref, st = orc.layer_norm(v, w.q)
            assert st == 0 and norms[k, m] == ref and norms_prev[k, m] == ref, (k, m)
            oracle_norms[(k, m)] = ref
        return oracle_norms[(k, m)]

    # sampled blocks: symbols of every worker, then the aggregate and the update, one block range at a time
    def check_blocks(m, b0, nb):
        d = w.layer_sizes[m]
        lo = b0 * 1024; hi = min(d, lo + nb * 1024)
        e0 = plan.elem_offsets[m]
        decoded = np.zeros((K, hi - lo), np.float32); sq_part = np.zeros(K)
        for k in range(K):
            v = grads[k, e0 + lo: e0 + hi].cpu().numpy()
            on = oracle_norm(k, m)
            idx, sg, _ = orc.quantize_layer(v, on, levels[m], W.PHILOX_SEED, 2, k, m, first_index=lo)
            wo = plan.word_offsets[m] + b0 * 32 * C
            words = pk[0][k, wo: wo + nb * 32 * C].cpu().numpy().view(np.uint32)
            gi, gs = orc.unpack_layer(words, hi - lo, w.bits)
            assert np.array_equal(gi, idx) and np.array_equal(gs, sg), (m, b0, k)
            decoded[k] = orc.decode_layer(idx, sg, on, levels[m])
            pidx, psg, _ = orc.quantize_layer(v, on, uniform, W.PHILOX_SEED, 1, k, m, first_index=lo)
            sq_part[k] = orc.sq_diff(decoded[k], orc.decode_layer(pidx, psg, on, uniform))
        want = orc.aggregate(decoded)
        assert np.array_equal(gbar[e0 + lo: e0 + hi].cpu().numpy(), want), (m, b0)
        y = Y_before[e0 + lo: e0 + hi].cpu().numpy().copy(); x1 = X1[e0 + lo: e0 + hi].cpu().numpy()
        xh = np.zeros_like(y)
        orc.qoda_update(want, x1, y, xh, None, np.float32(eta))
        assert _rel(Y[e0 + lo: e0 + hi].cpu().numpy(), y) <= 1e-6 and _rel(Xh[e0 + lo: e0 + hi].cpu().numpy(), xh) <= 1e-5
        return sq_part

    nblk0 = (w.layer_sizes[0] + 1023) // 1024
    for b0 in [0, 127, 128, int(rng.integers(0, nblk0 - 4)), int(rng.integers(0, nblk0 - 4)), nblk0 - 2]:
        check_blocks(0, b0, 2)                                               # embedding, its ragged last block included
    for m in [1, 3, 7, 9, 104, Lr - 2]:
        nb = (w.layer_sizes[m] + 1023) // 1024
        check_blocks(m, max(0, nb - 3), min(3, nb))
    # small layers whole: their statistic is the oracle's, term by term
    for m in [2, 11, 12, 13, 14, Lr - 1]:
        nb = (w.layer_sizes[m] + 1023) // 1024
        part = check_blocks(m, 0, nb)
        assert np.allclose(sq[:, m].numpy(), part, rtol=1e-9, atol=0), m

    # properties at any size: rows that are zero in all workers leave Y alone; untouched padding aside, every
    # output is finite; the step size follows from the statistic
    emb = slice(plan.elem_offsets[0], plan.elem_offsets[0] + w.layer_sizes[0])
    zero_all = (grads[:, emb] == 0).all(dim=0)
    assert zero_all.float().mean() > 0.3
    assert torch.equal(Y[emb][zero_all], Y_before[emb][zero_all]) and bool((gbar[emb][zero_all] == 0).all())
    assert bool(torch.isfinite(Xh).all()) and bool(torch.isfinite(Y).all())
    assert abs(eta - 1.0 / math.sqrt(1.0 + S)) <= 1e-6 * eta


def test_config4_transformer_xl_two_whole_workers(lqm, orc):
    """The same two iterations with the oracle run over two WHOLE workers of the full-size workload (the K workers'
    layers dealt to host threads; the C routines release the interpreter lock): every layer's norm, every word of
    their messages and every layer's term of the step-size statistic; then S and eta from the GPU's own terms."""
    from concurrent.futures import ThreadPoolExecutor
    from paper_2505_14371_b200 import workloads as W
    if torch.cuda.mem_get_info()[0] < 20e9:
        pytest.skip("needs about 12 GB of free device memory")
    w = W.transformer_xl_workload()
    K, Lr = w.num_workers, w.num_layers
    plan = lqm.Plan(w.layer_sizes, w.bits, w.q, K, W.PHILOX_SEED)
    grads = W.make_gradients(w, plan.elem_offsets, plan.padded_elems, "cuda")
    pk = [plan.empty_packed(), plan.empty_packed()]; nm = [plan.empty_norms(), plan.empty_norms()]
    X1 = torch.zeros(plan.padded_elems, device="cuda"); Y = torch.empty_like(X1); Xh = torch.empty_like(X1)
    plan.qoda_init(X1, Y, Xh)
    hist = plan.zero_hist()
    plan.lq_quantize_pack(grads, 1, pk[1], nm[1], hist=hist)
    plan.lq_fit_levels(hist, nm[1], K)
    plan.qoda_step(pk[1], nm[1], X1, Y, Xh)
    _, S1, _ = plan.qoda_get_scalars()
    plan.lq_quantize_pack(grads, 2, pk[0], nm[0], prev_packed=pk[1], prev_norms=nm[1])
    plan.qoda_step(pk[0], nm[0], X1, Y, Xh)
    torch.cuda.synchronize()
    _, S2, eta = plan.qoda_get_scalars()
    sq, _ = plan.lq_get_statistics()
    levels = [np.array(plan.lq_get_levels(m), np.float32) for m in range(Lr)]
    uniform = orc.uniform_levels(w.bits)
    norms = nm[0].cpu().numpy()
    workers = (0, 5)
    host = {k: grads[k].cpu().numpy() for k in workers}
    words = {k: pk[0][k].cpu().numpy().view(np.uint32) for k in workers}

    def one_layer(job):
        k, m = job
        d = w.layer_sizes[m]
        v = host[k][plan.elem_offsets[m]: plan.elem_offsets[m] + d]
        on, st = orc.layer_norm(v, w.q)
        idx, sg, _ = orc.quantize_layer(v, on, levels[m], W.PHILOX_SEED, 2, k, m)
        got = words[k][plan.word_offsets[m]: plan.word_offsets[m] + orc.packed_words(d, w.bits)]
        same = bool(np.array_equal(got, orc.pack_layer(idx, sg, w.bits)))
        pidx, psg, _ = orc.quantize_layer(v, on, uniform, W.PHILOX_SEED, 1, k, m)
        term = orc.sq_diff(orc.decode_layer(idx, sg, on, levels[m]), orc.decode_layer(pidx, psg, on, uniform))
        return k, m, st, on, same, term

    with ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 1)) as pool:
        results = list(pool.map(one_layer, [(k, m) for k in workers for m in range(Lr)]))
    for k, m, st, on, same, term in results:
        assert st == 0 and norms[k, m] == on, (k, m)
        assert same, (k, m)
        assert abs(float(sq[k, m]) - term) <= max(1e-12, 2.0 * w.layer_sizes[m] * 2.0 ** -53) * term, (k, m)
    # the running sum and the step size follow from the terms the GPU reports for all K workers
    delta = float(sq.numpy().astype(np.float64).sum()) / (K * K)
    assert abs((S2 - S1) - delta) <= 1e-12 * delta
    assert abs(eta - 1.0 / math.sqrt(1.0 + S2)) <= 1e-6 * eta


def test_config4_bucket_scope_full_size_sampled(lqm, orc):
    """The same workload in bucket scope (`bench.py --norm-scope bucket`): sampled blocks' bucket norms, symbols and
    aggregate against the oracle applied bucket by bucket; zero buckets carry norm 0 and leave Y alone."""
    from paper_2505_14371_b200 import workloads as W
    if torch.cuda.mem_get_info()[0] < 20e9:
        pytest.skip("needs about 12 GB of free device memory")
    w = W.transformer_xl_workload()
    K, Lr = w.num_workers, w.num_layers
    plan = lqm.Plan(w.layer_sizes, w.bits, w.q, K, W.PHILOX_SEED)
    plan.lq_set_norm_scope("bucket")
    grads = W.make_gradients(w, plan.elem_offsets, plan.padded_elems, "cuda")
    pk = [plan.empty_packed(), plan.empty_packed()]; nm = [plan.empty_norms(), plan.empty_norms()]
    X1 = torch.zeros(plan.padded_elems, device="cuda")
    Y = torch.empty_like(X1); Xh = torch.empty_like(X1); gbar = torch.empty_like(X1)
    plan.qoda_init(X1, Y, Xh)
    hist = plan.zero_hist()
    plan.lq_quantize_pack(grads, 1, pk[1], nm[1], hist=hist)
    plan.lq_fit_levels(hist, nm[1], K)
    plan.qoda_step(pk[1], nm[1], X1, Y, Xh)
    del hist
    Y_before = Y.clone()
    plan.lq_quantize_pack(grads, 2, pk[0], nm[0], prev_packed=pk[1], prev_norms=nm[1])
    plan.qoda_step(pk[0], nm[0], X1, Y, Xh, None, gbar)
    torch.cuda.synchronize()
    _, flags = plan.lq_get_statistics()
    assert int(flags.sum()) == 0
    levels = [np.array(plan.lq_get_levels(m), np.float32) for m in range(Lr)]
    C = w.bits + 1
    block_off = np.concatenate([[0], np.cumsum([(d + 1023) // 1024 for d in w.layer_sizes])])
    rng = np.random.default_rng(11)

    def check_blocks(m, b0, nb):
        d = w.layer_sizes[m]
        lo = b0 * 1024; hi = min(d, lo + nb * 1024)
        e0 = plan.elem_offsets[m]
        decoded = np.zeros((K, hi - lo), np.float32)
        for k in range(K):
            v = grads[k, e0 + lo: e0 + hi].cpu().numpy()
            got_bn = nm[0][k, 8 * (block_off[m] + b0): 8 * (block_off[m] + b0 + nb)].cpu().numpy()
            idx = np.zeros(hi - lo, np.uint8); sg = np.zeros(hi - lo, np.uint8)
            for i in range(0, hi - lo, 128):
                seg = v[i: i + 128]
                bn, _ = orc.layer_norm(seg, w.q)
                assert got_bn[i // 128] == bn, (m, b0, k, i)
                idx[i: i + 128], sg[i: i + 128], _ = orc.quantize_layer(seg, bn, levels[m], W.PHILOX_SEED, 2, k, m,
                                                                         first_index=lo + i)
                decoded[k, i: i + 128] = orc.decode_layer(idx[i: i + 128], sg[i: i + 128], bn, levels[m])
            assert not got_bn[(hi - lo + 127) // 128:].any()                 # rows past the layer's end
            wo = plan.word_offsets[m] + b0 * 32 * C
            words = pk[0][k, wo: wo + nb * 32 * C].cpu().numpy().view(np.uint32)
            gi, gs = orc.unpack_layer(words, hi - lo, w.bits)
            assert np.array_equal(gi, idx) and np.array_equal(gs, sg), (m, b0, k)
        assert np.array_equal(gbar[e0 + lo: e0 + hi].cpu().numpy(), orc.aggregate(decoded)), (m, b0)

    nblk0 = (w.layer_sizes[0] + 1023) // 1024
    for b0 in [0, 127, int(rng.integers(0, nblk0 - 4)), nblk0 - 2]:
        check_blocks(0, b0, 2)
    for m in [1, 7, 12, 104, Lr - 1]:
        nb = (w.layer_sizes[m] + 1023) // 1024
        check_blocks(m, max(0, nb - 2), min(2, nb))
    emb = slice(plan.elem_offsets[0], plan.elem_offsets[0] + w.layer_sizes[0])
    zero_all = (grads[:, emb] == 0).all(dim=0)
    assert torch.equal(Y[emb][zero_all], Y_before[emb][zero_all]) and bool((gbar[emb][zero_all] == 0).all())
    assert bool(torch.isfinite(Xh).all()) and bool(torch.isfinite(Y).all())


# ------------------------------------------------------------------------------ config 5
@pytest.mark.parametrize("bits", [2, 3, 4, 8])
@pytest.mark.parametrize("K", [1, 4, 16])
@pytest.mark.parametrize("q", [2, 0])
def test_config5_sweep_points(lqm, orc, bits, K, q):
    """Points of the bandwidth sweep at a size the oracle finishes quickly: a flat N(0,1) layer and a ragged
    set of layers with sizes log-uniform in [64, 40000], uniform levels."""
    from paper_2505_14371_b200 import workloads as W
    for w in (W.flat_workload(15, bits, K, q), W.ragged_workload(bits, K, q, num_layers=24, lo=64, hi=40000)):
        plan = lqm.Plan(w.layer_sizes, w.bits, w.q, K, W.PHILOX_SEED + bits)
        grads = W.make_gradients(w, plan.elem_offsets, plan.padded_elems, "cuda")
        packed = plan.empty_packed(); norms = plan.empty_norms()
        gbar = torch.empty(plan.padded_elems, device="cuda")
        plan.lq_quantize_pack(grads, 3, packed, norms)
        plan.lq_decode_aggregate(packed, norms, gbar)
        model = oracle_model(orc, plan)
        ref = model.quantize(to_unpadded(plan, grads), 3)
        assert compare_messages(orc, plan, packed, ref) == (0, 0)
        assert np.array_equal(norms.cpu().numpy()[:, :plan.num_layers], ref["norms"])
        assert np.array_equal(to_unpadded(plan, gbar), model.mean_decoded(ref["decoded"]))


# --------------------------------------------------------------------------- maximum size
def test_largest_layer_sampled(lqm, orc):
    """One layer of 2^31 - 5 coordinates (the plan's limit is 2^31 - 1): byte offsets pass 2^33 and the
    Philox counter word index/4 passes 2^28.  Sampled blocks - the first, two in the middle, the ragged last -
    against the oracle; the norm against a library fp64 norm."""
    if torch.cuda.mem_get_info()[0] < 40e9:
        pytest.skip("needs about 25 GB of free device memory")
    d = (1 << 31) - 5
    plan = lqm.Plan([d], 3, 2, 1, SEED_BIG)
    assert plan.padded_elems == (1 << 31)
    grads = torch.empty((1, plan.padded_elems), device="cuda")
    g = torch.Generator(device="cuda").manual_seed(2031)
    for s in range(0, plan.padded_elems, 1 << 28):
        grads[0, s: s + (1 << 28)].normal_(generator=g)
    grads[0, 5 << 20: 9 << 20] = 0.0                                          # a run of all-zero rows and blocks
    packed = plan.empty_packed(); norms = plan.empty_norms()
    gbar = torch.empty(plan.padded_elems, device="cuda")
    plan.lq_quantize_pack(grads, 9, packed, norms)
    plan.lq_decode_aggregate(packed, norms, gbar)
    torch.cuda.synchronize()
    ref_norm = float(torch.linalg.vector_norm(grads[0, :d].double()))
    N = float(norms[0, 0])
    assert abs(N - ref_norm) <= 1e-6 * ref_norm
    levels = np.array(plan.lq_get_levels(0), np.float32)
    nblk = (d + 1023) // 1024
    C = 4
    for b0 in [0, (6 << 20) // 1024, nblk // 2 + 1, (3 << 29) // 1024 + 7, nblk - 2]:                 # coordinate 3 * 2^29 is byte 6 * 2^30
        lo = b0 * 1024; hi = min(d, lo + 2048)
        v = grads[0, lo:hi].cpu().numpy()
        idx, sg, _ = orc.quantize_layer(v, np.float32(N), levels, SEED_BIG, 9, 0, 0, first_index=lo)
        words = packed[0, b0 * 32 * C: (b0 + 2) * 32 * C].cpu().numpy().view(np.uint32)
        gi, gs = orc.unpack_layer(words, hi - lo, 3)
        assert np.array_equal(gi, idx) and np.array_equal(gs, sg), b0
        assert np.array_equal(gbar[lo:hi].cpu().numpy(), orc.decode_layer(idx, sg, np.float32(N), levels)), b0
    assert bool((packed[0, (5 << 20) // 1024 * 32 * C: (9 << 20) // 1024 * 32 * C] == 0).all())


SEED_BIG = 0x0123456789ABCDEF
