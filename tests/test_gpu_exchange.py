"""The exchange path (one process per worker range, messages by all-gather) against one process holding all K
workers: bit-identical messages, iterates and step sizes.  The two ranks run as child processes on the same GPU
with the gloo backend: their kernels never wait on one another (the collectives run on the host)."""
import os
import socket
import subprocess
import sys

import numpy as np
import pytest

pytestmark = pytest.mark.gpu
HERE = os.path.dirname(os.path.abspath(__file__))


def _free_port() -> str:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return str(s.getsockname()[1])


@pytest.mark.parametrize("scope", ["layer", "bucket"])
def test_two_ranks_equal_one_process(tmp_path, scope):
    sys.path.insert(0, HERE)
    import exchange_rank
    want = exchange_rank.run(0, 1, scope, False)                  # all K workers in this process
    port = _free_port()
    procs = [subprocess.Popen([sys.executable, os.path.join(HERE, "exchange_rank.py"), str(r), "2", port,
                               str(tmp_path), scope], stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
             for r in range(2)]
    outs = []
    for p in procs:
        try:
            outs.append(p.communicate(timeout=300)[0])
        except subprocess.TimeoutExpired:
            p.kill()
            outs.append(p.communicate()[0])
    assert all(p.returncode == 0 for p in procs), "\n".join(outs)
    for r in range(2):
        got = np.load(tmp_path / f"rank{r}.npz")
        for key in want:
            assert np.array_equal(got[key], want[key]), (r, key)
    _check_against_oracle(dict(np.load(tmp_path / "rank0.npz")), scope)


def _check_against_oracle(got, scope):
    """Rank 0's final state against the CPU oracle run over the same three iterations (the fitted levels are taken
    from the GPU, as in the other parity tests: the level fit has its own test)."""
    import torch
    import exchange_rank as R
    import paper_2505_14371_b200 as lqm
    from oracle import oracle as orc
    from helpers import to_unpadded, bucket_norms_by_layer
    orc.build()
    plan = lqm.Plan(R.SIZES, R.BITS, R.Q, R.K, R.SEED)              # only for the padded layout
    plan.lq_set_norm_scope(scope)
    model = orc.OracleModel(R.SIZES, R.BITS, R.Q, R.K, R.SEED)
    model.norm_scope = scope
    g = torch.Generator(device="cuda").manual_seed(5)
    X1 = torch.randn(plan.padded_elems, generator=g, device="cuda") * 0.1
    model.qoda_init(to_unpadded(plan, X1))
    ref = None
    for t in (1, 2, 3):
        grads = torch.randn((R.K, plan.padded_elems), generator=g, device="cuda") * (0.5 ** t)
        grads[1, 100:700] = 0.0
        ref = model.quantize(to_unpadded(plan, grads), t)
        model.qoda_step()
        if t == 1:
            for m in range(len(R.SIZES)):
                model.levels[m] = got[f"levels{m}"]
    packed = got["packed"].view(np.uint32)
    for k in range(R.K):
        for m, (d, b) in enumerate(zip(R.SIZES, R.BITS)):
            words = packed[k, plan.word_offsets[m]: plan.word_offsets[m] + orc.packed_words(d, b)]
            assert np.array_equal(words, ref["packed"][k][m]), (k, m)
    if scope == "layer":
        assert np.array_equal(got["norms"][:, :len(R.SIZES)], ref["norms"])
    else:
        by_layer, stray = bucket_norms_by_layer(plan, torch.from_numpy(got["norms"]))
        assert stray == 0.0
        for m in range(len(R.SIZES)):
            for k in range(R.K):
                assert np.array_equal(by_layer[m][k], ref["bucket_norms"][k][m]), (k, m)
    tt, S, eta = got["scalars"]
    assert tt == 4 and abs(S - model.S) <= 1e-12 * model.S and eta == float(model.eta)

    def unpad(a):
        return np.concatenate([a[o:o + d] for o, d in zip(plan.elem_offsets, R.SIZES)])
    for key, want in (("Y", model.Y), ("Xh", model.Xhalf), ("X", model.X)):
        a = unpad(got[key])
        assert np.max(np.abs(a - want)) <= 1e-6 * np.max(np.abs(want)), key


def test_changing_the_range_restarts_the_message_stream():
    import torch
    import paper_2505_14371_b200 as lqm
    lqm.load_library()
    plan = lqm.Plan([5000], 4, 2, 4, 3)
    grads = torch.randn((4, plan.padded_elems), device="cuda")
    a, b = plan.empty_packed(), plan.empty_packed(); na, nb = plan.empty_norms(), plan.empty_norms()
    plan.lq_quantize_pack(grads, 1, a, na)
    plan.lq_set_worker_range(2, 2)
    with pytest.raises(lqm.LqError):
        plan.lq_quantize_pack(grads[2:4].contiguous(), 2, b, nb, prev_packed=a, prev_norms=na)
    b.copy_(a); nb.copy_(na)
    plan.lq_quantize_pack(grads[2:4].contiguous(), 1, b, nb)     # same step, same workers: the same rows come out
    torch.cuda.synchronize()
    assert torch.equal(a, b) and torch.equal(na, nb)
    plan.lq_quantize_pack(grads[2:4].contiguous(), 2, a, na, prev_packed=b, prev_norms=nb)   # the stream continues
    with pytest.raises(lqm.LqError):
        plan.lq_set_worker_range(3, 2)
