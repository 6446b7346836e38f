"""Two iterations recorded into a CUDA graph and replayed (lq_quantize_pack with LQ_STEP_AUTO + qoda_step) against
the same iterations issued call by call with explicit step numbers: bit-identical messages and iterates."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _setup(lqm, scope):
    plan = lqm.Plan([50000, 300, 4097, 128], [4, 3, 2, 5], 2, 4, 77)
    plan.lq_set_norm_scope(scope)
    g = torch.Generator(device="cuda").manual_seed(3)
    X1 = torch.randn(plan.padded_elems, generator=g, device="cuda") * 0.1
    Y = torch.empty_like(X1); Xh = torch.empty_like(X1)
    plan.qoda_init(X1, Y, Xh)
    pk = [plan.empty_packed(), plan.empty_packed()]; nm = [plan.empty_norms(), plan.empty_norms()]
    return plan, X1, Y, Xh, pk, nm


@pytest.mark.parametrize("scope", ["layer", "bucket"])
def test_graph_replay_equals_call_by_call(scope):
    import paper_2505_14371_b200 as lqm
    lqm.load_library()
    T = 8
    g = torch.Generator(device="cuda").manual_seed(11)
    probe = lqm.Plan([50000, 300, 4097, 128], [4, 3, 2, 5], 2, 4, 77)
    grads = [torch.randn((4, probe.padded_elems), generator=g, device="cuda") * (0.9 ** t) for t in range(T)]
    for t in range(T):
        grads[t][1, 1000:9000] = 0.0

    # call by call, explicit step numbers
    plan, X1, Y, Xh, pk, nm = _setup(lqm, scope)
    for t in range(1, T + 1):
        c, p = t % 2, (t + 1) % 2
        plan.lq_quantize_pack(grads[t - 1], t, pk[c], nm[c], prev_packed=pk[p] if t > 1 else None,
                              prev_norms=nm[p] if t > 1 else None)
        plan.qoda_step(pk[c], nm[c], X1, Y, Xh)
    torch.cuda.synchronize()
    want = [x.cpu().numpy().copy() for x in (Y, Xh, pk[0], pk[1], nm[0], nm[1])]
    want_scalars = plan.qoda_get_scalars()

    # two iterations call by call, then iterations 3-4 recorded once and replayed three times
    plan, X1, Y, Xh, pk, nm = _setup(lqm, scope)
    gin = [torch.empty_like(grads[0]), torch.empty_like(grads[0])]
    for t in (1, 2):
        c, p = t % 2, (t + 1) % 2
        plan.lq_quantize_pack(grads[t - 1], lqm.STEP_AUTO, pk[c], nm[c], prev_packed=pk[p] if t > 1 else None,
                              prev_norms=nm[p] if t > 1 else None)
        plan.qoda_step(pk[c], nm[c], X1, Y, Xh)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for i, t in enumerate((3, 4)):
            c, p = t % 2, (t + 1) % 2
            plan.lq_quantize_pack(gin[i], lqm.STEP_AUTO, pk[c], nm[c], prev_packed=pk[p], prev_norms=nm[p])
            plan.qoda_step(pk[c], nm[c], X1, Y, Xh)
    for r in range(3):
        gin[0].copy_(grads[2 + 2 * r]); gin[1].copy_(grads[3 + 2 * r])
        graph.replay()
    torch.cuda.synchronize()
    got = [x.cpu().numpy() for x in (Y, Xh, pk[0], pk[1], nm[0], nm[1])]
    for a, b in zip(got, want):
        assert np.array_equal(a, b)
    assert plan.qoda_get_scalars() == want_scalars
