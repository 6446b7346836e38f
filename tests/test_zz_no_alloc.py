"""The allocation-free norm entry point against the plan-based one (runs last: the file name sorts
after every other test file).

lq_vector_norm_static serves callers that cannot allocate device memory when they need a norm
(their memory belongs to another allocator, or an allocation's device-wide synchronisation is not
acceptable there), so they cannot create a plan; its reduction scratch is a fixed array inside the
library.  Two calls in a row share that array: the second call must not see anything of the
first, also when it covers fewer tiles.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu
TILE = 32 * 1024


def _plan_norm(lqm, v, q):
    plan = lqm.Plan([v.numel()], 4, q, 1, 0)
    grads = torch.zeros((1, plan.padded_elems), device="cuda")
    grads[0, : v.numel()] = v
    norms = plan.empty_norms()
    plan.lq_layer_norms(grads, norms)
    torch.cuda.synchronize()
    _, flags = plan.lq_get_statistics()
    return float(norms[0, 0]), int(flags[0, 0])


@pytest.mark.parametrize("q", [2, 0, 1, 3])
def test_two_calls_in_a_row_match_the_plan_based_norm(q):
    import paper_2505_14371_b200 as lqm
    lqm.load_library()
    g = torch.Generator(device="cuda").manual_seed(77 + q)
    big = torch.randn(5 * TILE + 1234, generator=g, device="cuda") * 0.01      # 6 tiles, ragged tail
    small = torch.randn(TILE // 2 + 7, generator=g, device="cuda") * 3.0       # 1 tile
    out = torch.full((2,), -1.0, device="cuda")
    st = torch.full((2,), -1, dtype=torch.int32, device="cuda")
    lqm.lq_vector_norm_static(big, q, out[0:1], st[0:1])
    lqm.lq_vector_norm_static(small, q, out[1:2], st[1:2])                     # same stream: ordered
    torch.cuda.synchronize()
    for i, v in enumerate([big, small]):
        want, flag = _plan_norm(lqm, v, q)
        got = float(out[i])
        assert abs(got - want) <= 1e-6 * want, (q, i, got, want)
        assert int(st[i]) == flag == 0
        ref = np.linalg.norm(v.cpu().numpy().astype(np.float64), ord=np.inf if q == 0 else q)
        assert abs(got - ref) <= 1e-6 * ref


def test_calls_allocate_no_device_memory():
    """What the entry point exists for: after a first call (which may load the library's module on the device),
    further calls leave the device's free memory and torch's own allocation count unchanged."""
    import paper_2505_14371_b200 as lqm
    lqm.load_library()
    v = torch.randn(3 * TILE + 5, device="cuda")
    out = torch.zeros(1, device="cuda"); st = torch.zeros(1, dtype=torch.int32, device="cuda")
    lqm.lq_vector_norm_static(v, 2, out, st)
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    held0 = torch.cuda.memory_allocated()
    for q in (2, 0, 1, 2):
        lqm.lq_vector_norm_static(v, q, out, st)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0 and torch.cuda.memory_allocated() == held0


def test_flags_limits_and_empty_input():
    import paper_2505_14371_b200 as lqm
    lib = lqm.load_library()
    out = torch.full((1,), -1.0, device="cuda"); st = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    v = torch.ones(1000, device="cuda"); v[123] = float("inf")
    lqm.lq_vector_norm_static(v, 2, out, st)
    torch.cuda.synchronize()
    assert float(out[0]) == 0.0 and int(st[0]) == lqm.STATUS_NONFINITE
    lqm.lq_vector_norm_static(torch.zeros(5000, device="cuda"), 2, out, st)
    torch.cuda.synchronize()
    assert float(out[0]) == 0.0 and int(st[0]) == lqm.STATUS_ZERO_NORM
    out.fill_(-1.0)
    rc = lib.lq_vector_norm_static(None, 0, 2, out.data_ptr(), None, None)     # n = 0: nothing to read
    torch.cuda.synchronize()
    assert rc == 0 and float(out[0]) == 0.0
    too_many = 4096 * TILE + 1                                                 # one value past the fixed scratch
    rc = lib.lq_vector_norm_static(v.data_ptr(), too_many, 2, out.data_ptr(), None, None)
    assert rc == -1 and b"fixed scratch" in lib.lq_last_error()
    with pytest.raises(lqm.LqError):
        lqm.lq_vector_norm_static(v[1:], 2, out, st)                           # not 16-byte aligned
