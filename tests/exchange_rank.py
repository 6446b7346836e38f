"""One rank of the exchange test (run as a child process by test_gpu_exchange.py; not a test module).

argv: rank world port out_dir scope.  All ranks draw the same K rows of gradients from one seed and keep their own
rows; three iterations with a histogram and a level fit after the first; the final state goes to a .npz file."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

SIZES, BITS, K, Q, SEED = [40000, 1000, 129, 5000], [4, 3, 2, 5], 4, 2, 99


def run(rank: int, world: int, scope: str, group_ready: bool):
    import paper_2505_14371_b200 as lqm
    from paper_2505_14371_b200.exchange import ExchangeStep
    lqm.load_library()
    plan = lqm.Plan(SIZES, BITS, Q, K, SEED)
    plan.lq_set_norm_scope(scope)
    ex = ExchangeStep(plan, rank, world)
    g = torch.Generator(device="cuda").manual_seed(5)
    X1 = torch.randn(plan.padded_elems, generator=g, device="cuda") * 0.1
    Y = torch.empty_like(X1); Xh = torch.empty_like(X1)
    X = torch.zeros_like(X1); gbar = torch.zeros_like(X1)       # padding elements are never written
    plan.qoda_init(X1, Y, Xh)
    for t in (1, 2, 3):
        grads = torch.randn((K, plan.padded_elems), generator=g, device="cuda") * (0.5 ** t)
        grads[1, 100:700] = 0.0
        hist = plan.zero_hist() if t == 1 else None
        ex.step(grads[ex.first: ex.first + ex.count].contiguous(), t, X1, Y, Xh, X, gbar, hist=hist)
        if t == 1:
            ex.fit_levels(hist)
    torch.cuda.synchronize()
    tt, S, eta = plan.qoda_get_scalars()
    return dict(Y=Y.cpu().numpy(), Xh=Xh.cpu().numpy(), X=X.cpu().numpy(), gbar=gbar.cpu().numpy(),
                packed=ex.packed[ex.cur].cpu().numpy(), norms=ex.norms[ex.cur].cpu().numpy(),
                scalars=np.array([tt, S, eta]), levels=np.array(plan.lq_get_levels(0), np.float32),
                **{f"levels{m}": np.array(plan.lq_get_levels(m), np.float32) for m in range(len(SIZES))})


if __name__ == "__main__":
    rank, world, port, out_dir, scope = int(sys.argv[1]), int(sys.argv[2]), sys.argv[3], sys.argv[4], sys.argv[5]
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=port)
    torch.cuda.set_device(0)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    out = run(rank, world, scope, True)
    np.savez(os.path.join(out_dir, f"rank{rank}.npz"), **out)
    dist.barrier()
    dist.destroy_process_group()
