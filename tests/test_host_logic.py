"""CPU-only checks of the host side: the C-ABI library loads and exports every symbol the header
declares, and the benchmark's multi-rank bookkeeping (max over ranks, whole-job value) works
across two gloo ranks.  No kernel is launched here.
"""
import ctypes
import json
import os
import re
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "lq.h")


def _declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)             # drop comments
    text = re.sub(r"^\s*#.*$", "", text, flags=re.M)              # drop preprocessor lines
    names = re.findall(r"\b([a-z_][a-z0-9_]*)\s*\([^;{]*\)\s*;", text)
    return sorted(set(names))


def test_header_declares_the_named_entry_points():
    names = _declared_functions()
    for required in ["lq_plan_create", "lq_fit_levels", "lq_quantize_pack", "lq_decode_aggregate", "qoda_step"]:
        assert required in names
    assert len(names) >= 19


def test_library_builds_loads_and_exports_every_declared_symbol():
    from paper_2505_14371_b200 import build as b
    path = b.build()
    lib = ctypes.CDLL(path)
    for name in _declared_functions():
        assert hasattr(lib, name), f"liblq.so does not export {name}"
    # the binding declares the same set
    from paper_2505_14371_b200 import binding
    assert sorted(binding.EXPORTS) == _declared_functions()
    # entry points that touch no device
    lib.lq_error_string.restype = ctypes.c_char_p
    assert lib.lq_error_string(0) == b"ok"
    assert lib.lq_error_string(-1) == b"invalid argument"
    lib.lq_plan_padded_elems.restype = ctypes.c_int64
    lib.lq_plan_padded_elems.argtypes = [ctypes.c_void_p]
    assert lib.lq_plan_padded_elems(None) == -1                   # LQ_EINVAL, reported not crashed
    assert lib.lq_plan_destroy(None) == 0


def test_binding_has_no_cpu_fallback(monkeypatch):
    from paper_2505_14371_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", os.path.join(ROOT, "does_not_exist", "liblq.so"))
    with pytest.raises(binding.LqError):
        binding.load_library()


def test_product_package_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2505_14371_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.lower().replace("cpu oracle", ""), f


_RANK_SCRIPT = r"""
import json, os, sys
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
local_ms = 2.0 if rank == 0 else 5.0            # rank 1 is the slow one
ms = bench.aggregate_over_ranks(local_ms, world)
value = bench.whole_job_value(10.0, world, ms)
open(os.path.join({out!r}, "rank%d.json" % rank), "w").write(json.dumps({{"rank": rank, "ms": ms, "value": value}}))
dist.destroy_process_group()
"""


def test_two_gloo_ranks_take_the_max_time_and_sum_the_units(tmp_path):
    script = tmp_path / "rank.py"
    script.write_text(_RANK_SCRIPT.format(root=ROOT, out=str(tmp_path)))
    port = 29500 + os.getpid() % 2000
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                          "--master-addr", "127.0.0.1", "--master-port", str(port), str(script)],
                         capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    rows = [json.loads((tmp_path / f"rank{r}.json").read_text()) for r in range(2)]
    assert sorted(r["rank"] for r in rows) == [0, 1]
    for r in rows:
        assert r["ms"] == 5.0                                     # max over ranks
        assert abs(r["value"] - 2 * 10.0 / 5e-3) < 1e-9           # all ranks' units / slowest rank's time


def test_bench_gpus_n_starts_its_own_ranks():
    """`python bench.py --gpus 2` with no launcher around it starts two ranks by itself; with the stand-in step
    (gloo, no GPU) rank 0 reports the world size, the slowest rank's time and the whole job's units."""
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--stub-step", "--steps", "3"],
                         capture_output=True, text=True, timeout=300, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                        # rank 0 alone prints
    assert lines[0]["n_gpus"] == 2 and lines[0]["ms_per_step"] == 2.0 and lines[0]["steps"] == 3
    assert abs(lines[0]["value"] - 2 * 1.0 / 2e-3) < 1e-9


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                         capture_output=True, text=True, timeout=120, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_library_code_builder_is_optimal_like_the_oracles(orc):
    """lq_code_build runs on the host only.  Huffman lengths are not unique under ties, so the two builders are
    compared through what is unique: the expected length (optimal), Kraft's equality and the length limit."""
    import numpy as np
    from paper_2505_14371_b200 import binding
    binding.load_library()
    rng = np.random.default_rng(12)
    for n in (1, 2, 4, 8, 16, 32, 256):
        for _ in range(5):
            w = rng.dirichlet(np.ones(n) * 0.3) if n > 1 else np.ones(1)
            if n > 2:
                w[rng.integers(0, n)] = 0.0
            ours = np.array(binding.lq_code_build(w))
            ref = orc.huffman_lengths(w).astype(int)
            assert ours.min() >= 1 and ours.max() <= 12
            if n > 1:
                assert abs(sum(2.0 ** -int(x) for x in ours) - 1.0) < 1e-12
            wf = np.maximum(w, w.sum() * 2.0 ** -40)
            assert abs(float((wf * ours).sum()) - float((wf * ref).sum())) <= 1e-9 * float((wf * ref).sum())
    geometric = 0.5 ** np.arange(40)
    assert max(binding.lq_code_build(geometric)) == 12
    assert binding.lq_code_build([0.4, 0.3, 0.2, 0.1]) == [1, 2, 3, 3]
    with pytest.raises(binding.LqError):
        binding.lq_code_build([0.5, -0.1])


# ---------------------------------------------------------------------------------------------- exchange plumbing
class _FakePlan:
    """Stands in for a Plan on a machine without a GPU: records the call order and lets "encode" write
    worker-specific values into the rows of its range, so that the all-gather's assembly can be checked."""

    def __init__(self, K, L, W):
        self.num_workers, self.num_layers, self.W = K, L, W
        self.calls = []

    def lq_set_worker_range(self, first, count):
        self.first, self.count = first, count

    def empty_packed(self, device):
        import torch
        return torch.empty((self.num_workers, self.W), dtype=torch.int32, device=device)

    def empty_norms(self, device):
        import torch
        return torch.empty((self.num_workers, self.num_layers), dtype=torch.float32, device=device)

    def lq_quantize_pack(self, grads, step, packed, norms, hist=None, prev_packed=None, prev_norms=None):
        self.calls.append(("quantize", step, prev_packed is not None))
        for i in range(self.count):
            k = self.first + i
            packed[k] = 1000 * step + k
            norms[k] = float(k) + 0.5
            if hist is not None:
                hist[k] = k + 1
        self.step = step

    def lq_side_data_export(self, sq, w, f):
        for i in range(self.count):
            k = self.first + i
            sq[k] = 10.0 * self.step + k; w[k] = k; f[k] = k % 2

    def lq_side_data_import(self, sq, w, f):
        self.imported = (sq.clone(), w.clone(), f.clone())

    def qoda_step(self, packed, norms, X1, Y, Xhalf, X, gbar):
        self.calls.append(("qoda_step",))
        self.seen = (packed.clone(), norms.clone())


def _exchange_rank(rank, world, port, out_dir):
    import json
    import os
    import torch
    import torch.distributed as dist
    from paper_2505_14371_b200.exchange import ExchangeStep
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    K, L, W = 4, 3, 8
    plan = _FakePlan(K, L, W)
    ex = ExchangeStep(plan, rank, world, device="cpu")
    hist = torch.zeros((K, L, 4), dtype=torch.int32)
    for t in (1, 2):
        ex.step(torch.zeros((ex.count, 16)), t, None, None, None, hist=hist if t == 1 else None)
    packed, norms = plan.seen
    sq, w, f = plan.imported
    ok = all(int(packed[k, 0]) == 2000 + k and float(norms[k, 0]) == k + 0.5 and float(sq[k, 0]) == 20.0 + k
             and float(w[k, 0]) == k and int(f[k, 0]) == k % 2 and int(hist[k, 0, 0]) == k + 1 for k in range(K))
    with open(os.path.join(out_dir, f"x{rank}.json"), "w") as fh:
        json.dump({"ok": ok, "calls": plan.calls, "range": [ex.first, ex.count]}, fh)
    dist.barrier()
    dist.destroy_process_group()


def test_exchange_worker_ranges():
    from paper_2505_14371_b200.exchange import worker_range
    assert [worker_range(r, 4, 8) for r in range(4)] == [(0, 2), (2, 2), (4, 2), (6, 2)]
    assert worker_range(0, 1, 8) == (0, 8)
    with pytest.raises(ValueError):
        worker_range(0, 3, 8)
    with pytest.raises(ValueError):
        worker_range(2, 2, 8)


def test_exchange_assembles_all_rows_with_gloo_two_ranks(tmp_path):
    import json
    import socket
    import torch.multiprocessing as mp
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_exchange_rank, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    for r in range(2):
        rec = json.load(open(tmp_path / f"x{r}.json"))
        assert rec["ok"] and rec["range"] == [2 * r, 2]
        # the second message is encoded against the first; each encode is followed by one update
        assert rec["calls"] == [["quantize", 1, False], ["qoda_step"], ["quantize", 2, True], ["qoda_step"]]


def test_universal_code_lengths_match_the_recursive_code(orc):
    import paper_2505_14371_b200 as lqm
    for n in (2, 4, 8, 16, 32, 63):
        assert lqm.lq_code_universal(n) == [len(orc.elias_omega(j + 1)) for j in range(n)]
    with pytest.raises(lqm.LqError):
        lqm.lq_code_universal(64)                                      # its last word would have 13 bits
