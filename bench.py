#!/usr/bin/env python
"""Benchmark of the QODA hot path on B200: one step = lq_quantize_pack (norm + stochastic
rounding + packing + step-size statistic) followed by qoda_step (fused decode + aggregate +
update) over one Transformer-XL-shaped synthetic gradient set for K = 8 simulated workers.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload NAME]

Prints ONE JSON line.  `value` is GB/s of fp32 input (4*K*D bytes per step) with the inputs
resident in HBM; `e2e` is the same with the gradients copied from pinned host memory and the
new iterate copied back inside the timed region.  `roofline` describes the kernel that takes the
most time on the bytes that really cross DRAM (ncu counters), with the algorithmic-bytes figure
beside it and the same kernel on dense data under `roofline.dense`.  With --impl reference the
CPU oracle is timed on a bounded sample instead.  With N > 1 every rank runs an independent
replica of the workload (one process per GPU: started by torch.distributed.run, or by this
script itself when it is called with --gpus N and no launcher): the method does not shard inside
one node's GPU, so there is no collective on the data path, only the barrier and the
max-over-ranks of the timing.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "quantize+pack and decode+aggregate+QODA GB/s (fp32 in)"

# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum, one ncu capture per kernel) with the hash
# of the kernel's sources at capture time: once a source changes, the figure no longer describes the kernel and
# `traffic` is reported as null.  The Transformer-XL-shaped job is too large to capture under ncu, so its figures
# come from two cut-down versions of the same recipe (profiles/dram_traffic__transformer_xl_scaled.md): the traffic
# of a launch is a * E + b * N for E worker-coordinates in the embedding (90 % zero rows) and N in the other layers,
# and (a, b) solve the two captures.  `inst` is the same for executed warp instructions (smsp__inst_executed.sum).
KERNEL_SOURCES = {"norm_partial": ["lq_norm.cu", "lq_internal.cuh"],
                  "quantize_pack": ["lq_quantize.cu", "lq_quantize.cuh", "lq_internal.cuh"],
                  "decode": ["lq_decode.cu", "lq_internal.cuh"]}
NCU_SCALED = {"transformer_xl": {          # kernel: bytes per embedding / other worker-coordinate, warp instr likewise
    "norm_partial": {"bytes": (4.0063, 4.0085), "inst": (0.15710, 0.16787), "sources": "16beee4053b150a1"},
    "quantize_pack": {"bytes": (1.3329, 5.3699), "inst": (0.22306, 1.29301), "sources": "2647a4d8ec44ca40"},
    "decode": {"bytes": (2.1174, 2.6372), "inst": (0.23964, 0.24161), "sources": "2027312c991fef2d"}}}
NCU_DIRECT = {"flat:26:4:8:2": {           # kernel: bytes and warp instructions of one launch
    "quantize_pack": {"bytes": 2485848064.0 + 367199744.0, "inst": 679714816.0, "sources": "2647a4d8ec44ca40"}}}
DENSE_POINT = "flat:26:4:8:2"             # dense companion of the headline workload: no zero rows to skip
ISSUE_PEAK = 148 * 4 * 1.965e9            # warp instructions per second: 148 SMs x 4 schedulers x 1 per clock at 1965 MHz


def source_hash(kernel: str) -> str:
    import hashlib
    h = hashlib.sha1()
    for f in KERNEL_SOURCES[kernel]:
        h.update(open(os.path.join(ROOT, "paper_2505_14371_b200", "csrc", f), "rb").read())
    return h.hexdigest()[:16]


def ncu_counters(key: str, workload, kernel: str):
    """(DRAM bytes, warp instructions) of one launch of `kernel` on the workload named `key` (the --workload
    string) from the committed ncu captures, or (None, None) when there is none or the kernel's sources have
    changed since."""
    rec = NCU_DIRECT.get(key, {}).get(kernel)
    if rec is not None:
        if rec["sources"] != source_hash(kernel) or rec["bytes"] is None:
            return None, None
        return rec["bytes"], rec["inst"]
    rec = NCU_SCALED.get("transformer_xl" if key.startswith("transformer_xl") else key, {}).get(kernel)
    if rec is None or rec["sources"] != source_hash(kernel) or rec["bytes"][0] is None:
        return None, None
    K = workload.num_workers
    emb = K * workload.layer_sizes[0]                      # the first layer of this recipe is the embedding
    rest = K * (workload.num_coords - workload.layer_sizes[0])
    return (rec["bytes"][0] * emb + rec["bytes"][1] * rest, rec["inst"][0] * emb + rec["inst"][1] * rest)


# ------------------------------------------------------------------------------ workloads
def pick_workload(name: str):
    from paper_2505_14371_b200 import workloads as W
    if name == "transformer_xl":
        return W.transformer_xl_workload()
    if name == "wgan":
        return W.wgan_workload()
    if name.startswith("wgan:"):                       # wgan:<bits>: the same shapes at another code width (Section 7.1 runs 5 bits)
        w = W.wgan_workload()
        w.bits = int(name.split(":")[1])
        return w
    if name == "mlp":
        return W.mlp_workload()
    if name == "transformer_xl_small":
        return W.transformer_xl_workload(num_blocks=2, vocab=8192)
    if name == "transformer_xl_medium":                # all 16 blocks, a quarter of the vocabulary
        return W.transformer_xl_workload(num_blocks=16, vocab=65536)
    if name.startswith("transformer_xl:"):             # transformer_xl:<blocks>:<vocabulary>: the same recipe cut down
        nb, vocab = (int(x) for x in name.split(":")[1:3])
        return W.transformer_xl_workload(num_blocks=nb, vocab=vocab)
    if name.startswith("powersgd:"):                   # powersgd:<rank>: low-rank factor shapes (Section 7.2)
        return W.powersgd_factor_workload(int(name.split(":")[1]))
    if name.startswith("flat:"):                       # flat:<log2 n>:<bits>:<K>:<q>
        n, b, k, q = (int(x) for x in name.split(":")[1:5])
        return W.flat_workload(n, b, k, q)
    if name.startswith("ragged:"):                     # ragged:<bits>:<K>:<q>
        b, k, q = (int(x) for x in name.split(":")[1:4])
        return W.ragged_workload(b, k, q)
    raise SystemExit(f"unknown workload {name}")


# --------------------------------------------------------------------------- clock sampler
class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [c.strip() for c in line.split(",")]))

    def stop(self, t0: float, t1: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        self.thread.join(timeout=2)
        rows = [r for t, r in self.rows if t0 - 0.05 <= t <= t1 + 0.15] or [r for _, r in self.rows[-3:]]
        sm, mx, reasons = [], [], set()
        for r in rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for name, v in zip(["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"], r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# -------------------------------------------------------------------------- CPU oracle leg
def oracle_sample_workload():
    """Bounded sample of the Transformer-XL-shaped workload for the CPU oracle: 8192 embedding
    rows and one transformer block, all 8 workers, same value recipe."""
    from paper_2505_14371_b200 import workloads as W
    return W.transformer_xl_workload(num_blocks=1, vocab=8192)


def time_oracle(steps: int, warmup: int, threads: int = 1) -> dict:
    """Times the oracle, as it stands (single-threaded C behind ctypes), on the sample.  threads = 1: the oracle's
    own K-worker loop.  threads > 1: the same per-(worker, layer) calls, the K workers dealt to a pool of host
    threads (ctypes releases the interpreter lock inside the C routines), then the oracle's aggregation and
    update on one thread."""
    import numpy as np
    import torch
    from concurrent.futures import ThreadPoolExecutor
    from oracle import oracle as orc
    from paper_2505_14371_b200 import workloads as W
    orc.build()
    w = oracle_sample_workload()
    offs = np.concatenate([[0], np.cumsum(w.layer_sizes)]).astype(np.int64)
    D = int(offs[-1])
    grads = W.make_gradients(w, [int(x) for x in offs[:-1]], D, "cpu").numpy()
    K, Lr = w.num_workers, w.num_layers
    model = orc.OracleModel(w.layer_sizes, [w.bits] * Lr, w.q, K, W.PHILOX_SEED)
    g = torch.Generator(device="cpu").manual_seed(W.SEED_BASE + 99)
    model.qoda_init(torch.randn(D, generator=g).numpy())

    def worker_message(k, step, decoded, sq, prev):
        for m in range(Lr):
            a, b = int(offs[m]), int(offs[m + 1])
            v = grads[k, a:b]
            norm, _ = orc.layer_norm(v, w.q)
            idx, sgn, _ = orc.quantize_layer(v, norm, model.levels[m], W.PHILOX_SEED, step, k, m)
            orc.pack_layer(idx, sgn, w.bits)
            decoded[k, a:b] = orc.decode_layer(idx, sgn, norm, model.levels[m])
            sq[k, m] = orc.sq_diff(decoded[k, a:b], None if prev is None else prev[k, a:b])

    pool = ThreadPoolExecutor(max_workers=threads) if threads > 1 else None
    times = []
    for s_ in range(warmup + steps):
        t0 = time.perf_counter()
        if pool is None:
            model.quantize(grads, s_ + 1)
        else:
            decoded = np.zeros((K, D), np.float32); sq = np.zeros((K, Lr), np.float64)
            list(pool.map(lambda k: worker_message(k, s_ + 1, decoded, sq, model.prev_decoded), range(K)))
            model.pending_sq, model.cur_decoded = sq, decoded
        model.qoda_step()
        t1 = time.perf_counter()
        if s_ >= warmup:
            times.append(t1 - t0)
    if pool is not None:
        pool.shutdown()
    sec = sum(times) / len(times)
    return {"value": 4.0 * K * D / sec / 1e9, "unit": "GB/s", "cores": min(threads, K), "kind": "oracle",
            "sample": f"transformer_xl shapes cut to 8192 embedding rows + 1 block "
                      f"({D} coords x K={K}), {len(times)} step(s), {sec:.2f} s/step",
            "ms_per_step": sec * 1e3}


def cpu_baseline_record() -> dict:
    """The oracle on all host cores (the K workers on a thread pool) with the one-core figure beside it."""
    ncores = os.cpu_count() or 1
    one = time_oracle(2, 0, 1)
    rec = {k: one[k] for k in ("value", "unit", "cores", "kind", "sample")}
    rec["host_cores"] = ncores
    if ncores > 1:
        many = time_oracle(2, 0, ncores)
        rec = {k: many[k] for k in ("value", "unit", "cores", "kind", "sample")}
        rec.update({"host_cores": ncores, "value_1core": one["value"],
                    "note": "cores = threads that had work (one per worker); value_1core = the oracle's own loop on one core"})
    return rec


def run_reference(args) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps, warmup = max(1, min(args.steps, 3)), min(args.warmup, 1)
    r = time_oracle(steps, warmup, os.cpu_count() or 1)
    w = pick_workload(args.workload)
    line = {"impl": "reference", "metric": METRIC, "value": r["value"], "unit": "GB/s", "n_gpus": args.gpus,
            "steps": steps, "warmup": warmup, "ms_per_step": r["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": "transformer_xl_shaped", "num_workers": w.num_workers, "bits": w.bits,
                       "q": w.q, "note": "CPU oracle on a bounded sample of this workload"},
            "cpu_baseline": dict({k: r[k] for k in ("value", "unit", "cores", "kind", "sample")}, host_cores=os.cpu_count() or 1),
            "e2e": {"value": r["value"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------- GPU leg
def aggregate_over_ranks(local_ms: float, world: int, device=None, backend_reduce=None) -> float:
    """Max over ranks of the per-rank step time (host logic shared with the CPU gloo test)."""
    if world == 1:
        return local_ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(units_per_rank: float, world: int, max_ms: float) -> float:
    """Units all ranks processed divided by the slowest rank's time (weak scaling)."""
    return units_per_rank * world / (max_ms * 1e-3)


def kernel_roofline(alg_bytes: float, traffic, inst, avg_ms: float, peak: float) -> dict:
    """Roofline entries of one kernel: on the bytes that move (ncu DRAM traffic) when known, and on the method's
    algorithmic bytes; plus the share of the GPU's instruction-issue slots its executed instructions take."""
    sec = avg_ms * 1e-3
    out = {"traffic": traffic,
           "gbs": traffic / sec / 1e9 if traffic else None,
           "frac": traffic / sec / 1e9 / peak if traffic else None,
           "gbs_algorithmic": alg_bytes / sec / 1e9, "frac_algorithmic": alg_bytes / sec / 1e9 / peak,
           "issue_frac": inst / sec / ISSUE_PEAK if inst else None}
    return out


def dense_point(pkg, W, dev, peak: float, steps: int = 12) -> dict:
    """The encoder on dense data (a flat layer of 2^26 N(0,1) coordinates x 8 workers, 4 bits): no zero rows to
    skip, so the kernel does its full work per coordinate.  Same measurement as the main run, fewer steps."""
    w = pick_workload(DENSE_POINT)
    K, D = w.num_workers, w.num_coords
    plan = pkg.Plan(w.layer_sizes, w.bits, w.q, K, W.PHILOX_SEED)
    import torch
    grads = W.make_gradients(w, plan.elem_offsets, plan.padded_elems, dev)
    pk = [plan.empty_packed(dev), plan.empty_packed(dev)]; nm = [plan.empty_norms(dev), plan.empty_norms(dev)]
    X1 = torch.randn(plan.padded_elems, device=dev); Y = torch.empty_like(X1); Xh = torch.empty_like(X1)
    plan.qoda_init(X1, Y, Xh)
    for t in range(1, 4 + steps):
        if t == 4:
            torch.cuda.synchronize()
            plan.lq_profile_enable(True); plan.lq_profile_read()
        c, p = t % 2, (t + 1) % 2
        plan.lq_quantize_pack(grads, t, pk[c], nm[c], prev_packed=None if t == 1 else pk[p], prev_norms=None if t == 1 else nm[p])
        plan.qoda_step(pk[c], nm[c], X1, Y, Xh)
    prof = plan.lq_profile_read()
    plan.close()
    cb = (w.bits + 1) / 8.0
    tot, cnt = prof["quantize_pack"]
    traffic, inst = ncu_counters(DENSE_POINT, w, "quantize_pack")
    rec = {"workload": DENSE_POINT, "kernel": "quantize_pack", "coords_x_workers": K * D, "avg_ms": tot / cnt}
    rec.update(kernel_roofline((4.0 + 2 * cb) * K * D, traffic, inst, tot / cnt, peak))
    rec["lq_quantize_pack_ms"] = sum(prof[n][0] / prof[n][1] for n in ("norm_partial", "norm_finalize", "quantize_pack", "stat_finalize") if prof[n][1])
    return rec


def run_gpu(args) -> None:
    import torch
    import torch.distributed as dist
    import paper_2505_14371_b200 as pkg
    from paper_2505_14371_b200 import workloads as W

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        os.environ.setdefault("NCCL_DEBUG", "INFO")      # the communicator lines (on stderr) show how many ranks joined
        dist.init_process_group("nccl", device_id=dev)
    pkg.load_library()

    w = pick_workload(args.workload)
    K, D = w.num_workers, w.num_coords
    plan = pkg.Plan(w.layer_sizes, w.bits, w.q, K, W.PHILOX_SEED)
    plan.lq_set_norm_scope(args.norm_scope)
    bucket = args.norm_scope == "bucket"
    grads = W.make_gradients(w, plan.elem_offsets, plan.padded_elems, dev)
    packed = [plan.empty_packed(dev), plan.empty_packed(dev)]
    norms = [plan.empty_norms(dev), plan.empty_norms(dev)]
    ex = None
    if args.exchange:
        # the K workers are shared out over the ranks; messages travel by all-gather (strong scaling)
        from paper_2505_14371_b200.exchange import ExchangeStep
        ex = ExchangeStep(plan, rank, world, device=dev)
        grads = grads[ex.first: ex.first + ex.count].contiguous()
        del packed, norms
    share = 1.0 / world if args.exchange else 1.0     # this rank's part of the job's 4 K D input bytes
    g = torch.Generator(device=dev).manual_seed(W.SEED_BASE + 99)
    X1 = torch.randn(plan.padded_elems, generator=g, device=dev)
    Y = torch.empty_like(X1); Xh = torch.empty_like(X1)
    plan.qoda_init(X1, Y, Xh)

    state = {"t": 0}

    def step():
        state["t"] += 1
        t = state["t"]
        if ex is not None:
            ex.step(grads, t, X1, Y, Xh)
            return
        c, p = t % 2, (t + 1) % 2
        plan.lq_quantize_pack(grads, t, packed[c], norms[c],
                              prev_packed=None if t == 1 else packed[p],
                              prev_norms=None if t == 1 else norms[p])
        plan.qoda_step(packed[c], norms[c], X1, Y, Xh)

    # adaptive levels: one histogram + fit before the steady state (Algorithm 1 lines 2-7)
    hist = plan.zero_hist(dev)
    state["t"] += 1
    if ex is not None:
        ex.step(grads, 1, X1, Y, Xh, hist=hist)
        ex.fit_levels(hist)
    else:
        plan.lq_quantize_pack(grads, 1, packed[1], norms[1], hist=hist)
        plan.lq_fit_levels(hist, norms[1], K)
        plan.qoda_step(packed[1], norms[1], X1, Y, Xh)
    del hist
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing ----------------------------------------------------------
    sampler = ClockSampler(local)
    plan.lq_profile_enable(True); plan.lq_profile_read()
    barrier()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.time()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    t1 = time.time()
    clocks = sampler.stop(t0, t1)
    local_ms = e0.elapsed_time(e1) / args.steps
    prof = plan.lq_profile_read()
    plan.lq_profile_enable(False)
    ms = aggregate_over_ranks(local_ms, world, dev)
    graph_ms, graph_error = None, None
    if args.graph and ex is None:
        # two iterations recorded once (messages and masks are double-buffered), replayed steps / 2 times; the step
        # index comes from the plan's device-side counter, so nothing in the recording changes between replays
        def auto_step():
            state["t"] += 1
            c, p = state["t"] % 2, (state["t"] + 1) % 2
            plan.lq_quantize_pack(grads, pkg.STEP_AUTO, packed[c], norms[c], prev_packed=packed[p], prev_norms=norms[p])
            plan.qoda_step(packed[c], norms[c], X1, Y, Xh)
        try:
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                auto_step(); auto_step()
            for _ in range(3):
                graph.replay()
            torch.cuda.synchronize()
            reps = max(1, args.steps // 2)
            e0.record()
            for _ in range(reps):
                graph.replay()
            e1.record()
            torch.cuda.synchronize()
            graph_ms = e0.elapsed_time(e1) / (2 * reps)
        except RuntimeError as exc:      # the headline number above does not depend on this extra measurement
            graph_error = str(exc)[:200]
        # every rank takes part in the reduction, also one whose recording failed
        graph_ms = aggregate_over_ranks(graph_ms if graph_ms is not None else float("inf"), world, dev)
        if graph_ms == float("inf"):
            graph_ms, graph_error = None, graph_error or "the recording failed on another rank"

    # ---- end to end: pinned host gradients in, new iterate out ------------------------------
    e2e = None
    try:
        host_grads = torch.empty(grads.shape, dtype=torch.float32, pin_memory=True)
        host_grads.copy_(grads)
        host_out = torch.empty(Xh.shape, dtype=torch.float32, pin_memory=True)
        e2e_steps = max(1, min(args.steps, 5))

        # the result travels back on a second stream, so that it shares the link with the next step's input
        # (PCIe is full duplex); the next update waits for that copy before it overwrites the iterate
        back = torch.cuda.Stream(device=dev)
        done_step, done_copy = torch.cuda.Event(), torch.cuda.Event()
        done_copy.record()

        def e2e_step():
            grads.copy_(host_grads, non_blocking=True)
            torch.cuda.current_stream().wait_event(done_copy)
            step()
            done_step.record()
            with torch.cuda.stream(back):
                back.wait_event(done_step)
                host_out.copy_(Xh, non_blocking=True)
                done_copy.record()

        e2e_step(); barrier()
        e0.record()
        for _ in range(e2e_steps):
            e2e_step()
        e1.record()
        barrier()
        e2e_ms = aggregate_over_ranks(e0.elapsed_time(e1) / e2e_steps, world, dev)
        e2e = {"value": whole_job_value(4.0 * K * D * share / 1e9, world, e2e_ms), "unit": "GB/s",
               "h2d_bytes_per_step": host_grads.numel() * 4, "d2h_bytes_per_step": host_out.numel() * 4,
               "ms_per_step": e2e_ms}
        del host_grads, host_out
    except RuntimeError as exc:      # pinned allocation can fail on a small host
        e2e = {"value": None, "unit": "GB/s", "error": str(exc)[:200]}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    dense = None
    if world == 1 and args.workload == "transformer_xl" and args.norm_scope == "layer" and not args.no_dense:
        del grads
        torch.cuda.empty_cache()
        peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
        pk_ = float(json.load(open(peaks_path))["hbm_gbs"]) if os.path.exists(peaks_path) else 6650.0
        dense = dense_point(pkg, W, dev, pk_)

    # ---- roofline of the dominant kernel --------------------------------------------------
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        peak, peak_src = float(json.load(open(peaks_path))["hbm_gbs"]), "measured"
    else:
        peak, peak_src = 6650.0, "fallback"
    c = (w.bits + 1) / 8.0
    # algorithmic bytes per launch: what the method itself must move, per kernel
    alg = {"norm_partial": 4.0 * K * D, "quantize_pack": (4.0 + 2 * c) * K * D, "decode": (K * c + 16.0) * D}
    if bucket:                                # one pass, and 4 bytes of norm per 128 coordinates wherever a message moves
        cb = c + 4.0 / 128.0
        alg = {"quantize_pack": (4.0 + 2 * cb) * K * D, "decode": (K * cb + 16.0) * D}
    if args.exchange:                         # a rank encodes only its share of the workers (and decodes all of them)
        for name in ("norm_partial", "quantize_pack"):
            if name in alg:
                alg[name] *= share
    counted = args.norm_scope == "layer" and not args.exchange    # the counters were taken in the default configuration
    kern = {}
    for name, (tot, cnt) in prof.items():
        if cnt:
            avg = tot / cnt
            kern[name] = {"avg_ms": avg, "launches_per_step": cnt / args.steps}
            if name in alg:
                traffic, inst = ncu_counters(args.workload, w, name) if counted else (None, None)
                kern[name].update(kernel_roofline(alg[name], traffic, inst, avg, peak))
    dominant = max((n for n in kern if n in alg), key=lambda n: kern[n]["avg_ms"] * kern[n]["launches_per_step"])
    kd = kern[dominant]
    roofline = {"bound": "hbm", "kernel": dominant, "achieved": kd["gbs"], "peak": peak, "peak_source": peak_src,
                "unit": "GB/s", "frac": kd["frac"], "traffic": kd["traffic"],
                "achieved_algorithmic": kd["gbs_algorithmic"], "frac_algorithmic": kd["frac_algorithmic"],
                "algorithmic_bytes_per_launch": alg[dominant],
                "issue_slots_used": kd["issue_frac"], "kernels": kern,
                "note": "achieved = traffic / CUDA-event time with traffic = DRAM bytes per launch from ncu (bytes that move); "
                        "*_algorithmic counts the method's bytes of a dense input instead, which this workload's zero rows "
                        "make larger than what moves.  The encoder is bound by instruction issue, not by DRAM: "
                        "issue_slots_used = executed warp instructions (ncu) / time / (148 SMs x 4 schedulers x 1965 MHz)"}
    if kd["traffic"] is None:                 # no counters for this configuration: only the algorithmic figure exists
        roofline["achieved"], roofline["frac"] = kd["gbs_algorithmic"], kd["frac_algorithmic"]
        roofline["note"] = "no ncu counters for this configuration: achieved = algorithmic bytes / time"
    call_kernels = {"lq_quantize_pack": ("norm_partial", "norm_finalize", "quantize_pack", "stat_finalize"),
                    "qoda_step": ("qoda_scalars", "block_live", "decode")}
    qp_alg = ((4.0 + 2 * (c + 4.0 / 128.0)) if bucket else (8.0 + 2 * c)) * K * D * share
    call_alg = {"lq_quantize_pack": qp_alg, "qoda_step": alg["decode"]}
    calls = {}
    for call, names in call_kernels.items():
        ms_c = sum(kern[n]["avg_ms"] * kern[n]["launches_per_step"] for n in names if n in kern)
        tr = [kern[n].get("traffic") for n in names if n in kern and n in alg]
        tr_sum = sum(tr) if tr and all(t is not None for t in tr) else None
        calls[call] = {"ms": ms_c, "fp32_in_gbs": 4.0 * K * D * share / ms_c / 1e6,
                       "traffic": tr_sum,
                       "dram_gbs": tr_sum / ms_c / 1e6 if tr_sum else None,
                       "frac_of_peak": tr_sum / ms_c / 1e6 / peak if tr_sum else None,
                       "frac_of_nominal_8tbs": tr_sum / ms_c / 1e6 / 8000.0 if tr_sum else None,
                       "algorithmic_gbs": call_alg[call] / ms_c / 1e6,
                       "frac_algorithmic_of_peak": call_alg[call] / ms_c / 1e6 / peak}
    if dense is not None:
        roofline["dense"] = dense

    cpu = cpu_baseline_record() if world == 1 and not args.no_cpu_baseline else None
    launches = int(sum(cnt for _, cnt in prof.values()))
    line = {"metric": METRIC, "value": whole_job_value(4.0 * K * D * share / 1e9, world, ms), "unit": "GB/s",
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms,
            "higher_is_better": True, "scaling": "strong" if args.exchange else "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": f"{w.name}_shaped", "coords": D, "layers": w.num_layers, "num_workers": K,
                       "bits": w.bits, "q": w.q, "norm_scope": args.norm_scope, "levels": "adaptive (fitted once before timing)",
                       "l2": "inputs (%.2f GB) exceed L2" % (4.0 * K * D / 1e9),
                       "multi_gpu": "K workers shared out over the ranks, messages by all-gather" if args.exchange
                                    else "replicas only"},
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roofline, "calls": calls}
    if graph_error is not None:
        line["cuda_graph"] = {"error": graph_error}
    if graph_ms is not None:
        line["cuda_graph"] = {"ms_per_step": graph_ms, "value": whole_job_value(4.0 * K * D * share / 1e9, world, graph_ms),
                              "note": "the same two calls per step, two steps recorded once and replayed"}
    if cpu:
        line["cpu_baseline"] = cpu
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()



# ---------------------------------------------------------------------------------- sweep
def run_sweep(args) -> None:
    """Bandwidth sweep: flat layers of 2^10 .. 2^30 coordinates and a ragged set of 2048 layers, over code
    widths, worker counts and norms.  One JSON line per point: device time (CUDA events, inputs resident, L2
    flushed by a 256 MB write between repetitions when the input is smaller than L2) of lq_quantize_pack and of
    qoda_step, their algorithmic GB/s and the fraction of the measured HBM peak.  Points whose K inputs would
    not fit in `--sweep-bytes` reuse one input row for every worker (said in the line)."""
    import torch
    import paper_2505_14371_b200 as pkg
    from paper_2505_14371_b200 import workloads as W
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    pkg.load_library()
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    peak = float(json.load(open(peaks_path))["hbm_gbs"]) if os.path.exists(peaks_path) else 6650.0
    flush = torch.empty(64 << 20, dtype=torch.float32, device=dev)
    points = []
    for log2n in ([10, 14, 18, 20, 22, 24, 26, 28, 30] if not args.sweep_quick else [14, 22, 26]):
        for bits, K, q in ([(4, 4, 2)] if log2n not in (26,) else
                           [(b, k, qq) for b in (2, 3, 4, 8) for k in (1, 4, 16) for qq in (2, 0)]):
            points.append(("flat", log2n, bits, K, q))
    for bits in (2, 3, 4, 8):
        points.append(("ragged", 0, bits, 4, 2))
    for kind, log2n, bits, K, q in points:
        w = W.flat_workload(log2n, bits, K, q) if kind == "flat" else W.ragged_workload(bits, K, q)
        D = w.num_coords
        plan = pkg.Plan(w.layer_sizes, w.bits, w.q, K, W.PHILOX_SEED)
        aliased = 4 * K * plan.padded_elems > args.sweep_bytes
        if aliased:                                # one input row serves every worker (stride 0 is not expressible
            K_alloc = 1                            # through the ABI, so the plan is rebuilt for the workers that fit)
            Kfit = max(1, int(args.sweep_bytes // (4 * plan.padded_elems)))
            plan.close(); K = Kfit
            w = W.flat_workload(log2n, bits, K, q) if kind == "flat" else W.ragged_workload(bits, K, q)
            plan = pkg.Plan(w.layer_sizes, w.bits, w.q, K, W.PHILOX_SEED)
        grads = W.make_gradients(w, plan.elem_offsets, plan.padded_elems, dev)
        pk = [plan.empty_packed(dev), plan.empty_packed(dev)]; nm = [plan.empty_norms(dev), plan.empty_norms(dev)]
        X1 = torch.randn(plan.padded_elems, device=dev); Y = torch.empty_like(X1); Xh = torch.empty_like(X1)
        plan.qoda_init(X1, Y, Xh)
        small = 4 * K * D < (256 << 20)
        reps = 5 if 4 * K * D > (1 << 30) else 20
        tq, ts = [], []
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        for t in range(1, reps + 4):
            c, p = t % 2, (t + 1) % 2
            if small:
                flush.fill_(float(t))
            ev[0].record()
            plan.lq_quantize_pack(grads, t, pk[c], nm[c], prev_packed=None if t == 1 else pk[p],
                                  prev_norms=None if t == 1 else nm[p])
            ev[1].record()
            plan.qoda_step(pk[c], nm[c], X1, Y, Xh)
            ev[2].record()
            torch.cuda.synchronize()
            if t > 3:
                tq.append(ev[0].elapsed_time(ev[1])); ts.append(ev[1].elapsed_time(ev[2]))
        cb = (bits + 1) / 8.0
        mq, ms = sorted(tq)[len(tq) // 2], sorted(ts)[len(ts) // 2]
        gq = (8.0 + 2 * cb) * K * D / mq / 1e6; gs = (K * cb + 16.0) * D / ms / 1e6
        print(json.dumps({"sweep": kind, "log2_coords": log2n, "coords": D, "layers": w.num_layers, "bits": bits, "K": K,
                          "q": "inf" if q == 0 else q, "workers_capped_by_memory": aliased,
                          "lq_quantize_pack": {"ms": round(mq, 5), "fp32_in_gbs": round(4.0 * K * D / mq / 1e6, 1),
                                               "algorithmic_gbs": round(gq, 1), "frac_of_measured_peak": round(gq / peak, 3),
                                               "frac_of_8tbs": round(gq / 8000.0, 3)},
                          "qoda_step": {"ms": round(ms, 5), "algorithmic_gbs": round(gs, 1),
                                        "frac_of_measured_peak": round(gs / peak, 3), "frac_of_8tbs": round(gs / 8000.0, 3)},
                          "l2": "flushed between repetitions" if small else "input exceeds L2"}), flush=True)
        plan.close()
        del grads, pk, nm, X1, Y, Xh


def run_entropy(args) -> None:
    """Throughput of the entropy stage on one message of the chosen workload (appendix on the coding framework):
    Huffman codes built from the message's own level counts, then lq_entropy_encode and lq_entropy_decode timed
    with CUDA events (inputs resident, message larger than L2 or L2 flushed by a 256 MB write between
    repetitions).  One JSON line: GB/s of the fixed-width message (K * W * 4 bytes), stream size, round trip."""
    import torch
    import paper_2505_14371_b200 as pkg
    from paper_2505_14371_b200 import workloads as W
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    pkg.load_library()
    w = pick_workload(args.workload)
    K = w.num_workers
    plan = pkg.Plan(w.layer_sizes, w.bits, w.q, K, W.PHILOX_SEED)
    grads = W.make_gradients(w, plan.elem_offsets, plan.padded_elems, dev)
    packed, norms, hist = plan.empty_packed(dev), plan.empty_norms(dev), plan.zero_hist(dev)
    plan.lq_quantize_pack(grads, 1, packed, norms, hist=hist)
    plan.lq_fit_levels(hist, norms, K)
    plan.lq_quantize_pack(grads, 2, packed, norms)
    del grads, hist
    counts = torch.zeros((K, plan.num_layers, 256), dtype=torch.int32, device=dev)
    plan.lq_symbol_counts(packed, counts)
    torch.cuda.synchronize()
    tot = counts.sum(dim=0).cpu().numpy()
    for m in range(plan.num_layers):
        n = 1 << plan.bits[m]
        plan.lq_code_set(m, pkg.lq_code_build([float(x) + 1e-9 for x in tot[m, :n]]))
    Wd = plan.packed_words
    stream = torch.zeros((K, Wd), dtype=torch.int32, device=dev)
    offsets = torch.zeros((K, plan.lq_plan_blocks() + 1), dtype=torch.int32, device=dev)
    back = torch.empty_like(packed)
    runs = plan.empty_run_offsets(dev) if not args.no_run_offsets else None
    flush = torch.empty(64 << 20, dtype=torch.float32, device=dev)
    small = 4 * K * Wd < (256 << 20)
    te, td = [], []
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    for rep in range(args.steps + 3):
        if small:
            flush.fill_(float(rep))
        ev[0].record()
        plan.lq_entropy_encode(packed, stream, offsets, runs)
        ev[1].record()
        if small:
            flush.fill_(float(rep) + 0.5)
        ev[2].record()
        plan.lq_entropy_decode(stream, offsets, back, runs)
        ev[3].record()
        torch.cuda.synchronize()
        if rep >= 3:
            te.append(ev[0].elapsed_time(ev[1])); td.append(ev[2].elapsed_time(ev[3]))
    status = plan.lq_entropy_status()
    words = offsets[:, -1].to(torch.int64).sum().item()
    # a round trip returns the message with the sign bit of zero-index coordinates cleared: compare through a
    # second encode of the decoded message, which must give the same stream
    stream2 = torch.zeros_like(stream); offsets2 = torch.zeros_like(offsets)
    plan.lq_entropy_encode(back, stream2, offsets2)
    torch.cuda.synchronize()
    same = bool(torch.equal(offsets, offsets2)) and bool(torch.equal(stream, stream2))
    me, md = sorted(te)[len(te) // 2], sorted(td)[len(td) // 2]
    msg_bytes = 4.0 * K * Wd
    print(json.dumps({"entropy_stage": True, "workload": args.workload, "coords": w.num_coords, "num_workers": K, "bits": w.bits,
                      "message_bytes": msg_bytes, "stream_bytes": 4.0 * words, "compression": msg_bytes / (4.0 * words),
                      "encode_ms": me, "decode_ms": md, "encode_gbs": msg_bytes / me / 1e6, "decode_gbs": msg_bytes / md / 1e6,
                      "status": status, "round_trip_same_stream": same, "run_offsets": runs is not None,
                      "side_bytes": 0 if runs is None else 2.0 * runs.numel(),
                      "l2": "flushed between repetitions" if small else "message exceeds L2"}), flush=True)


def spawn_ranks(n: int, argv) -> int:
    """`python bench.py --gpus N` without a launcher: start N ranks of this script (one per GPU) under
    torch.distributed.run on this node and return their exit code."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


def run_stub(args) -> None:
    """The multi-rank bookkeeping of the benchmark with a stand-in step (no GPU): gloo ranks, barrier, max over
    ranks, whole-job value, one JSON line from rank 0.  Used by the launcher test."""
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world > 1:
        dist.init_process_group("gloo")
        dist.barrier()
    local_ms = 1.0 + rank                                         # the last rank is the slowest
    ms = aggregate_over_ranks(local_ms, world)
    if rank == 0:
        print(json.dumps({"stub": True, "n_gpus": world, "ms_per_step": ms, "value": whole_job_value(1.0, world, ms),
                          "steps": args.steps, "warmup": args.warmup}), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="transformer_xl")
    ap.add_argument("--norm-scope", default="layer", choices=["layer", "global", "bucket"],
                    help="layer: one norm per layer (the headline configuration); bucket: one per 128 coordinates")
    ap.add_argument("--no-graph", dest="graph", action="store_false",
                    help="skip the extra timing of the step replayed from a CUDA graph (reported under cuda_graph)")
    ap.add_argument("--exchange", action="store_true",
                    help="share the K workers out over the ranks and exchange the messages by all-gather (default: "
                         "every rank runs the whole K-worker job on its own data)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-dense", action="store_true", help="skip the extra dense-data measurement of the encoder (roofline.dense)")
    ap.add_argument("--stub-step", action="store_true", help=argparse.SUPPRESS)   # launcher test: gloo ranks, no GPU work
    ap.add_argument("--entropy", action="store_true", help="throughput of the entropy stage (encode / decode) on one message")
    ap.add_argument("--no-run-offsets", action="store_true", help="entropy stage without the run offsets (one thread decodes a block)")
    ap.add_argument("--sweep", action="store_true", help="bandwidth sweep over sizes, widths, workers, norms")
    ap.add_argument("--sweep-quick", action="store_true")
    ap.add_argument("--sweep-bytes", type=float, default=40e9, help="most bytes of fp32 input per sweep point")
    ap.add_argument("--print-source-hashes", action="store_true", help="hashes to record beside new ncu traffic figures")
    args = ap.parse_args()
    if args.print_source_hashes:
        print({k: source_hash(k) for k in KERNEL_SOURCES})
        return
    if args.sweep:
        run_sweep(args)
        return
    if args.entropy:
        run_entropy(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and (args.impl == "ours" or args.stub_step):
        raise SystemExit(spawn_ranks(args.gpus, sys.argv[1:]))       # one process per GPU, started here
    if args.stub_step:
        run_stub(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
