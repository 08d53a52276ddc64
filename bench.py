#!/usr/bin/env python
"""Benchmark of the routed SwiGLU expert layer under preemptive routing.

A step is one pass of the whole hot path over one batch: routing-plan build,
forward (gather, up/gate GEMM + SwiGLU, down GEMM, combine) and backward (dY
gather, dH GEMM + SwiGLU backward + d-gate, three weight-gradient GEMMs, dX
GEMM, dX reduce), all through the C ABI.  Metric: tokens per second of
fwd+bwd.  One JSON line is printed by rank 0.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload large] [--impl reference]

N > 1 (launched with torch.distributed.run): every rank owns its own batch of
the same shape (weak scaling over independent token shards, no collective on
the data path; the weight-gradient all-reduce of data parallelism belongs to
the optimizer step, outside the layer).  `--impl reference` times the fp64 CPU
oracle on the host cores for the same metric.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2603_06626_b200 import synth  # noqa: E402
from paper_2603_06626_b200 import shard  # noqa: E402

METRIC = "moe_layer_fwd_bwd_tokens_per_sec"
UNIT = "tokens/s"
GEMM_SLOTS = ["gemm_up_swiglu", "gemm_down", "gemm_dH", "wgrad_down", "gemm_dX", "wgrad_gate_up"]
MOVER_SLOTS = ["gather_X", "combine_Y", "gather_dY", "reduce_dX"]
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def kernel_source_tag() -> str:
    """Short hash of the CUDA sources (comments and blank space left out): DRAM counters taken with other code are not
    reported."""
    import hashlib
    import re
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2603_06626_b200", "csrc")
    for name in sorted(os.listdir(csrc)):
        with open(os.path.join(csrc, name)) as f:
            code = re.sub(r"//[^\n]*", "", f.read())
        h.update(name.encode() + b"\0" + "".join(code.split()).encode())
    return h.hexdigest()[:12]


def recorded_traffic(workload: str, kernel: str):
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu capture summarised in
    profiles/dram_traffic.txt, or None when there is no capture of this kernel on this workload with this build."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    if not os.path.exists(path):
        return None
    tag = kernel_source_tag()
    for line in open(path):
        parts = line.split()
        if len(parts) >= 4 and not line.startswith("#") and parts[0] == workload and parts[1] == kernel and parts[3] == tag:
            return float(parts[2])
    return None


def plan_at_scale(dev, T=1 << 22, k=8, E=128, iters=5):
    """The plan build at a size where bytes, not launch latency, decide its time: uniform ids, T*k = 2^25 slots.
    Algorithmic bytes: ids read twice (histogram pass, permutation pass) and the two permutations written."""
    import torch
    from paper_2603_06626_b200 import binding
    layer = binding.GrouterLayer(T, 8, 8, E, k, device=str(dev))
    g = torch.Generator(device=dev)
    g.manual_seed(7)
    idx = torch.randint(0, E, (T, k), dtype=torch.uint8, device=dev, generator=g)
    for _ in range(2):
        layer.plan(idx)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        layer.plan(idx)
    e1.record()
    torch.cuda.synchronize()
    layer.check_status()
    ms = e0.elapsed_time(e1) / iters
    R = T * k
    assert int(layer.counts.sum().item()) == R
    layer.close()
    by = 2.0 * R + 2.0 * R * 4
    return {"T": T, "k": k, "E": E, "ms": ms, "algorithmic_bytes": by, "gbs": by / (ms * 1e-3) / 1e9}


def router_head_leg(dev, T=32768, d_h=512, E_src=128, E_tgt=128, k=8, iters=20):
    """The step before the plan (Eq. 2): scores of a 512-wide router over 128 experts, top-8, softmax, uint8/bf16 record.
    Synthetic hidden states and score layer.  Algorithmic bytes: H and W_s read, the 3k-byte record written."""
    import torch
    from paper_2603_06626_b200 import binding
    lib = binding.load_library()
    g = torch.Generator(device=dev)
    g.manual_seed(11)
    H = torch.randn((T, d_h), device=dev, generator=g).to(torch.bfloat16)
    W = (torch.randn((E_src, d_h), device=dev, generator=g) / d_h ** 0.5).to(torch.bfloat16)
    idx = torch.empty((T, k), dtype=torch.uint8, device=dev)
    gates = torch.empty((T, k), dtype=torch.bfloat16, device=dev)
    ws = torch.empty(lib.grouter_route_workspace_bytes(T, E_src, E_tgt), dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    st = torch.cuda.current_stream().cuda_stream

    def call():
        rc = lib.grouter_route(H.data_ptr(), W.data_ptr(), None, T, d_h, E_src, E_tgt, k, binding.NORM_SOFTMAX, idx.data_ptr(),
                               gates.data_ptr(), None, ws.data_ptr(), status.data_ptr(), st)
        assert rc == 0, rc

    for _ in range(3):
        call()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        call()
    e1.record()
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ms = e0.elapsed_time(e1) / iters
    by = T * d_h * 2.0 + E_src * d_h * 2.0 + 3.0 * k * T
    return {"T": T, "d_h": d_h, "E": E_src, "k": k, "ms": ms, "tokens_per_s": T / (ms * 1e-3), "algorithmic_bytes": by,
            "gbs": by / (ms * 1e-3) / 1e9, "gpu_launches_per_call": 2}


def routing_stats_leg(dev, idx, E, seq_len=4096, n_nodes=8, iters=20):
    """Loads, co-activation matrix, affinity vectors, MaxVio and Algorithm-1 placement over the step's routing table.
    Algorithmic bytes: the ids read once, the statistics written."""
    import torch
    from paper_2603_06626_b200 import binding
    lib = binding.load_library()
    T, k = idx.shape
    S = T // seq_len
    i32 = dict(dtype=torch.int32, device=dev)
    node = (torch.arange(E, device=dev, dtype=torch.int32) % n_nodes).contiguous()
    loads, coact = torch.empty(E, **i32), torch.empty((E, E), **i32)
    phi, mv = torch.empty((S, E), dtype=torch.float32, device=dev), torch.empty(1, dtype=torch.float32, device=dev)
    lt, bn, status = torch.empty((S, n_nodes), **i32), torch.empty(S, **i32), torch.zeros(1, **i32)
    st = torch.cuda.current_stream().cuda_stream

    def call():
        rc = lib.grouter_routing_stats(idx.data_ptr(), binding.IDX_U8, T, k, E, seq_len, node.data_ptr(), n_nodes, loads.data_ptr(),
                                       coact.data_ptr(), phi.data_ptr(), mv.data_ptr(), lt.data_ptr(), bn.data_ptr(), status.data_ptr(), st)
        assert rc == 0, rc

    for _ in range(3):
        call()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        call()
    e1.record()
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and int(loads.sum().item()) == T * k
    ms = e0.elapsed_time(e1) / iters
    by = T * k * 1.0 + 4.0 * (E + E * E + S * E + S * n_nodes + S)
    return {"T": T, "k": k, "E": E, "seq_len": seq_len, "n_nodes": n_nodes, "ms": ms, "tokens_per_s": T / (ms * 1e-3),
            "algorithmic_bytes": by, "gbs": by / (ms * 1e-3) / 1e9, "max_vio": float(mv.item())}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return p, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def kernel_work(w: synth.Workload, counts: np.ndarray, chunk_rows: int):
    """Algorithmic work per launch: FLOPs over valid routed rows only (padding earns nothing) for the
    GEMMs; bytes (T + R) * d * 2 for the row movers; plan: ids read, two permutations written; the zero-fill
    writes the fp32 gradients of the experts whose rows are contracted in several chunks (more than
    `chunk_rows` padded rows)."""
    R, d, F, T = w.R, w.d, w.ffn, w.T
    n_split = int((((counts + 127) // 128) * 128 > chunk_rows).sum())
    dF = 2.0 * R * d * F
    idb = 1 if w.E_src <= 256 else 4
    return {
        "gemm_up_swiglu": ("flop", 2 * dF), "gemm_down": ("flop", dF), "gemm_dH": ("flop", dF), "wgrad_down": ("flop", dF),
        "gemm_dX": ("flop", 2 * dF), "wgrad_gate_up": ("flop", 2 * dF),
        "gather_X": ("byte", (T + R) * d * 2.0), "combine_Y": ("byte", (T + R) * d * 2.0),
        "gather_dY": ("byte", (T + R) * d * 2.0), "reduce_dX": ("byte", (T + R) * d * 2.0),
        "plan_hist": ("byte", R * idb + 0.0), "plan_permute": ("byte", R * idb + 2.0 * R * 4),
        "zero_split_dW": ("byte", n_split * 3.0 * d * F * 4),
    }


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi.  Started before the warm-up (nvidia-smi takes a
    while to come up); only samples whose timestamp falls inside the timed region are kept."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.proc = None
        self.idx = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "50",
                                          "-i", str(self.idx)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self, t_begin: float, t_end: float):
        """t_begin/t_end: time.time() at the two ends of the timed region."""
        import datetime
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.1)
        self.proc.terminate()
        try:
            text, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            return out
        sm, mx, pw = [], [], []
        reasons = set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in text.strip().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                if ts < t_begin or ts > t_end + 0.05:
                    continue
                sm.append(float(parts[1])); mx.append(float(parts[2])); pw.append(float(parts[3]))
            except ValueError:
                continue
            for n, v in zip(names, parts[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), power_w_max=max(pw), reasons=sorted(reasons), samples=len(sm))
        return out


def oracle_sample_tokens_per_sec(w: synth.Workload, li, n_tokens: int):
    """The fp64 oracle, as it stands, on the first n_tokens tokens of the workload (full fwd + bwd incl. every
    expert's weight gradients for those tokens).  Returns (tokens/s, seconds, threads)."""
    from oracle import grouter_oracle as orc
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] or [os.cpu_count() or 1])
    except Exception:
        threads = os.cpu_count() or 1
    sub = slice(0, n_tokens)
    X = synth.bf16_bits_to_f64(li.X[sub]); dY = synth.bf16_bits_to_f64(li.dY[sub]); gates = synth.bf16_bits_to_f64(li.gates[sub])
    idx = li.idx[sub]
    if li.W_gu is not None:
        getter = lambda e: (synth.bf16_bits_to_f64(li.W_gu[e]), synth.bf16_bits_to_f64(li.W_d[e]))  # noqa: E731
    else:
        cache = {}

        def getter(e):
            if e not in cache:
                cache[e] = (synth.expert_W_gu(w, e), synth.expert_W_d(w, e))
            return synth.bf16_bits_to_f64(cache[e][0]), synth.bf16_bits_to_f64(cache[e][1])
        used = np.unique(orc.fold_ids(idx, li.fold_map))
        for e in used:           # draw the weights before the clock starts
            getter(int(e))
    weights = orc.Weights(getter=getter, ffn=w.ffn)
    used = [int(e) for e in np.unique(orc.fold_ids(idx, li.fold_map))]
    t0 = time.perf_counter()
    orc.moe_forward(X, idx, gates, weights, w.E_tgt, li.fold_map)
    orc.moe_backward(dY, X, idx, gates, weights, w.E_tgt, li.fold_map, experts=used)
    dt = time.perf_counter() - t0
    return n_tokens / dt, dt, threads


def run_reference(args):
    """Reference arm: the CPU oracle timed on the host cores, same metric and workload config."""
    rank, _, _ = shard.env_rank_world()
    if rank != 0:
        return
    w = synth.WORKLOADS[args.workload]
    li = synth.make_layer_inputs(w, with_weights=False)
    n = args.ref_tokens
    times = []
    threads = 1
    for i in range(args.warmup + args.steps):
        _, dt, threads = oracle_sample_tokens_per_sec(w, li, n)
        if i >= args.warmup:
            times.append(dt)
    total = sum(times)
    value = n * len(times) / total
    sample = f"first {n} tokens of the workload per step (all their experts, fwd + full bwd), fp64 numpy"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, args.gpus),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_config(w: synth.Workload, n_gpus: int):
    return {"workload": w.name, "T": w.T, "d": w.d, "ffn": w.ffn, "E_src": w.E_src, "E_tgt": w.E_tgt, "k": w.k, "load": w.load,
            "zipf_s": w.zipf_s, "tokens_per_gpu": w.T, "global_tokens": w.T * n_gpus, "parallelism": f"dp{n_gpus}",
            "l2": "working set (weights + expert-ordered activations, several GB) exceeds the 126 MB L2"
            if w.name in ("skewed", "large", "fine_fold", "small") else "fits L2: flushed between steps"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="large", choices=list(synth.WORKLOADS))
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--ref-tokens", type=int, default=2, help="tokens per step of the reference arm's oracle sample")
    ap.add_argument("--cpu-baseline-tokens", type=int, default=48)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-plan-scale", action="store_true")
    ap.add_argument("--no-isolated", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=10)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist
    from paper_2603_06626_b200 import binding

    rank, local_rank, world = shard.env_rank_world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    warm = max(args.warmup, 3)

    base = synth.WORKLOADS[args.workload]
    w = shard.rank_workload(base, rank)
    li = synth.make_layer_inputs(w, threads=min(16, os.cpu_count() or 1))

    def bf16(a):
        return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).to(dev).view(torch.bfloat16)

    layer = binding.GrouterLayer(w.T, w.d, w.ffn, w.E_src, w.k, E_tgt=w.E_tgt, device=str(dev), host_staging=not args.no_e2e)
    idx = torch.from_numpy(li.idx).to(dev)
    fm = None if li.fold_map is None else torch.from_numpy(li.fold_map).to(dev)
    gates, X, dY = bf16(li.gates), bf16(li.X), bf16(li.dY)
    W_gu, W_d = bf16(li.W_gu), bf16(li.W_d)
    Y, dX = torch.empty_like(X), torch.empty_like(X)
    dW_gu = torch.empty(W_gu.shape, dtype=torch.float32, device=dev)
    dW_d = torch.empty(W_d.shape, dtype=torch.float32, device=dev)
    dgates = torch.empty((w.T, w.k), dtype=torch.float32, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if w.name == "tiny" else None

    def step():
        if flush is not None:
            flush.zero_()
        layer.plan(idx, fm)
        layer.forward(X, gates, W_gu, W_d, Y)
        layer.backward(dY, X, gates, W_gu, W_d, dX, dW_gu, dW_d, dgates)

    def barrier():
        shard.barrier(world)

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    for _ in range(warm):
        step()
    layer.check_status()
    barrier()
    torch.cuda.synchronize()
    layer.timing_enable(len(binding.KERNEL_SLOTS) * args.steps)
    wall0 = time.time()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps - 1)]   # between steps: median / best step
    ev0.record()
    for i in range(args.steps):
        step()
        if i < args.steps - 1:
            marks[i].record()
    ev1.record()
    torch.cuda.synchronize()
    edges = [ev0] + marks + [ev1]
    step_ms = sorted(edges[i].elapsed_time(edges[i + 1]) for i in range(args.steps))
    wall1 = time.time()
    barrier()
    ms_total = ev0.elapsed_time(ev1)
    clocks = sampler.stop(wall0, wall1) if rank == 0 else None
    per_kernel = layer.timing_read()
    layer.timing_enable(0)
    layer.check_status()
    ms_total = shard.max_over_ranks(ms_total, dev, world)
    ms_step = ms_total / args.steps
    value = shard.job_tokens_per_sec(world, w.T, ms_step)

    # ---- every kernel alone: 30 ms of idle time after each launch, so that none starts at the power cap ----
    isolated = None
    if world == 1 and not args.no_isolated:
        layer.timing_gap(30000)
        layer.timing_enable(len(binding.KERNEL_SLOTS) * 3)
        for _ in range(3):
            step()
        isolated = layer.timing_read()
        layer.timing_enable(0)
        layer.timing_gap(0)
        layer.check_status()

    # ---- where the issuers' cycles go (a few steps with the accounting on; not part of any timed number) ----
    gemm_cycles = None
    if world == 1 and not args.no_isolated:
        layer.gemm_cycles_enable(True)
        step()
        layer.gemm_cycles_read()
        for _ in range(5):
            step()
        raw = layer.gemm_cycles_read()
        layer.gemm_cycles_enable(False)
        layer.check_status()
        gemm_cycles = {}
        for name, c in raw.items():
            if c["k_steps"] > 0 and c["cycles"] > 0:
                gemm_cycles[name] = {"cycles_per_k_step": c["cycles"] / c["k_steps"], "tensor_core_cycles_per_k_step": 512,
                                     "wait_operands_frac": c["wait_operands"] / c["cycles"],
                                     "wait_accumulator_frac": c["wait_accumulator"] / c["cycles"],
                                     "tiles_per_pair_per_launch": c["tiles"] / 5.0 / max(1, torch.cuda.get_device_properties(dev).multi_processor_count // 2)}

    # ---- end to end: host buffers in, host results out, every step ----
    e2e = None
    if not args.no_e2e:
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()  # noqa: E731
        # two sets of pinned host buffers, used alternately: one step stays in flight while the host reads the previous one
        host = []
        for _ in range(2):
            host.append(dict(idx=pin(li.idx), gates=pin(li.gates.view(np.int16)), X=pin(li.X.view(np.int16)), dY=pin(li.dY.view(np.int16)),
                             Y=torch.empty((w.T, w.d), dtype=torch.int16).pin_memory(),
                             dX=torch.empty((w.T, w.d), dtype=torch.int16).pin_memory(),
                             dg=torch.empty((w.T, w.k), dtype=torch.float32).pin_memory()))
        idx_h, gates_h, X_h, dY_h, Y_h, dX_h, dg_h = (host[0][k] for k in ("idx", "gates", "X", "dY", "Y", "dX", "dg"))

        def e2e_step(i):
            h = host[i & 1]
            layer.step_host(h["idx"], h["gates"], h["X"], h["dY"], fm, W_gu, W_d, h["Y"], h["dX"], h["dg"], dW_gu, dW_d)
            layer.host_wait(1)          # the previous step's Y, dX, dgates are on the host now and may be read

        for i in range(2):
            e2e_step(i)
        layer.host_wait(0)
        barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(args.e2e_steps):
            e2e_step(i)
        layer.host_wait(0)              # every timed step's results have landed
        e1.record()
        torch.cuda.synchronize()
        barrier()
        ms_e2e = e0.elapsed_time(e1)
        ms_e2e = shard.max_over_ranks(ms_e2e, dev, world)
        layer.check_status()
        h2d = idx_h.numel() * idx_h.element_size() + gates_h.numel() * 2 + X_h.numel() * 2 + dY_h.numel() * 2
        d2h = Y_h.numel() * 2 + dX_h.numel() * 2 + dg_h.numel() * 4
        e2e = {"value": shard.job_tokens_per_sec(world, w.T, ms_e2e / args.e2e_steps), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": args.e2e_steps,
               "note": "idx, gates, X, dY copied from pinned host memory and Y, dX, dgates copied back every step "
                       "(grouter_moe_step_host, copies on their own streams overlapping the neighbouring steps' compute, one step "
                       "in flight); weights and weight gradients stay on the device"}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel, and the per-kernel table ----
    peaks, peak_src = load_peaks()
    work = kernel_work(w, layer.counts.cpu().numpy().astype(np.int64), layer.wgrad_chunk_rows())
    kernels = {}
    for name, (ms, n) in per_kernel.items():
        if n == 0:
            continue
        kind, amount = work[name]
        avg_s = ms / n * 1e-3
        ent = {"launches": n, "avg_ms": ms / n, "share": ms / sum(v[0] for v in per_kernel.values())}
        if kind == "flop":
            ent["tflops"] = amount / avg_s / 1e12
            ent["frac_of_sustained"] = ent["tflops"] / peaks["bf16_tflops_sustained"]
            ent["frac_of_burst"] = ent["tflops"] / peaks["bf16_tflops"]
        else:
            ent["gbs"] = amount / avg_s / 1e9
            ent["frac_of_hbm"] = ent["gbs"] / peaks["hbm_gbs"]
        if isolated is not None and isolated.get(name, (0.0, 0))[1] > 0:
            iso_s = isolated[name][0] / isolated[name][1] * 1e-3
            ent["alone_ms"] = iso_s * 1e3
            if kind == "flop":
                ent["alone_tflops"] = amount / iso_s / 1e12
                ent["alone_frac_of_burst"] = ent["alone_tflops"] / peaks["bf16_tflops"]
            else:
                ent["alone_gbs"] = amount / iso_s / 1e9
                ent["alone_frac_of_hbm"] = ent["alone_gbs"] / peaks["hbm_gbs"]
        kernels[name] = ent
    dom = max(GEMM_SLOTS, key=lambda k: per_kernel[k][0])
    traffic = recorded_traffic(w.name, dom)
    for name, ent in kernels.items():
        ent["traffic"] = recorded_traffic(w.name, name)
    roofline = {"kernel": dom, "bound": "tensor", "achieved": kernels[dom]["tflops"], "peak": peaks["bf16_tflops_sustained"],
                "unit": "TFLOP/s", "frac": kernels[dom]["tflops"] / peaks["bf16_tflops_sustained"], "traffic": traffic,
                "peak_source": f"{peak_src} cuBLAS bf16, sustained (kernel timed inside a long step); burst peak "
                               f"{peaks['bf16_tflops']} gives frac {kernels[dom]['tflops'] / peaks['bf16_tflops']:.3f}"}
    if "alone_tflops" in kernels[dom]:
        roofline["alone"] = {"achieved": kernels[dom]["alone_tflops"], "peak": peaks["bf16_tflops"], "frac": kernels[dom]["alone_frac_of_burst"],
                             "note": "the same kernel timed alone (30 ms idle after every launch) against the burst peak"}
    gemm_ms = sum(per_kernel[k][0] for k in GEMM_SLOTS)
    gemm_flops = sum(work[k][1] * per_kernel[k][1] for k in GEMM_SLOTS)
    summary = {"all_gemms_tflops": gemm_flops / (gemm_ms * 1e-3) / 1e12,
               "all_gemms_frac_of_burst": gemm_flops / (gemm_ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
               "step_flops": 18.0 * w.d * w.ffn * w.R}
    # one routing plan can serve every layer of the model, forward and backward (the router runs before the model):
    # the same step with the plan's two launches left out of the time
    n_timed = per_kernel["gemm_up_swiglu"][1]
    plan_ms = (per_kernel["plan_hist"][0] + per_kernel["plan_permute"][0]) / max(n_timed, 1)
    plan = {"ms": plan_ms, "share_of_step": plan_ms / ms_step,
            "value_plan_amortised": value * ms_step / (ms_step - plan_ms) if ms_step > plan_ms else None,
            "note": "tokens/s if the plan is built once and reused by many layers"}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warm,
        "ms_per_step": ms_step, "ms_per_step_median": step_ms[len(step_ms) // 2], "ms_per_step_best": step_ms[0], "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic", "config": workload_config(base, world), "clocks": clocks,
        "gpu_launches": int(sum(v[1] for v in per_kernel.values())), "roofline": roofline, "kernels": kernels, "gemm_summary": summary, "plan": plan,
        "gemm_cycles": gemm_cycles,
        "load_stats": synth.load_stats(li.idx, li.fold_map, w.E_tgt),
    }
    if e2e is not None:
        line["e2e"] = e2e
    if world == 1 and not args.no_plan_scale:
        layer.close()
        ps = plan_at_scale(dev)
        ps["frac_of_hbm"] = ps["gbs"] / peaks["hbm_gbs"]
        line["plan_scaled"] = ps
        rh = router_head_leg(dev)
        rh["frac_of_hbm"] = rh["gbs"] / peaks["hbm_gbs"]
        line["router_head"] = rh
        if w.E_src <= 256 and w.T % 4096 == 0:
            line["routing_stats"] = routing_stats_leg(dev, idx, w.E_src)
    if world == 1 and not args.no_cpu_baseline:
        v, dt, threads = oracle_sample_tokens_per_sec(w, li, args.cpu_baseline_tokens)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle", "seconds": dt,
                                "sample": f"first {args.cpu_baseline_tokens} tokens of the workload (all their experts, fwd + full bwd), "
                                          "fp64 numpy oracle"}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
