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


TRAFFIC_FILE = os.path.join(ROOT, "profiles", "dram_traffic.txt")


def algorithmic_dram_bytes(w: synth.Workload, kernel: str) -> float:
    """Bytes a launch must move through DRAM if every operand is read once and every result written once (valid
    rows only).  Used to scale DRAM counters captured on a small workload to the benchmarked one."""
    R, T, d, F, E = float(w.R), float(w.T), float(w.d), float(w.ffn), float(w.E_tgt)
    act_d, act_f, w_gu, w_d = R * d * 2, R * F * 2, E * 2 * F * d * 2, E * d * F * 2
    table = {
        "gemm_up_swiglu": act_d + w_gu + 3 * act_f, "gemm_down": act_f + w_d + act_d,
        "gemm_dH": act_d + w_d + 2 * act_f + 2 * act_f + 2 * ((w.ffn + 255) // 256) * R * 4, "gemm_dX": 2 * act_f + w_gu + act_d,
        "wgrad_down": act_d + act_f + 2 * w_d, "wgrad_gate_up": 2 * act_f + act_d + 2 * w_gu,
        "gather_X": (T + R) * d * 2, "combine_Y": (T + R) * d * 2, "gather_dY": (T + R) * d * 2, "reduce_dX": (T + R) * d * 2,
    }
    return table.get(kernel, 0.0)


def recorded_traffic(w: synth.Workload, kernel: str):
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of `kernel` on workload `w`.

    profiles/dram_traffic.txt holds one-pass ncu counters taken on a workload of a few GB (lines: workload kernel bytes
    source-tag).  A line for `w` itself is used as it stands; otherwise the small workload's figure is scaled by the
    ratio of the two workloads' algorithmic bytes (DRAM traffic of these kernels follows their operand and result sizes:
    the capture reads within a few per cent of the algorithmic bytes).  None when the CUDA sources have changed since
    the capture (other source tag) or there is no line for the kernel."""
    if not os.path.exists(TRAFFIC_FILE):
        return None
    tag = kernel_source_tag()
    scaled = None
    for line in open(TRAFFIC_FILE):
        parts = line.split()
        if len(parts) < 4 or line.startswith("#") or parts[1] != kernel or parts[3] != tag:
            continue
        if parts[0] == w.name:
            return float(parts[2])
        src = synth.WORKLOADS.get(parts[0])
        if src is not None and algorithmic_dram_bytes(src, kernel) > 0:
            scaled = float(parts[2]) * algorithmic_dram_bytes(w, kernel) / algorithmic_dram_bytes(src, kernel)
    return scaled


def plan_at_scale(dev, T=1 << 24, k=8, E=128, iters=5):
    """The plan build at a size where bytes, not launch latency, decide its time: uniform 8-bit ids, T*k = 2^27 slots.
    Algorithmic bytes: the ids read once, the two permutations written, counts and offsets written."""
    import torch
    from paper_2603_06626_b200 import binding
    layer = binding.GrouterLayer(T, 8, 8, E, k, device=str(dev), plan_only=True)
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
    by = 1.0 * R + 2.0 * R * 4 + (2 * E + 1) * 4
    return {"T": T, "k": k, "E": E, "ms": ms, "algorithmic_bytes": by, "gbs": by / (ms * 1e-3) / 1e9,
            "note": "bytes as defined for the plan: ids read once; the two kernels that read the ids move 1 byte per slot more"}


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
            "gbs": by / (ms * 1e-3) / 1e9,
            "gpu_launches_per_call": 1 if (E_src <= 256 and k <= 8) else 2}


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


def combine_ab_leg(dev, w, layer, idx, fm, gates, X, W_gu, W_d, rounds=5, per_round=3):
    """Forward pass with the combine as its own kernel against the combine folded into the down product's epilogue
    (GROUTER_FLAG_FUSED_COMBINE), interleaved in one process so that both see the same clocks."""
    import torch
    from paper_2603_06626_b200 import binding
    fused = binding.GrouterLayer(w.T, w.d, w.ffn, w.E_src, w.k, E_tgt=w.E_tgt, device=str(dev), flags=binding.FLAG_FUSED_COMBINE)
    Y = torch.empty_like(X)
    layer.plan(idx, fm)
    fused.plan(idx, fm)
    times = {"separate": [], "fused": []}
    for name, ly in (("separate", layer), ("fused", fused)):     # warm-up
        ly.forward(X, gates, W_gu, W_d, Y)
    torch.cuda.synchronize()
    for _ in range(rounds):
        for name, ly in (("separate", layer), ("fused", fused)):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(per_round):
                ly.forward(X, gates, W_gu, W_d, Y)
            e1.record()
            torch.cuda.synchronize()
            times[name].append(e0.elapsed_time(e1) / per_round)
    fused.check_status()
    fused.close()
    med = {k: statistics.median(v) for k, v in times.items()}
    return {"forward_ms_separate_combine": med["separate"], "forward_ms_fused_combine": med["fused"],
            "fused_over_separate": med["fused"] / med["separate"], "rounds": rounds, "forwards_per_round": per_round}


def run_expert_parallel(args, rank, local_rank, world, dev):
    """--parallelism ep: every rank keeps its own T tokens and 1/N of the experts; routed rows travel to the experts'
    rank and back (NCCL all-to-all into the receiver's own memory, split sizes from the plans' counts, which are gathered
    once ahead of the timed steps: the routing is known before the step).  With one rank the exchanges are local copies."""
    import torch
    import torch.distributed as dist
    from paper_2603_06626_b200 import binding, ep
    base = synth.WORKLOADS[args.workload]
    w = shard.rank_workload(base, rank)
    if base.E_tgt % world:
        raise SystemExit(f"--parallelism ep needs E_tgt ({base.E_tgt}) divisible by the number of ranks ({world})")
    li = synth.make_layer_inputs(w, with_weights=False)
    owner = np.arange(base.E_tgt) // (base.E_tgt // world)
    relabel, first = ep.relabel_experts(owner, world)
    fm = relabel if li.fold_map is None else relabel[li.fold_map]
    fold = torch.from_numpy(np.ascontiguousarray(fm, dtype=np.int32)).to(dev)

    def bf16(a):
        return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).to(dev).view(torch.bfloat16)

    mine = range(int(first[rank]), int(first[rank + 1]))          # identity relabelling: new id == old id
    W_gu = bf16(np.stack([synth.expert_W_gu(base, e) for e in mine]))
    W_d = bf16(np.stack([synth.expert_W_d(base, e) for e in mine]))
    idx, gates, X, dY = torch.from_numpy(li.idx).to(dev), bf16(li.gates), bf16(li.X), bf16(li.dY)
    r = ep.ExpertParallelRank(rank, world, w.T, w.d, w.ffn, w.E_src, w.E_tgt, w.k, first, device=str(dev))
    counts = r.plan(idx, fold)
    if world > 1:
        allc = [torch.empty_like(counts) for _ in range(world)]
        dist.all_gather(allc, counts)
        counts_all = torch.stack(allc).cpu().numpy()
    else:
        counts_all = counts.cpu().numpy()[None, :]
    r.set_counts(counts_all)
    Y, dX = torch.empty_like(X), torch.empty_like(X)
    dg = torch.empty((w.T, w.k), dtype=torch.float32, device=dev)
    dW_gu = torch.empty(W_gu.shape, dtype=torch.float32, device=dev)
    dW_d = torch.empty(W_d.shape, dtype=torch.float32, device=dev)

    def step():
        r.plan(idx, fold)
        r.run_step(X, dY, gates, W_gu, W_d, Y, dX, dg, dW_gu, dW_d)

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    for _ in range(max(args.warmup, 3)):
        step()
    shard.barrier(world)
    torch.cuda.synchronize()
    wall0 = time.time()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    wall1 = time.time()
    shard.barrier(world)
    clocks = sampler.stop(wall0, wall1) if rank == 0 else None
    ms_step = shard.max_over_ranks(e0.elapsed_time(e1), dev, world) / args.steps
    assert r.src.status() == 0 and (r.exp is None or r.exp.status() == 0)
    rows_out = int(r.layout["send_counts"].sum() - r.layout["send_counts"][rank])
    placement = None
    if rank == 0 and w.E_src <= 256 and w.T % 4096 == 0:
        # What the method's sample placement (Algorithm 1) is worth on a routing table whose samples lean towards one
        # node's experts each (synthetic stand-in; 8 nodes however many ranks this run has): rows that must cross nodes
        # when samples are dealt out in turn against each sample on its arg-max node.
        nodes, seq_len = 8, 4096
        own8 = (np.arange(w.E_src) * nodes // w.E_src).astype(np.int32)
        idx_s, _ = synth.make_idx_sample_affinity(w, seq_len, own8, nodes, boost=8.0)
        best, _ = ep.place_samples(torch.from_numpy(idx_s).to(dev), w.E_src, seq_len, own8, nodes)
        S = w.T // seq_len
        placement = {"nodes": nodes, "seq_len": seq_len, "samples": S, "routed_rows": int(idx_s.size),
                     "rows_crossing_nodes_dealt_in_turn": ep.rows_crossing_ranks(idx_s, own8, np.arange(S) % nodes, seq_len),
                     "rows_crossing_nodes_algorithm_1": ep.rows_crossing_ranks(idx_s, own8, best, seq_len),
                     "most_samples_on_one_node": int(np.bincount(best, minlength=nodes).max()),
                     "routing": "synthetic: each sample's home node's experts 8x as likely"}
    if rank == 0:
        peaks, peak_src = load_peaks()
        flops_rank = 18.0 * w.d * w.ffn * float(r.n_recv)
        line = {"metric": METRIC, "value": shard.job_tokens_per_sec(world, w.T, ms_step), "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "bf16", "data": "synthetic", "config": dict(workload_config(base, world), parallelism=f"ep{world}"),
                "clocks": clocks, "gpu_launches": int((3 + 4 + 5 + 3 + 7) * args.steps),
                "roofline": {"bound": "tensor", "achieved": flops_rank / (ms_step * 1e-3) / 1e12, "peak": peaks["bf16_tflops_sustained"],
                             "unit": "TFLOP/s", "frac": flops_rank / (ms_step * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"], "traffic": None,
                             "peak_source": f"{peak_src} cuBLAS bf16, sustained; the whole step (exchanges included) of rank 0's experts"},
                "exchange": {"rows_sent_to_other_ranks_per_direction": rows_out, "bytes_per_step": 4.0 * rows_out * w.d * 2,
                             "transfers_per_step": 4, "split_sizes": "from the plans' counts, gathered once before the timed steps"},
                "placement": placement}
        print(json.dumps(line))
    r.close()


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
        "plan_hist": ("byte", R * idb + 0.0), "plan_permute": ("byte", R * idb + 2.0 * R * 4), "plan_scan": ("byte", (2.0 * w.E_tgt + 1) * 4),
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


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] or [os.cpu_count() or 1])
    except Exception:
        return os.cpu_count() or 1


def oracle_sample_tokens_per_sec(w: synth.Workload, li, n_experts: int = 1):
    """The fp64 oracle, as it stands, on whole experts: forward and full backward (dX, dgates, and the expert's dW_gu,
    dW_d) of the tokens routed to the `n_experts` experts whose loads are closest to the median load, each expert's
    weights widened to fp64 before the clock starts.  The layer costs the same arithmetic per routed row whichever
    expert owns it, so tokens/s of the whole workload = (T * k / rows timed) ... / seconds, i.e. the timed rows
    extrapolated to all T * k routed rows.  Returns (tokens/s extrapolated, seconds, BLAS threads, description)."""
    from oracle import grouter_oracle as orc
    ids = orc.fold_ids(li.idx, li.fold_map).reshape(w.T, w.k)
    loads = np.bincount(ids.reshape(-1), minlength=w.E_tgt)
    nz = np.nonzero(loads)[0]
    order = nz[np.argsort(np.abs(loads[nz] - np.median(loads[nz])), kind="stable")]
    chosen = [int(e) for e in order[:n_experts]]
    cache = {}
    for e in chosen:                      # weights drawn and widened before the clock starts
        if li.W_gu is not None:
            cache[e] = (synth.bf16_bits_to_f64(li.W_gu[e]), synth.bf16_bits_to_f64(li.W_d[e]))
        else:
            cache[e] = (synth.bf16_bits_to_f64(synth.expert_W_gu(w, e)), synth.bf16_bits_to_f64(synth.expert_W_d(w, e)))
    weights = orc.Weights(getter=lambda e: cache[e], ffn=w.ffn)
    pairs_all = int(np.unique(np.arange(w.T, dtype=np.int64)[:, None] * w.E_tgt + ids).shape[0])    # (token, expert) evaluations of f_e
    pairs = 0
    dt = 0.0
    for e in chosen:
        hit = ids == e
        tok = np.nonzero(hit.any(axis=1))[0]
        # sub-problem: these tokens, one slot each on expert e carrying the token's coefficient r(x)_e (Eq. 1)
        idx_e = np.full((tok.shape[0], 1), e, dtype=np.int64)
        gates_e = np.where(hit[tok], synth.bf16_bits_to_f64(li.gates[tok]), 0.0).sum(axis=1, keepdims=True)
        X = synth.bf16_bits_to_f64(li.X[tok])
        dY = synth.bf16_bits_to_f64(li.dY[tok])
        t0 = time.perf_counter()
        orc.moe_forward(X, idx_e, gates_e, weights, w.E_tgt)
        orc.moe_backward(dY, X, idx_e, gates_e, weights, w.E_tgt, experts=[e])
        dt += time.perf_counter() - t0
        pairs += int(tok.shape[0])
    tokens_per_s = w.T / (dt * pairs_all / pairs)
    what = (f"fp64 numpy oracle on whole experts: the {len(chosen)} expert(s) of median load ({pairs} of the workload's {pairs_all} "
            f"(token, expert) evaluations), forward + full backward incl. the expert's weight gradients, weights widened outside "
            f"the clock; extrapolated to the whole workload (same arithmetic per evaluation)")
    return tokens_per_s, dt, blas_threads(), what


def run_reference(args):
    """Reference arm: the CPU oracle timed on the host cores, same metric and workload config."""
    rank, _, _ = shard.env_rank_world()
    if rank != 0:
        return
    w = synth.WORKLOADS[args.workload]
    li = synth.make_layer_inputs(w, with_weights=False)
    times = []
    threads = 1
    value = 0.0
    sample = ""
    for i in range(args.warmup + args.steps):
        v, dt, threads, sample = oracle_sample_tokens_per_sec(w, li, 1)
        if i >= args.warmup:
            times.append((v, dt))
    total = sum(dt for _, dt in times)
    value = sum(v * dt for v, dt in times) / total            # time-weighted: total tokens' worth of work / total seconds
    sample = "per step: " + sample
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
            "dw_allreduce_in_step": False,
            "l2": "working set (weights + expert-ordered activations, several GB) exceeds the 126 MB L2"
            if w.name in ("skewed", "large", "fine_fold", "small") else "fits L2: flushed between steps"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="large", choices=list(synth.WORKLOADS))
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--parallelism", default="dp", choices=["dp", "ep"],
                    help="dp: token-sharded replicas (default); ep: experts split over the ranks, routed rows exchanged")
    ap.add_argument("--dw-allreduce", action="store_true",
                    help="dp with more than one rank: all-reduce the weight gradients inside every timed step")
    ap.add_argument("--cpu-baseline-experts", type=int, default=12, help="whole experts the CPU baseline times")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-plan-scale", action="store_true")
    ap.add_argument("--no-isolated", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=0, help="steps of the end-to-end leg (0: as many as --steps)")
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
    if args.parallelism == "ep":
        run_expert_parallel(args, rank, local_rank, world, dev)
        if world > 1:
            dist.destroy_process_group()
        return

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
        if args.dw_allreduce and world > 1:       # the one collective data parallelism adds: summed weight gradients
            dist.all_reduce(dW_gu)
            dist.all_reduce(dW_d)

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
    # ---- the headline: K whole steps back to back, nothing but the step's own launches on the stream ----
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
    layer.check_status()
    ms_total = shard.max_over_ranks(ms_total, dev, world)
    ms_step = ms_total / args.steps
    value = shard.job_tokens_per_sec(world, w.T, ms_step)

    # ---- the per-kernel table: a pass of its own with an event pair around every launch (not part of `value`) ----
    # (with every kernel in line on the one stream: the event pairs then bracket one kernel each)
    n_table = min(args.steps, 10)
    layer.set_overlap(False)
    layer.timing_enable(len(binding.KERNEL_SLOTS) * n_table)
    for _ in range(n_table):
        step()
    per_kernel = layer.timing_read()
    layer.timing_enable(0)
    layer.check_status()
    # what running the backward pass's two bandwidth-bound kernels beside the GEMMs is worth: whole steps, interleaved
    overlap_ab = None
    if world == 1 and not args.no_isolated:
        t_ab = {True: [], False: []}
        for _ in range(3):
            for on in (True, False):
                layer.set_overlap(on)
                step()
                a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a0.record()
                for _ in range(5):
                    step()
                a1.record()
                torch.cuda.synchronize()
                t_ab[on].append(a0.elapsed_time(a1) / 5)
        overlap_ab = {"step_ms_beside_gemms": statistics.median(t_ab[True]), "step_ms_in_line": statistics.median(t_ab[False]),
                      "rounds": 3, "steps_per_round": 5}
    layer.set_overlap(True)
    # the plan build alone, back to back on the stream (its three launches are too short for event pairs around each)
    pe0, pe1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    pe0.record()
    for _ in range(50):
        layer.plan(idx, fm)
    pe1.record()
    torch.cuda.synchronize()
    plan_alone_ms = pe0.elapsed_time(pe1) / 50

    # ---- every kernel alone: 30 ms of idle time after each launch, so that none starts at the power cap ----
    isolated = None
    if world == 1 and not args.no_isolated:
        layer.set_overlap(False)
        layer.timing_gap(30000)
        layer.timing_enable(len(binding.KERNEL_SLOTS) * 3)
        for _ in range(3):
            step()
        isolated = layer.timing_read()
        layer.timing_enable(0)
        layer.timing_gap(0)
        layer.set_overlap(True)
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
    if args.e2e_steps <= 0:
        args.e2e_steps = args.steps
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
    traffic = recorded_traffic(w, dom)
    for name, ent in kernels.items():
        ent["traffic"] = recorded_traffic(w, name)
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
    plan_ms = (per_kernel["plan_hist"][0] + per_kernel["plan_scan"][0] + per_kernel["plan_permute"][0]) / max(n_timed, 1)
    plan = {"ms": plan_alone_ms, "ms_event_pairs_in_step": plan_ms, "launches": 3, "share_of_step": plan_alone_ms / ms_step,
            "value_plan_amortised": value * ms_step / (ms_step - plan_alone_ms) if ms_step > plan_alone_ms else None,
            "note": "tokens/s if the plan is built once and reused by many layers"}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warm,
        "ms_per_step": ms_step, "ms_per_step_median": step_ms[len(step_ms) // 2], "ms_per_step_best": step_ms[0], "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic", "config": dict(workload_config(base, world), dw_allreduce_in_step=bool(args.dw_allreduce and world > 1)), "clocks": clocks,
        "gpu_launches": int(sum(v[1] for v in per_kernel.values()) // max(n_timed, 1) * args.steps), "roofline": roofline, "kernels": kernels, "gemm_summary": summary, "plan": plan,
        "gemm_cycles": gemm_cycles, "overlap_ab": overlap_ab,
        "load_stats": synth.load_stats(li.idx, li.fold_map, w.E_tgt),
    }
    if e2e is not None:
        line["e2e"] = e2e
    if world == 1 and not args.no_isolated:
        line["combine_ab"] = combine_ab_leg(dev, w, layer, idx, fm, gates, X, W_gu, W_d)
    if world == 1 and not args.no_plan_scale:
        torch.cuda.synchronize()
        time.sleep(3.0)     # the step loop ran at the power cap; these short kernels are timed on a GPU that has settled
        for _ in range(5):
            layer.plan(idx, fm)
        pe0.record()
        for _ in range(50):
            layer.plan(idx, fm)
        pe1.record()
        torch.cuda.synchronize()
        line["plan"]["ms_alone_settled"] = pe0.elapsed_time(pe1) / 50
        line["plan"]["note_clocks"] = ("`ms`: 50 builds back to back right after the step loop, at the SM clock the power cap left; "
                                       "`ms_alone_settled`: the same after three idle seconds")
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
        v, dt, threads, what = oracle_sample_tokens_per_sec(w, li, args.cpu_baseline_experts)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle", "seconds": dt, "sample": what,
                                "extrapolated": True}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
