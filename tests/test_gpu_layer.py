"""Forward/backward parity of the CUDA path against the fp64 oracle.

Bar: relative Frobenius error <= 1e-2 per tensor (bf16 storage, fp32 accumulate
against an unrounded fp64 oracle); experts without slots must give exact zeros.
Beside every tensor-level ratio there is a per-row bound (one token's row of Y,
dX, dgates; one output row of a checked expert's dW): row error <= 3e-2 of the
row's norm (floored at the tensor's rms row norm), so that a fault confined to
one tile cannot hide inside a tensor-wide norm.
Small workloads are compared in full; the large ones on >= 1024 sampled tokens
(Y, dX, dgates) and on the heaviest, the lightest non-empty, every empty and
four seeded-random experts (dW_gu, dW_d), each compared element by element.
"""
import numpy as np
import pytest
import torch

from oracle import grouter_oracle as orc
from paper_2603_06626_b200 import synth
from tests.gpu_util import bits_to_bf16, to_dev

pytestmark = pytest.mark.gpu
TOL = 1e-2
ROW_TOL = 3e-2


def rows_ok(name, got, want):
    worst = float(orc.rel_rows(got, want).max()) if np.asarray(want).size else 0.0
    assert worst < ROW_TOL, f"{name}: worst row error {worst:.3e}"
    return worst


def run_gpu(w, li, gate_f32=False, idx_i32=False, flags=0):
    """One plan + fwd + bwd through the C ABI.  Returns device tensors."""
    from paper_2603_06626_b200 import binding
    layer = binding.GrouterLayer(w.T, w.d, w.ffn, w.E_src, w.k, E_tgt=w.E_tgt,
                                 idx_dtype=binding.IDX_I32 if idx_i32 else binding.IDX_U8,
                                 gate_dtype=binding.GATE_F32 if gate_f32 else binding.GATE_BF16, flags=flags)
    idx = to_dev(li.idx.astype(np.int32) if idx_i32 else li.idx)
    fm = None if li.fold_map is None else to_dev(li.fold_map)
    gates = bits_to_bf16(li.gates)
    if gate_f32:
        gates = gates.float()
    X, dY = bits_to_bf16(li.X), bits_to_bf16(li.dY)
    W_gu, W_d = bits_to_bf16(li.W_gu), bits_to_bf16(li.W_d)
    layer.plan(idx, fm)
    Y = layer.forward(X, gates, W_gu, W_d)
    dX, dW_gu, dW_d, dgates = layer.backward(dY, X, gates, W_gu, W_d)
    layer.check_status()
    out = dict(Y=Y, dX=dX, dW_gu=dW_gu, dW_d=dW_d, dgates=dgates, counts=layer.counts.cpu().numpy())
    layer.close()
    return out


def oracle_inputs(li):
    w = li.w
    X = synth.bf16_bits_to_f64(li.X)
    dY = synth.bf16_bits_to_f64(li.dY)
    gates = synth.bf16_bits_to_f64(li.gates)
    if li.W_gu is not None:
        weights = orc.Weights(getter=lambda e: (synth.bf16_bits_to_f64(li.W_gu[e]), synth.bf16_bits_to_f64(li.W_d[e])), ffn=w.ffn)
    else:
        weights = orc.Weights(getter=lambda e: (synth.bf16_bits_to_f64(synth.expert_W_gu(w, e)),
                                                synth.bf16_bits_to_f64(synth.expert_W_d(w, e))), ffn=w.ffn)
    return X, dY, gates, weights


def f64(t):
    return t.detach().to(torch.float64).cpu().numpy()


def check_full(w, li, out):
    X, dY, gates, weights = oracle_inputs(li)
    Y = orc.moe_forward(X, li.idx, gates, weights, w.E_tgt, li.fold_map)
    dX, dgates, dW = orc.moe_backward(dY, X, li.idx, gates, weights, w.E_tgt, li.fold_map)
    errs = {"Y": orc.rel_frobenius(f64(out["Y"]), Y), "dX": orc.rel_frobenius(f64(out["dX"]), dX),
            "dgates": orc.rel_frobenius(f64(out["dgates"]), dgates)}
    dWgu = np.stack([dW[e][0] for e in range(w.E_tgt)])
    dWd = np.stack([dW[e][1] for e in range(w.E_tgt)])
    errs["dW_gu"] = orc.rel_frobenius(f64(out["dW_gu"]), dWgu)
    errs["dW_d"] = orc.rel_frobenius(f64(out["dW_d"]), dWd)
    rows = {"Y": rows_ok("Y", f64(out["Y"]), Y), "dX": rows_ok("dX", f64(out["dX"]), dX),
            "dgates": rows_ok("dgates", f64(out["dgates"]), dgates), "dW": 0.0}
    for e in range(w.E_tgt):
        if out["counts"][e] == 0:
            assert not out["dW_gu"][e].any() and not out["dW_d"][e].any(), f"expert {e} has no slot: dW must be exact zeros"
        else:
            assert orc.rel_frobenius(f64(out["dW_gu"][e]), dW[e][0]) < TOL, f"dW_gu[{e}]"
            assert orc.rel_frobenius(f64(out["dW_d"][e]), dW[e][1]) < TOL, f"dW_d[{e}]"
            rows["dW"] = max(rows["dW"], rows_ok(f"dW_gu[{e}]", f64(out["dW_gu"][e]), dW[e][0]),
                             rows_ok(f"dW_d[{e}]", f64(out["dW_d"][e]), dW[e][1]))
    errs["worst_row"] = max(rows.values())
    for t in out.values():
        if torch.is_tensor(t):
            assert torch.isfinite(t).all()
    assert max(v for n, v in errs.items() if n != "worst_row") < TOL, errs
    return errs


def check_sampled(w, li, out, n_tokens, experts):
    X, dY, gates, weights = oracle_inputs(li)
    rng = np.random.default_rng(1234 + w.seed)
    tokens = np.sort(rng.choice(w.T, size=min(n_tokens, w.T), replace=False))
    Y = orc.moe_forward(X, li.idx, gates, weights, w.E_tgt, li.fold_map, tokens=tokens)
    dX, dgates = orc.moe_backward_tokens(dY, X, li.idx, gates, weights, w.E_tgt, li.fold_map, tokens=tokens)
    tk = torch.from_numpy(tokens).to(out["Y"].device)
    errs = {"Y": orc.rel_frobenius(f64(out["Y"][tk]), Y), "dX": orc.rel_frobenius(f64(out["dX"][tk]), dX),
            "dgates": orc.rel_frobenius(f64(out["dgates"][tk]), dgates)}
    worst = max(rows_ok("Y", f64(out["Y"][tk]), Y), rows_ok("dX", f64(out["dX"][tk]), dX),
                rows_ok("dgates", f64(out["dgates"][tk]), dgates))
    for e in experts:
        dWgu, dWd = orc.moe_backward_expert(dY, X, li.idx, gates, weights, w.E_tgt, int(e), li.fold_map)
        if out["counts"][e] == 0:
            assert not dWgu.any() and not dWd.any()
            assert not out["dW_gu"][e].any() and not out["dW_d"][e].any()
        else:
            errs[f"dW_gu[{e}]"] = orc.rel_frobenius(f64(out["dW_gu"][e]), dWgu)
            errs[f"dW_d[{e}]"] = orc.rel_frobenius(f64(out["dW_d"][e]), dWd)
            worst = max(worst, rows_ok(f"dW_gu[{e}]", f64(out["dW_gu"][e]), dWgu), rows_ok(f"dW_d[{e}]", f64(out["dW_d"][e]), dWd))
    for name in ("Y", "dX", "dgates", "dW_gu", "dW_d"):
        assert torch.isfinite(out[name]).all(), name
    assert max(errs.values()) < TOL, errs
    errs["worst_row"] = worst
    return errs


def pick_experts(counts, n_random, seed):
    """heaviest, lightest non-empty, every empty one, and a few random ones"""
    nz = np.nonzero(counts)[0]
    chosen = {int(nz[np.argmax(counts[nz])]), int(nz[np.argmin(counts[nz])])}
    chosen |= {int(e) for e in np.nonzero(counts == 0)[0]}
    rng = np.random.default_rng(seed)
    chosen |= {int(e) for e in rng.choice(len(counts), size=min(n_random, len(counts)), replace=False)}
    return sorted(chosen)


@pytest.mark.parametrize("name", ["tiny", "small"])
def test_full_parity(name):
    w = synth.WORKLOADS[name]
    li = synth.make_layer_inputs(w)
    out = run_gpu(w, li)
    errs = check_full(w, li, out)
    print(name, errs)


def test_fine_fold_sampled():
    w = synth.WORKLOADS["fine_fold"]
    li = synth.make_layer_inputs(w)
    out = run_gpu(w, li)
    assert out["counts"].sum() == w.R
    print(check_sampled(w, li, out, 1024, pick_experts(out["counts"], 4, 0)))


def test_skewed_sampled_with_empty_experts():
    w = synth.WORKLOADS["skewed"]
    li = synth.make_layer_inputs(w)
    out = run_gpu(w, li)
    assert (out["counts"] == 0).sum() == 4
    experts = pick_experts(out["counts"], 4, 1)
    assert set(np.nonzero(out["counts"] == 0)[0].tolist()) <= set(experts) and len(experts) >= 6
    print(check_sampled(w, li, out, 1024, experts))


def test_large_sampled():
    w = synth.WORKLOADS["large"]
    li = synth.make_layer_inputs(w)
    out = run_gpu(w, li)
    counts = out["counts"]
    nz = np.nonzero(counts)[0]
    median = int(nz[np.argsort(counts[nz])[len(nz) // 2]])
    experts = sorted(set(pick_experts(counts, 4, 4)) | {median})     # heaviest (the one split into chunks), lightest, 4 random, median
    print(check_sampled(w, li, out, 1024, experts))


@pytest.mark.parametrize("T,d,F,E,k,kw", [
    (300, 64, 64, 1, 1, {}),                       # dense special case, one ragged tile
    (257, 128, 72, 5, 3, {}),                      # F not a multiple of 64; segments far below one tile
    (1000, 720, 720, 32, 4, {}),                   # a model shape from the paper's configuration table
    (640, 384, 344, 128, 8, {}),                   # another: more experts than tiles per expert
    (900, 512, 704, 64, 6, {"load": "zipf", "zipf_s": 1.3, "n_dead": 7}),
    (512, 1024, 384, 128, 8, {}),
    (192, 256, 256, 128, 2, {"n_dead": 112}),      # long runs of experts without rows: tiles that contract nothing
])
def test_edge_shapes_full_parity(T, d, F, E, k, kw):
    w = synth.custom_workload("edge", T=T, d=d, ffn=F, E=E, k=k, seed=T + d, **kw)
    li = synth.make_layer_inputs(w)
    out = run_gpu(w, li)
    print(check_full(w, li, out))


def test_f32_gates_i32_idx_and_fold_collisions():
    w = synth.custom_workload("fold", T=700, d=256, ffn=256, E=24, k=4, E_tgt=5, fold_mod=5, seed=11)
    li = synth.make_layer_inputs(w)
    out = run_gpu(w, li, gate_f32=True, idx_i32=True)
    print(check_full(w, li, out))


@pytest.mark.parametrize("case", ["tiny", "small", "ragged", "fold", "paper_shape"])
def test_fused_combine_variant_full_parity(case):
    """GROUTER_FLAG_FUSED_COMBINE: the down product adds its gate-weighted rows straight into the tokens' fp32 rows.
    Same bar against the oracle as the two-kernel form; the backward pass is untouched and checked along."""
    from paper_2603_06626_b200 import binding
    kw = {}
    if case in ("tiny", "small"):
        w = synth.WORKLOADS[case]
    elif case == "ragged":
        w = synth.custom_workload("edge", T=257, d=128, ffn=72, E=5, k=3, seed=385)
    elif case == "paper_shape":
        w = synth.custom_workload("edge", T=640, d=384, ffn=344, E=128, k=8, seed=1024)
    else:
        w = synth.custom_workload("fold", T=700, d=256, ffn=256, E=24, k=4, E_tgt=5, fold_mod=5, seed=11)
        kw = dict(gate_f32=True, idx_i32=True)
    li = synth.make_layer_inputs(w)
    fused = run_gpu(w, li, flags=binding.FLAG_FUSED_COMBINE, **kw)
    print(check_full(w, li, fused))
    plain = run_gpu(w, li, **kw)
    # the two forms round differently (one bf16 rounding of the fp32 sum against k roundings of the rows): close, not equal
    assert orc.rel_frobenius(f64(fused["Y"]), f64(plain["Y"])) < 8e-3
    for name in ("dX", "dgates"):
        assert torch.equal(fused[name], plain[name]), name


def test_dense_special_case_unit_gate():
    """E=1, k=1, gate=1: the layer is a dense SwiGLU FFN."""
    w = synth.custom_workload("dense", T=384, d=128, ffn=256, E=1, k=1, seed=5)
    li = synth.make_layer_inputs(w)
    li.gates = synth.f32_to_bf16_bits(np.ones((w.T, 1), dtype=np.float32))
    out = run_gpu(w, li)
    print(check_full(w, li, out))


def test_plan_reuse_across_layers_and_determinism():
    """One plan serves several forward/backward calls (all layers share the frozen router); results are bit-stable."""
    from paper_2603_06626_b200 import binding
    w = synth.WORKLOADS["tiny"]
    li = synth.make_layer_inputs(w)
    layer = binding.GrouterLayer(w.T, w.d, w.ffn, w.E_src, w.k)
    idx, gates = to_dev(li.idx), bits_to_bf16(li.gates)
    X, dY, W_gu, W_d = bits_to_bf16(li.X), bits_to_bf16(li.dY), bits_to_bf16(li.W_gu), bits_to_bf16(li.W_d)
    layer.plan(idx)
    Y1 = layer.forward(X, gates, W_gu, W_d).clone()
    r1 = [t.clone() for t in layer.backward(dY, X, gates, W_gu, W_d)]
    Y2 = layer.forward(X, gates, W_gu, W_d)
    r2 = layer.backward(dY, X, gates, W_gu, W_d)
    layer.check_status()
    assert torch.equal(Y1, Y2)
    for a, b in zip(r1, r2):
        assert torch.equal(a, b)
    layer.close()


def test_accumulate_dw_over_micro_batches():
    """GROUTER_FLAG_ACCUMULATE_DW: two micro-batches with different routing add up in the caller's zeroed gradients;
    the sum is checked against the oracle's sum, expert by expert (one expert gets slots in neither batch)."""
    from paper_2603_06626_b200 import binding
    base = synth.custom_workload("acc", T=1536, d=256, ffn=384, E=12, k=3, seed=21)
    route = synth.custom_workload("acc", T=1536, d=256, ffn=384, E=11, k=3, load="zipf", zipf_s=1.2, seed=21)   # ids 0..10: expert 11 idle
    batches = [synth.make_layer_inputs(synth.reseeded(route, 21 + i), with_weights=False) for i in range(2)]
    W_gu_bits = np.stack([synth.expert_W_gu(base, e) for e in range(base.E_tgt)])
    W_d_bits = np.stack([synth.expert_W_d(base, e) for e in range(base.E_tgt)])
    W_gu, W_d = bits_to_bf16(W_gu_bits), bits_to_bf16(W_d_bits)
    layer = binding.GrouterLayer(base.T, base.d, base.ffn, base.E_src, base.k, flags=binding.FLAG_ACCUMULATE_DW)
    dW_gu = torch.zeros(W_gu.shape, dtype=torch.float32, device="cuda:0")
    dW_d = torch.zeros(W_d.shape, dtype=torch.float32, device="cuda:0")
    weights = orc.Weights(synth.bf16_bits_to_f64(W_gu_bits), synth.bf16_bits_to_f64(W_d_bits))
    want_gu = np.zeros(W_gu.shape, dtype=np.float64)
    want_d = np.zeros(W_d.shape, dtype=np.float64)
    touched = np.zeros(base.E_tgt, dtype=bool)
    for li in batches:
        idx, gates, X, dY = to_dev(li.idx), bits_to_bf16(li.gates), bits_to_bf16(li.X), bits_to_bf16(li.dY)
        layer.plan(idx)
        layer.forward(X, gates, W_gu, W_d)
        layer.backward(dY, X, gates, W_gu, W_d, dW_gu=dW_gu, dW_d=dW_d)
        touched |= layer.counts.cpu().numpy() > 0
        f64 = synth.bf16_bits_to_f64
        _, _, dW = orc.moe_backward(f64(li.dY), f64(li.X), li.idx, f64(li.gates), weights, base.E_tgt)
        for e in range(base.E_tgt):
            want_gu[e] += dW[e][0]
            want_d[e] += dW[e][1]
    layer.check_status()
    got_gu, got_d = dW_gu.double().cpu().numpy(), dW_d.double().cpu().numpy()
    assert not touched[11] and touched[:11].all()
    for e in range(base.E_tgt):
        if not touched[e]:
            assert not got_gu[e].any() and not got_d[e].any()
        else:
            assert orc.rel_frobenius(got_gu[e], want_gu[e]) < TOL and orc.rel_frobenius(got_d[e], want_d[e]) < TOL
    layer.close()
    with pytest.raises(binding.GrouterError):
        binding.GrouterLayer(64, 64, 64, 4, 2, flags=4)      # unknown flag bit


def test_whole_step_replays_from_a_cuda_graph():
    """plan + fwd + bwd only enqueue kernels on the caller's stream (no allocation, no synchronisation), so a step can be
    captured once and replayed; the replay is bit-identical for everything that is reproducible."""
    from paper_2603_06626_b200 import binding
    w = synth.WORKLOADS["tiny"]
    li = synth.make_layer_inputs(w)
    idx, gates, X, dY = to_dev(li.idx), bits_to_bf16(li.gates), bits_to_bf16(li.X), bits_to_bf16(li.dY)
    W_gu, W_d = bits_to_bf16(li.W_gu), bits_to_bf16(li.W_d)
    layer = binding.GrouterLayer(w.T, w.d, w.ffn, w.E_src, w.k, E_tgt=w.E_tgt)
    Y, dX = torch.empty_like(X), torch.empty_like(X)
    dg = torch.empty(w.T, w.k, device=X.device, dtype=torch.float32)
    dW_gu = torch.empty(W_gu.shape, device=X.device, dtype=torch.float32)
    dW_d = torch.empty(W_d.shape, device=X.device, dtype=torch.float32)

    def step():
        layer.plan(idx)
        layer.forward(X, gates, W_gu, W_d, Y)
        layer.backward(dY, X, gates, W_gu, W_d, dX, dW_gu, dW_d, dg)

    step()
    layer.check_status()
    want = [t.clone() for t in (Y.view(torch.int16), dX.view(torch.int16), dg, dW_gu, dW_d)]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):      # warm-up on a side stream, as capture requires
        step()
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for t in (Y, dX, dg, dW_gu, dW_d):
        t.zero_()
    for _ in range(3):
        graph.replay()
    layer.check_status()
    got = (Y.view(torch.int16), dX.view(torch.int16), dg, dW_gu, dW_d)
    for g, x in zip(got[:3], want[:3]):
        assert torch.equal(g, x)
    for g, x in zip(got[3:], want[3:]):      # experts cut into several chunks are summed with atomics
        assert (g - x).double().norm() <= 1e-6 * x.double().norm()
    layer.close()


def test_issuer_cycle_accounting_counts_every_tile_and_k_step():
    """The optional account of the MMA issuers: tile and k-step counts follow from the plan, the waits are part of the
    total, nothing is counted while it is off, and the results do not change."""
    from paper_2603_06626_b200 import binding
    w = synth.WORKLOADS["small"]
    li = synth.make_layer_inputs(w)
    idx, gates, X, dY = to_dev(li.idx), bits_to_bf16(li.gates), bits_to_bf16(li.X), bits_to_bf16(li.dY)
    W_gu, W_d = bits_to_bf16(li.W_gu), bits_to_bf16(li.W_d)
    layer = binding.GrouterLayer(w.T, w.d, w.ffn, w.E_src, w.k, E_tgt=w.E_tgt)

    def step():
        layer.plan(idx)
        Y = layer.forward(X, gates, W_gu, W_d)
        dX = layer.backward(dY, X, gates, W_gu, W_d)[0]
        return Y.clone(), dX.clone()

    Y0, dX0 = step()
    assert all(v == 0 for c in layer.gemm_cycles_read().values() for v in c.values())     # off by default
    layer.gemm_cycles_enable(True)
    Y1, dX1 = step()
    got = layer.gemm_cycles_read()
    layer.gemm_cycles_enable(False)
    step()
    assert all(v == 0 for c in layer.gemm_cycles_read().values() for v in c.values())
    layer.check_status()
    assert torch.equal(Y0, Y1) and torch.equal(dX0, dX1)

    counts = layer.counts.cpu().numpy().astype(np.int64)
    pair_tiles = int((((counts + 127) // 128 + 1) // 2).sum())
    cdiv = lambda a, b: (a + b - 1) // b
    d, F = w.d, w.ffn
    want = {"gemm_up_swiglu": (pair_tiles * cdiv(F, 128), cdiv(d, 64)), "gemm_down": (pair_tiles * cdiv(d, 256), cdiv(F, 64)),
            "gemm_dH": (pair_tiles * cdiv(F, 256), cdiv(d, 64)), "gemm_dX": (pair_tiles * cdiv(d, 256), cdiv(2 * F, 64))}
    for name, (tiles, k_per_tile) in want.items():
        c = got[name]
        assert c["tiles"] == tiles and c["k_steps"] == tiles * k_per_tile, (name, c)
        assert c["cycles"] >= c["wait_operands"] + c["wait_accumulator"] > 0, (name, c)
        assert c["cycles"] >= 512 * c["k_steps"] / 74, (name, c)      # summed over the pairs: at least the tensor-core time
    for name in ("wgrad_down", "wgrad_gate_up"):
        assert got[name]["tiles"] > 0 and got[name]["k_steps"] >= got[name]["tiles"]
    layer.close()


def test_active_tokens_on_a_larger_context_match_the_oracle():
    """grouter_set_active_tokens: a context laid out for 1000 tokens runs a batch of 613, then one of 1000, then 77."""
    from paper_2603_06626_b200 import binding
    full = synth.custom_workload("act", T=1000, d=256, ffn=320, E=10, k=3, seed=31)
    layer = binding.GrouterLayer(full.T, full.d, full.ffn, full.E_src, full.k)
    W_gu_bits = np.stack([synth.expert_W_gu(full, e) for e in range(full.E_tgt)])
    W_d_bits = np.stack([synth.expert_W_d(full, e) for e in range(full.E_tgt)])
    W_gu, W_d = bits_to_bf16(W_gu_bits), bits_to_bf16(W_d_bits)
    for n, seed in ((613, 40), (1000, 41), (77, 42)):
        w = synth.custom_workload("act", T=n, d=full.d, ffn=full.ffn, E=full.E_src, k=full.k, load="zipf", zipf_s=1.0, seed=seed)
        li = synth.make_layer_inputs(w, with_weights=False)
        li.W_gu, li.W_d = W_gu_bits, W_d_bits
        layer.set_active_tokens(n)
        plan = [t.cpu().numpy() for t in layer.plan(to_dev(li.idx))]
        for got, want in zip(plan, orc.plan(li.idx, None, w.E_tgt)):
            assert np.array_equal(got, want)
        X, dY, gates = bits_to_bf16(li.X), bits_to_bf16(li.dY), bits_to_bf16(li.gates)
        Y = layer.forward(X, gates, W_gu, W_d)
        dX, dW_gu, dW_d, dgates = layer.backward(dY, X, gates, W_gu, W_d)
        layer.check_status()
        assert Y.shape[0] == n and dgates.shape == (n, w.k)
        out = dict(Y=Y, dX=dX, dW_gu=dW_gu, dW_d=dW_d, dgates=dgates, counts=plan[0])
        print(n, check_full(w, li, out))
    with pytest.raises(binding.GrouterError):
        layer.set_active_tokens(1001)
    layer.set_active_tokens(5)
    with pytest.raises(binding.GrouterError):                 # a new token count needs a new plan
        layer.forward(bits_to_bf16(li.X[:5]), bits_to_bf16(li.gates[:5]), W_gu, W_d)
    layer.close()


def test_kernels_beside_the_gemms_change_no_bit():
    """The backward pass runs the dX reduction and the gradient zero-fill on a stream of the context beside the GEMMs
    (default) or in line: the same kernels on the same data, so every output is bit-identical either way, also when the
    two forms alternate on one context."""
    from paper_2603_06626_b200 import binding
    w = synth.custom_workload("side", T=2048, d=512, ffn=384, E=6, k=3, load="zipf", zipf_s=1.4, seed=17)   # the hot expert is split into chunks
    li = synth.make_layer_inputs(w)
    layer = binding.GrouterLayer(w.T, w.d, w.ffn, w.E_src, w.k)
    idx, gates, X, dY = to_dev(li.idx), bits_to_bf16(li.gates), bits_to_bf16(li.X), bits_to_bf16(li.dY)
    W_gu, W_d = bits_to_bf16(li.W_gu), bits_to_bf16(li.W_d)
    counts = None
    results = []
    for on in (True, False, True):
        layer.set_overlap(on)
        layer.plan(idx)
        Y = layer.forward(X, gates, W_gu, W_d)
        dX, dW_gu, dW_d, dg = layer.backward(dY, X, gates, W_gu, W_d)
        torch.cuda.synchronize()
        layer.check_status()
        counts = layer.counts.cpu().numpy()
        results.append([t.clone() for t in (Y, dX, dg, dW_gu, dW_d)])
    whole = torch.from_numpy(((counts + 127) // 128 * 128) <= layer.wgrad_chunk_rows()).to(X.device)   # experts contracted in one piece
    assert (~whole).any(), "the case is meant to contain an expert that is split into chunks"
    for other in results[1:]:
        for a, b in zip(results[0][:3], other[:3]):
            assert torch.equal(a, b)
        for a, b in zip(results[0][3:], other[3:]):
            assert torch.equal(a[whole], b[whole])
            assert (a - b).double().norm() <= 1e-6 * a.double().norm()      # chunks of a split expert are added in no fixed order
    out = dict(Y=results[0][0], dX=results[0][1], dgates=results[0][2], dW_gu=results[0][3], dW_d=results[0][4], counts=counts)
    print(check_full(w, li, out))
    layer.close()
