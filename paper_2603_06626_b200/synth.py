"""Seeded synthetic inputs for the routed expert layer under preemptive routing.

This module only draws random numbers and packs them into the storage formats
the layer consumes.  It holds none of the layer's arithmetic, so both the CUDA
path's tests/benchmarks and the CPU oracle's tests may use it.

Storage formats follow the paper's pre-dispatch cache (appendix "Efficiency
Experiment Detail", paragraph Pre-Dispatch; appendix "Overhead Analysis",
paragraph Storage Requirements): expert ids as uint8, routing scores as
bfloat16, i.e. 3*k bytes per token.  bf16 tensors are carried as uint16 bit
patterns in numpy (numpy has no bf16 type).

The five workloads are the synthetic stand-ins for C4-driven routing on the
paper's Qwen3-/DeepSeek-style MoE layers; the paper publishes no per-expert
load histogram, only that an untuned frozen router is strongly imbalanced,
hence uniform, Zipf-skewed and mixed expert-load recipes.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np

# Tags that separate the random streams of the different tensors.
_TAG_X, _TAG_DY, _TAG_WGU, _TAG_WD, _TAG_IDX, _TAG_GATE, _TAG_PERM = range(7)


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even); returns uint16 bits."""
    b = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    bias = np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))
    return ((b + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns exactly to float32."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns exactly to float64."""
    return bf16_bits_to_f32(bits).astype(np.float64)


@dataclass(frozen=True)
class Workload:
    """Sizes and routing recipe of one synthetic MoE layer."""
    name: str
    T: int            # tokens
    d: int            # model width
    ffn: int          # expert hidden width F
    E_src: int        # expert ids that may appear in idx
    E_tgt: int        # experts that own weights (== E_src unless folded)
    k: int            # experts per token
    load: str         # "uniform" | "zipf" | "mixed"
    zipf_s: float = 0.0
    n_dead: int = 0   # source experts that receive no token
    fold_mod: int = 0 # if > 0: fold_map[i] = i % fold_mod
    seed: int = 0
    w_std: float = 0.02

    @property
    def R(self) -> int:
        return self.T * self.k


WORKLOADS = {
    "tiny": Workload("tiny", T=512, d=256, ffn=512, E_src=8, E_tgt=8, k=2, load="uniform", seed=0),
    "small": Workload("small", T=4096, d=1024, ffn=2816, E_src=16, E_tgt=16, k=2, load="zipf", zipf_s=1.1, seed=1),
    "fine_fold": Workload("fine_fold", T=8192, d=2048, ffn=1024, E_src=64, E_tgt=16, k=8, load="uniform",
                          fold_mod=16, seed=2),
    "skewed": Workload("skewed", T=16384, d=2048, ffn=1408, E_src=64, E_tgt=64, k=8, load="zipf", zipf_s=1.5,
                       n_dead=4, seed=3),
    "large": Workload("large", T=32768, d=4096, ffn=1536, E_src=128, E_tgt=128, k=8, load="mixed", zipf_s=1.2,
                      seed=4),
}
WORKLOAD_ORDER = ["tiny", "small", "fine_fold", "skewed", "large"]


def _rng(seed: int, *tags: int) -> np.random.Generator:
    return np.random.default_rng([int(seed), *[int(t) for t in tags]])


def expert_probabilities(w: Workload) -> np.ndarray:
    """Selection probabilities over the E_src source ids.

    Popularity ranks are assigned to ids by a seeded permutation so that hot
    experts are not contiguous in id space.
    """
    E = w.E_src
    perm = _rng(w.seed, _TAG_PERM).permutation(E)
    p_rank = np.zeros(E, dtype=np.float64)
    live = E - w.n_dead
    if w.load == "uniform":
        p_rank[:live] = 1.0
    elif w.load == "zipf":
        p_rank[:live] = np.arange(1, live + 1, dtype=np.float64) ** (-w.zipf_s)
    elif w.load == "mixed":
        half = live // 2
        z = np.arange(1, half + 1, dtype=np.float64) ** (-w.zipf_s)
        p_rank[:half] = 0.5 * z / z.sum()
        p_rank[half:live] = 0.5 / (live - half)
    else:
        raise ValueError(w.load)
    p_rank /= p_rank.sum()
    p = np.zeros(E, dtype=np.float64)
    p[perm] = p_rank
    return p


def make_idx(w: Workload, T: Optional[int] = None, chunk: int = 1 << 16) -> np.ndarray:
    """uint8 [T,k] (int32 if E_src > 256): k distinct source experts per token.

    Drawn without replacement by the Gumbel-top-k trick from
    `expert_probabilities`, kept in descending-key order (ids not sorted).
    """
    T = w.T if T is None else T
    p = expert_probabilities(w)
    with np.errstate(divide="ignore"):
        logp = np.log(p)
    assert (p > 0).sum() >= w.k
    rng = _rng(w.seed, _TAG_IDX)
    dtype = np.uint8 if w.E_src <= 256 else np.int32
    out = np.empty((T, w.k), dtype=dtype)
    for t0 in range(0, T, chunk):
        n = min(chunk, T - t0)
        keys = logp[None, :] + rng.gumbel(size=(n, w.E_src))
        top = np.argpartition(-keys, w.k - 1, axis=1)[:, : w.k]
        order = np.argsort(-np.take_along_axis(keys, top, axis=1), axis=1, kind="stable")
        out[t0:t0 + n] = np.take_along_axis(top, order, axis=1).astype(dtype)
    return out


def make_idx_sample_affinity(w: Workload, seq_len: int, owner: np.ndarray, n_nodes: int, boost: float = 8.0):
    """Routing table whose samples (runs of seq_len tokens) lean towards the experts of one node each: a stand-in for the
    sequence-level routing structure the paper's sample placement exploits (its corpus statistics are not available).

    Sample s has a home node h(s) (seeded, uniform); the selection probability of every expert owned by h(s) is
    multiplied by `boost` before the k distinct experts of each token are drawn as in make_idx.
    Returns (idx [T,k], home [S])."""
    assert w.T % seq_len == 0
    S = w.T // seq_len
    p = expert_probabilities(w)
    with np.errstate(divide="ignore"):
        logp = np.log(p)
    rng = _rng(w.seed, _TAG_IDX, 77)
    home = rng.integers(0, n_nodes, size=S)
    dtype = np.uint8 if w.E_src <= 256 else np.int32
    out = np.empty((w.T, w.k), dtype=dtype)
    owner = np.asarray(owner)
    for s_ in range(S):
        lp = logp + np.log(boost) * (owner == home[s_])
        keys = lp[None, :] + rng.gumbel(size=(seq_len, w.E_src))
        top = np.argpartition(-keys, w.k - 1, axis=1)[:, : w.k]
        order = np.argsort(-np.take_along_axis(keys, top, axis=1), axis=1, kind="stable")
        out[s_ * seq_len:(s_ + 1) * seq_len] = np.take_along_axis(top, order, axis=1).astype(dtype)
    return out, home.astype(np.int32)


def make_gates(w: Workload, T: Optional[int] = None) -> np.ndarray:
    """bf16 bits [T,k]: softmax over the token's k chosen logits ~ N(0,1)."""
    T = w.T if T is None else T
    z = _rng(w.seed, _TAG_GATE).standard_normal((T, w.k))
    z -= z.max(axis=1, keepdims=True)
    e = np.exp(z)
    return f32_to_bf16_bits((e / e.sum(axis=1, keepdims=True)).astype(np.float32))


def make_fold_map(w: Workload) -> Optional[np.ndarray]:
    """int32 [E_src] -> [0,E_tgt) or None.  Compact form of the binary fold matrix M."""
    if w.fold_mod <= 0:
        return None
    return (np.arange(w.E_src, dtype=np.int32) % np.int32(w.fold_mod)).astype(np.int32)


def make_tokens(w: Workload, tag: int = _TAG_X) -> np.ndarray:
    """bf16 bits [T,d] ~ N(0,1)."""
    return f32_to_bf16_bits(_rng(w.seed, tag).standard_normal((w.T, w.d), dtype=np.float32))


def make_dY(w: Workload) -> np.ndarray:
    """bf16 bits [T,d] ~ N(0,1): the upstream gradient."""
    return make_tokens(w, _TAG_DY)


def expert_W_gu(w: Workload, e: int) -> np.ndarray:
    """bf16 bits [2*ffn, d] for expert e: rows 0..ffn-1 gate proj, ffn..2ffn-1 up proj."""
    a = _rng(w.seed, _TAG_WGU, e).standard_normal((2 * w.ffn, w.d), dtype=np.float32)
    return f32_to_bf16_bits(a * np.float32(w.w_std))


def expert_W_d(w: Workload, e: int) -> np.ndarray:
    """bf16 bits [d, ffn] for expert e (down projection, nn.Linear [out,in] layout)."""
    a = _rng(w.seed, _TAG_WD, e).standard_normal((w.d, w.ffn), dtype=np.float32)
    return f32_to_bf16_bits(a * np.float32(w.w_std))


@dataclass
class LayerInputs:
    w: Workload
    X: np.ndarray                 # u16 [T,d]
    dY: np.ndarray                # u16 [T,d]
    idx: np.ndarray               # u8/i32 [T,k]
    gates: np.ndarray             # u16 [T,k]
    fold_map: Optional[np.ndarray]
    W_gu: Optional[np.ndarray] = None   # u16 [E_tgt, 2F, d]
    W_d: Optional[np.ndarray] = None    # u16 [E_tgt, d, F]
    extra: dict = field(default_factory=dict)


def make_layer_inputs(w: Workload, with_weights: bool = True, threads: int = 0) -> LayerInputs:
    """All inputs of one fwd+bwd step.  Weights can be skipped and drawn per
    expert later with `expert_W_gu` / `expert_W_d` (same bits).  `threads` > 1
    draws the experts' weights in parallel (each expert has its own stream, so
    the bits do not depend on it)."""
    li = LayerInputs(w=w, X=make_tokens(w), dY=make_dY(w), idx=make_idx(w), gates=make_gates(w),
                     fold_map=make_fold_map(w))
    if with_weights:
        li.W_gu = np.empty((w.E_tgt, 2 * w.ffn, w.d), dtype=np.uint16)
        li.W_d = np.empty((w.E_tgt, w.d, w.ffn), dtype=np.uint16)

        def fill(e):
            li.W_gu[e] = expert_W_gu(w, e)
            li.W_d[e] = expert_W_d(w, e)

        if threads > 1:
            from concurrent.futures import ThreadPoolExecutor
            with ThreadPoolExecutor(max_workers=threads) as pool:
                list(pool.map(fill, range(w.E_tgt)))
        else:
            for e in range(w.E_tgt):
                fill(e)
    return li


def reseeded(w: Workload, seed: int) -> Workload:
    """Same shapes and load recipe, different random streams (one per data-parallel rank)."""
    from dataclasses import replace
    return replace(w, seed=int(seed))


def custom_workload(name: str, T: int, d: int, ffn: int, E: int, k: int, *, load: str = "uniform",
                    zipf_s: float = 0.0, n_dead: int = 0, E_tgt: Optional[int] = None, fold_mod: int = 0,
                    seed: int = 0) -> Workload:
    return Workload(name, T=T, d=d, ffn=ffn, E_src=E, E_tgt=E if E_tgt is None else E_tgt, k=k, load=load,
                    zipf_s=zipf_s, n_dead=n_dead, fold_mod=fold_mod, seed=seed)


def load_stats(idx: np.ndarray, fold_map: Optional[np.ndarray], E_tgt: int) -> dict:
    """Descriptive statistics of a routing table (no layer arithmetic)."""
    e = idx.astype(np.int64).ravel()
    if fold_map is not None:
        e = fold_map.astype(np.int64)[e]
    c = np.bincount(e, minlength=E_tgt)
    mean = c.mean()
    return {"max": int(c.max()), "min": int(c.min()), "empty": int((c == 0).sum()),
            "max_vio": float((c.max() - mean) / mean) if mean > 0 else 0.0}
