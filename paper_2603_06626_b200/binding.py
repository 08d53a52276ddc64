"""ctypes binding of libgrouter.so (the C ABI in include/grouter.h).

Argument marshalling only: every step of the layer runs in the CUDA library.
torch is used for device memory and streams.  There is no fallback: if the
library cannot be loaded this module raises.
"""
from __future__ import annotations

import contextlib
import ctypes
import os
from typing import Optional

import torch

from . import build as _build

IDX_U8, IDX_I32 = 0, 1
FLAG_ACCUMULATE_DW = 1
FLAG_FUSED_COMBINE = 2
NORM_SOFTMAX, NORM_SIGMOID = 0, 1
GATE_BF16, GATE_F32 = 0, 1

EXPORTS = ["grouter_create", "grouter_destroy", "grouter_workspace_bytes", "grouter_host_staging_bytes", "grouter_plan",
           "grouter_moe_fwd", "grouter_moe_bwd", "grouter_moe_step_host", "grouter_status", "grouter_strerror",
           "grouter_dense_gemm", "grouter_timing_enable", "grouter_timing_read", "grouter_plan_noalloc", "grouter_host_wait", "grouter_route", "grouter_route_workspace_bytes", "grouter_routing_stats",
           "grouter_fold_greedy_host", "grouter_timing_gap", "grouter_wgrad_chunk_rows", "grouter_gemm_cycles_enable", "grouter_gemm_cycles_read", "grouter_set_wait_limit", "grouter_wait_selftest", "grouter_set_overlap", "grouter_set_active_tokens",
           "grouter_checked_build",
           "grouter_ep_relabel_host", "grouter_ep_layout_host", "grouter_ep_expand_ids", "grouter_ep_dispatch_rows", "grouter_ep_combine_rows"]
KERNEL_SLOTS = ["plan_hist", "plan_permute", "gather_X", "gemm_up_swiglu", "gemm_down", "combine_Y", "gather_dY", "gemm_dH",
                "wgrad_down", "gemm_dX", "wgrad_gate_up", "reduce_dX", "zero_split_dW", "plan_scan"]


class GrouterDims(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("T", "d", "ffn", "E_src", "E_tgt", "k", "idx_dtype", "gate_dtype", "flags")]


class GrouterError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {strerror(code)} ({code})")
        self.code = code


_lib = None


def load_library(path: Optional[str] = None) -> ctypes.CDLL:
    """Loads (building in-tree first if stale or absent) and types the library."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    if path is None:
        path = _build.LIB
        try:
            _build.build(force=bool(os.environ.get("GROUTER_REBUILD")))     # returns at once when the library is newer than every source
        except (OSError, RuntimeError) as err:
            # no compiler here (or the build failed): an existing library is used, loudly; without one there is nothing to fall back to
            if not os.path.exists(path):
                raise
            import sys
            sys.stderr.write(f"paper_2603_06626_b200: could not rebuild libgrouter.so ({err}); loading the existing, possibly stale, library\n")
    lib = ctypes.CDLL(path)
    vp, i32p, f32p = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p
    lib.grouter_create.argtypes = [ctypes.POINTER(ctypes.c_void_p), ctypes.POINTER(GrouterDims)]
    lib.grouter_create.restype = ctypes.c_int
    lib.grouter_destroy.argtypes = [vp]
    lib.grouter_destroy.restype = None
    lib.grouter_workspace_bytes.argtypes = [ctypes.POINTER(GrouterDims)]
    lib.grouter_workspace_bytes.restype = ctypes.c_size_t
    lib.grouter_host_staging_bytes.argtypes = [ctypes.POINTER(GrouterDims)]
    lib.grouter_host_staging_bytes.restype = ctypes.c_size_t
    lib.grouter_plan.argtypes = [vp, vp, i32p, i32p, i32p, i32p, i32p, vp]
    lib.grouter_plan.restype = ctypes.c_int
    lib.grouter_plan_noalloc.argtypes = [vp, ctypes.c_int32, i32p] + [ctypes.c_int32] * 4 + [i32p] * 5 + [vp]
    lib.grouter_plan_noalloc.restype = ctypes.c_int
    lib.grouter_moe_fwd.argtypes = [vp] * 8
    lib.grouter_moe_fwd.restype = ctypes.c_int
    lib.grouter_moe_bwd.argtypes = [vp] * 12
    lib.grouter_moe_bwd.restype = ctypes.c_int
    lib.grouter_moe_step_host.argtypes = [vp] * 15
    lib.grouter_moe_step_host.restype = ctypes.c_int
    lib.grouter_route_workspace_bytes.argtypes = [ctypes.c_int32] * 3
    lib.grouter_route_workspace_bytes.restype = ctypes.c_size_t
    lib.grouter_route.argtypes = [vp, vp, i32p] + [ctypes.c_int32] * 6 + [vp, vp, f32p, vp, i32p, vp]
    lib.grouter_route.restype = ctypes.c_int
    lib.grouter_routing_stats.argtypes = [vp] + [ctypes.c_int32] * 5 + [i32p, ctypes.c_int32, i32p, i32p, f32p, f32p, i32p, i32p, i32p, vp]
    lib.grouter_routing_stats.restype = ctypes.c_int
    lib.grouter_fold_greedy_host.argtypes = [vp, ctypes.c_int32, ctypes.c_int32, vp]
    lib.grouter_fold_greedy_host.restype = ctypes.c_int
    lib.grouter_host_wait.argtypes = [vp, ctypes.c_int32]
    lib.grouter_host_wait.restype = ctypes.c_int
    lib.grouter_status.argtypes = [vp, vp]
    lib.grouter_status.restype = ctypes.c_int
    lib.grouter_strerror.argtypes = [ctypes.c_int]
    lib.grouter_strerror.restype = ctypes.c_char_p
    lib.grouter_dense_gemm.argtypes = [vp, ctypes.c_int, vp, ctypes.c_int, f32p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, vp, vp]
    lib.grouter_dense_gemm.restype = ctypes.c_int
    lib.grouter_timing_enable.argtypes = [vp, ctypes.c_int32]
    lib.grouter_timing_enable.restype = ctypes.c_int
    lib.grouter_timing_gap.argtypes = [vp, ctypes.c_int32]
    lib.grouter_timing_gap.restype = ctypes.c_int
    lib.grouter_gemm_cycles_enable.argtypes = [vp, ctypes.c_int32]
    lib.grouter_gemm_cycles_enable.restype = ctypes.c_int
    lib.grouter_gemm_cycles_read.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_uint64)]
    lib.grouter_gemm_cycles_read.restype = ctypes.c_int
    lib.grouter_wgrad_chunk_rows.argtypes = [vp]
    lib.grouter_wgrad_chunk_rows.restype = ctypes.c_int32
    lib.grouter_ep_relabel_host.argtypes = [ctypes.c_int32, ctypes.c_int32, vp, vp, vp]
    lib.grouter_ep_relabel_host.restype = ctypes.c_int
    lib.grouter_ep_layout_host.argtypes = [ctypes.c_int32] * 3 + [vp] * 7
    lib.grouter_ep_layout_host.restype = ctypes.c_int
    lib.grouter_ep_expand_ids.argtypes = [vp] + [ctypes.c_int32] * 4 + [vp, vp]
    lib.grouter_ep_expand_ids.restype = ctypes.c_int
    lib.grouter_ep_dispatch_rows.argtypes = [vp] * 5
    lib.grouter_ep_dispatch_rows.restype = ctypes.c_int
    lib.grouter_ep_combine_rows.argtypes = [vp] * 7
    lib.grouter_ep_combine_rows.restype = ctypes.c_int
    lib.grouter_set_active_tokens.argtypes = [vp, ctypes.c_int32]
    lib.grouter_set_active_tokens.restype = ctypes.c_int
    lib.grouter_set_overlap.argtypes = [vp, ctypes.c_int32]
    lib.grouter_set_overlap.restype = ctypes.c_int
    lib.grouter_set_wait_limit.argtypes = [vp, ctypes.c_int64]
    lib.grouter_set_wait_limit.restype = ctypes.c_int
    lib.grouter_wait_selftest.argtypes = [vp, ctypes.c_int64, ctypes.POINTER(ctypes.c_int64), vp]
    lib.grouter_wait_selftest.restype = ctypes.c_int
    lib.grouter_timing_read.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int32)]
    lib.grouter_timing_read.restype = ctypes.c_int
    lib.grouter_checked_build.argtypes = []
    lib.grouter_checked_build.restype = ctypes.c_int
    if path == _build.LIB:
        _lib = lib
    return lib


@contextlib.contextmanager
def checked_build():
    """Inside the block every call of this module goes through the checked build of the library (compiled on demand):
    kernels that test data-derived indices before use and report GROUTER_ERR_BOUNDS (-9) through the status word."""
    global _lib
    release = load_library()
    try:
        path = _build.build(debug=True)
    except (OSError, RuntimeError) as err:      # as in load_library: an existing library is used, loudly
        path = _build.LIB_DEBUG
        if not os.path.exists(path):
            raise
        import sys
        sys.stderr.write(f"paper_2603_06626_b200: could not rebuild libgrouter_debug.so ({err}); loading the existing, possibly stale, library\n")
    lib = load_library(path)
    if lib.grouter_checked_build() != 1:
        raise RuntimeError("libgrouter_debug.so was not compiled with the index tests")
    _lib = lib
    try:
        yield lib
    finally:
        _lib = release


def strerror(code: int) -> str:
    return load_library().grouter_strerror(code).decode()


def _check(code: int, what: str) -> None:
    if code != 0:
        raise GrouterError(code, what)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_contiguous()
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


class GrouterLayer:
    """One layer shape: owns the context and the workspace; thin calls into the C ABI."""

    def __init__(self, T: int, d: int, ffn: int, E_src: int, k: int, E_tgt: Optional[int] = None, idx_dtype: int = IDX_U8,
                 gate_dtype: int = GATE_BF16, device: str = "cuda:0", host_staging: bool = False, flags: int = 0,
                 plan_only: bool = False):
        self.lib = load_library()
        self.device = torch.device(device)
        self.dims = GrouterDims(T, d, ffn, E_src, E_src if E_tgt is None else E_tgt, k, idx_dtype, gate_dtype, flags)
        self.T, self.d, self.ffn, self.k = T, d, ffn, k
        self.T_active = T
        self.E_src, self.E_tgt = E_src, self.dims.E_tgt
        self.R = T * k
        with torch.cuda.device(self.device):
            h = ctypes.c_void_p()
            _check(self.lib.grouter_create(ctypes.byref(h), ctypes.byref(self.dims)), "grouter_create")
            self.ctx = h
            n = self.lib.grouter_workspace_bytes(ctypes.byref(self.dims))
            if n == 0:
                raise GrouterError(-3, "grouter_workspace_bytes")
            self.workspace_bytes = n
            if host_staging:
                n += self.lib.grouter_host_staging_bytes(ctypes.byref(self.dims))
            # plan_only: the caller only builds plans with this context (no forward/backward), so no workspace is needed
            self.workspace = None if plan_only else torch.empty(n, dtype=torch.uint8, device=self.device)
        i32 = dict(dtype=torch.int32, device=self.device)
        self.counts = torch.empty(self.E_tgt, **i32)
        self.offsets = torch.empty(self.E_tgt + 1, **i32)
        self.row_to_slot = torch.empty(self.R, **i32)
        self.slot_to_row = torch.empty(self.R, **i32)

    def close(self) -> None:
        if getattr(self, "ctx", None):
            self.lib.grouter_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def plan(self, idx: torch.Tensor, fold_map: Optional[torch.Tensor] = None):
        """idx [T,k] uint8/int32 (device); fold_map [E_src] int32 or None.  Results land in
        self.counts / offsets / row_to_slot / slot_to_row."""
        _check(self.lib.grouter_plan(self.ctx, _ptr(idx), _ptr(fold_map), _ptr(self.counts), _ptr(self.offsets),
                                     _ptr(self.row_to_slot), _ptr(self.slot_to_row), _stream()), "grouter_plan")
        n = self.T_active * self.k
        return self.counts, self.offsets, self.row_to_slot[:n], self.slot_to_row[:n]

    def forward(self, X, gates, W_gu, W_d, Y=None):
        if Y is None:
            Y = torch.empty_like(X)
        _check(self.lib.grouter_moe_fwd(self.ctx, _ptr(X), _ptr(gates), _ptr(W_gu), _ptr(W_d), _ptr(Y), _ptr(self.workspace),
                                        _stream()), "grouter_moe_fwd")
        return Y

    def backward(self, dY, X, gates, W_gu, W_d, dX=None, dW_gu=None, dW_d=None, dgates=None):
        f32 = dict(dtype=torch.float32, device=self.device)
        dX = torch.empty_like(X) if dX is None else dX
        dW_gu = torch.empty(W_gu.shape, **f32) if dW_gu is None else dW_gu
        dW_d = torch.empty(W_d.shape, **f32) if dW_d is None else dW_d
        dgates = torch.empty((self.T_active, self.k), **f32) if dgates is None else dgates
        _check(self.lib.grouter_moe_bwd(self.ctx, _ptr(dY), _ptr(X), _ptr(gates), _ptr(W_gu), _ptr(W_d), _ptr(dX), _ptr(dW_gu),
                                        _ptr(dW_d), _ptr(dgates), _ptr(self.workspace), _stream()), "grouter_moe_bwd")
        return dX, dW_gu, dW_d, dgates

    def host_wait(self, steps_in_flight: int = 0) -> None:
        """Blocks until all but the `steps_in_flight` (0 or 1) most recent step_host calls are complete."""
        _check(self.lib.grouter_host_wait(self.ctx, steps_in_flight), "grouter_host_wait")

    def step_host(self, idx_h, gates_h, X_h, dY_h, fold_map, W_gu, W_d, Y_h, dX_h, dgates_h, dW_gu, dW_d):
        """Whole step from pinned host tensors (idx, gates, X, dY in; Y, dX, dgates out).  Asynchronous: read the
        outputs (and reuse the inputs) only after host_wait() reports the step complete."""
        _check(self.lib.grouter_moe_step_host(self.ctx, _ptr(idx_h), _ptr(gates_h), _ptr(X_h), _ptr(dY_h), _ptr(fold_map), _ptr(W_gu),
                                              _ptr(W_d), _ptr(Y_h), _ptr(dX_h), _ptr(dgates_h), _ptr(dW_gu), _ptr(dW_d),
                                              _ptr(self.workspace), _stream()), "grouter_moe_step_host")

    def timing_enable(self, n_records: int) -> None:
        _check(self.lib.grouter_timing_enable(self.ctx, n_records), "grouter_timing_enable")

    def timing_gap(self, microseconds: int) -> None:
        """Idle time after every timed kernel (0 = none): kernels are then measured one at a time on a rested GPU."""
        _check(self.lib.grouter_timing_gap(self.ctx, microseconds), "grouter_timing_gap")

    def wgrad_chunk_rows(self) -> int:
        """Rows of one expert that the weight-gradient products contract in one piece."""
        return int(self.lib.grouter_wgrad_chunk_rows(self.ctx))

    def gemm_cycles_enable(self, on: bool) -> None:
        _check(self.lib.grouter_gemm_cycles_enable(self.ctx, 1 if on else 0), "grouter_gemm_cycles_enable")

    def gemm_cycles_read(self):
        """-> {GEMM name: dict(cycles, wait_operands, wait_accumulator, tiles, k_steps)} summed over CTA pairs and launches
        since the last read; synchronises the current stream."""
        buf = (ctypes.c_uint64 * 30)()
        _check(self.lib.grouter_gemm_cycles_read(self.ctx, _stream(), buf), "grouter_gemm_cycles_read")
        names = ["gemm_up_swiglu", "gemm_down", "gemm_dH", "gemm_dX", "wgrad_down", "wgrad_gate_up"]
        keys = ["cycles", "wait_operands", "wait_accumulator", "tiles", "k_steps"]
        return {n: {k: int(buf[5 * i + j]) for j, k in enumerate(keys)} for i, n in enumerate(names)}

    def ep_dispatch_rows(self, src, gates, rows):
        """rows[slot_to_row[s], :] = gate_s * src[token of s, :] (gates None: copy); rows [T*k, d] bf16."""
        _check(self.lib.grouter_ep_dispatch_rows(self.ctx, _ptr(src), _ptr(gates), _ptr(rows), _stream()), "grouter_ep_dispatch_rows")
        return rows

    def ep_combine_rows(self, rows, gates=None, out=None, dY=None, dgates=None):
        """out[t, :] = sum_j gate * rows[slot_to_row[t*k+j], :] and/or dgates[t, j] = <dY[t, :], rows[slot_to_row[t*k+j], :]>."""
        _check(self.lib.grouter_ep_combine_rows(self.ctx, _ptr(rows), _ptr(gates), _ptr(out), _ptr(dY), _ptr(dgates), _stream()),
               "grouter_ep_combine_rows")

    def set_active_tokens(self, tokens: int) -> None:
        """Later calls work on the first `tokens` tokens (<= the T the layer was created for): pass [tokens, ...] tensors.
        The plan outputs are views of the first entries of self.counts / offsets / row_to_slot / slot_to_row."""
        _check(self.lib.grouter_set_active_tokens(self.ctx, tokens), "grouter_set_active_tokens")
        self.T_active = tokens

    def set_overlap(self, on: bool) -> None:
        """Bandwidth-bound kernels of the backward pass beside the GEMMs (default) or in line."""
        _check(self.lib.grouter_set_overlap(self.ctx, 1 if on else 0), "grouter_set_overlap")

    def set_wait_limit(self, microseconds: int) -> None:
        """Limit of every bounded device-side wait of this context's later launches."""
        _check(self.lib.grouter_set_wait_limit(self.ctx, microseconds), "grouter_set_wait_limit")

    def wait_selftest(self, limit_microseconds: int) -> int:
        """One bounded wait that cannot succeed; returns the microseconds the kernel waited.  Leaves GROUTER_ERR_TIMEOUT in
        the status word (read and cleared by status())."""
        waited = ctypes.c_int64(0)
        _check(self.lib.grouter_wait_selftest(self.ctx, limit_microseconds, ctypes.byref(waited), _stream()), "grouter_wait_selftest")
        return int(waited.value)

    def timing_read(self):
        """-> {kernel name: (total ms, launches)} since the last read; synchronises the current stream."""
        n = len(KERNEL_SLOTS)
        ms = (ctypes.c_float * n)()
        cnt = (ctypes.c_int32 * n)()
        _check(self.lib.grouter_timing_read(self.ctx, _stream(), ms, cnt), "grouter_timing_read")
        return {KERNEL_SLOTS[i]: (float(ms[i]), int(cnt[i])) for i in range(n)}

    def status(self) -> int:
        """Synchronises the current stream; returns 0 or a negative GROUTER_ERR_* device status."""
        return self.lib.grouter_status(self.ctx, _stream())

    def check_status(self) -> None:
        _check(self.status(), "device status")


def route(H: torch.Tensor, W_s: torch.Tensor, fold_map: Optional[torch.Tensor], E_tgt: int, k: int, norm: int = NORM_SOFTMAX,
          want_scores: bool = False):
    """Router head (grouter_route): H [T,d_h] bf16, W_s [E_src,d_h] bf16 -> (idx uint8 [T,k], gates bf16 [T,k],
    folded scores f32 [T,E_tgt] or None).  Raises on a device-side status."""
    lib = load_library()
    T, d_h = H.shape
    E_src = W_s.shape[0]
    dev = H.device
    idx = torch.empty((T, k), dtype=torch.uint8, device=dev)
    gates = torch.empty((T, k), dtype=torch.bfloat16, device=dev)
    scores = torch.empty((T, E_tgt), dtype=torch.float32, device=dev) if want_scores else None
    ws = torch.empty(max(1, lib.grouter_route_workspace_bytes(T, E_src, E_tgt)), dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    with torch.cuda.device(dev):
        _check(lib.grouter_route(_ptr(H), _ptr(W_s), _ptr(fold_map), T, d_h, E_src, E_tgt, k, norm, _ptr(idx), _ptr(gates), _ptr(scores),
                                 _ptr(ws), _ptr(status), _stream()), "grouter_route")
        torch.cuda.synchronize(dev)
    st = int(status.item())
    if st != 0:
        raise GrouterError(-7 if st & 2 else -6, "grouter_route device status")
    return idx, gates, scores


def routing_stats(idx: torch.Tensor, E: int, seq_len: int, node_of_expert: Optional[torch.Tensor] = None, n_nodes: int = 0):
    """grouter_routing_stats: -> dict(loads, coact, phi, max_vio[, local_tokens, best_node]) of device tensors."""
    lib = load_library()
    T, k = idx.shape
    dev = idx.device
    S = T // max(seq_len, 1)
    i32 = dict(dtype=torch.int32, device=dev)
    out = dict(loads=torch.empty(E, **i32), coact=torch.empty((E, E), **i32), phi=torch.empty((S, E), dtype=torch.float32, device=dev),
               max_vio=torch.empty(1, dtype=torch.float32, device=dev))
    if node_of_expert is not None:
        out["local_tokens"] = torch.empty((S, n_nodes), **i32)
        out["best_node"] = torch.empty(S, **i32)
    status = torch.zeros(1, **i32)
    with torch.cuda.device(dev):
        _check(lib.grouter_routing_stats(_ptr(idx), IDX_U8 if idx.dtype == torch.uint8 else IDX_I32, T, k, E, seq_len, _ptr(node_of_expert),
                                         n_nodes, _ptr(out["loads"]), _ptr(out["coact"]), _ptr(out["phi"]), _ptr(out["max_vio"]),
                                         _ptr(out.get("local_tokens")), _ptr(out.get("best_node")), _ptr(status), _stream()),
               "grouter_routing_stats")
        torch.cuda.synchronize(dev)
    out["status"] = int(status.item())
    return out


def fold_greedy(coact, E_tgt: int):
    """grouter_fold_greedy_host: host int32 co-activation matrix [E_src,E_src] (numpy) -> fold_map int32 [E_src] (numpy)."""
    import numpy as np
    lib = load_library()
    P = np.ascontiguousarray(coact, dtype=np.int32)
    fold = np.empty(P.shape[0], dtype=np.int32)
    _check(lib.grouter_fold_greedy_host(P.ctypes.data, P.shape[0], E_tgt, fold.ctypes.data), "grouter_fold_greedy_host")
    return fold


def plan_noalloc(idx: torch.Tensor, fold_map: Optional[torch.Tensor], E_src: int, E_tgt: int, out=None, status=None,
                 null_status: bool = False):
    """Routing plan without a context and without any device allocation inside the library (grouter_plan_noalloc).

    For hosts that may not allocate: pass `out` = (counts[E_tgt], offsets[E_tgt+1], row_to_slot[R], slot_to_row[R])
    int32 device tensors and an int32[1] `status` tensor you already own, and nothing is allocated anywhere.
    When they are omitted this wrapper creates them with torch for convenience (the library still allocates nothing).
    With `null_status` the library is given no status word at all (it then keeps the bits in its own scratch and the
    caller learns nothing about bad ids); the last element of the result is None.
    Limits: T*k <= 524288, E_tgt <= 256.  Calls share one scratch array per GPU: keep them ordered on one stream.
    Returns (counts, offsets, row_to_slot, slot_to_row, status)."""
    lib = load_library()
    T, k = idx.shape
    dt = IDX_U8 if idx.dtype == torch.uint8 else IDX_I32
    i32 = dict(dtype=torch.int32, device=idx.device)
    if out is None:
        out = (torch.empty(E_tgt, **i32), torch.empty(E_tgt + 1, **i32), torch.empty(T * k, **i32), torch.empty(T * k, **i32))
    if status is None and not null_status:
        status = torch.empty(1, **i32)
    with torch.cuda.device(idx.device):
        _check(lib.grouter_plan_noalloc(_ptr(idx), dt, _ptr(fold_map), T, k, E_src, E_tgt, _ptr(out[0]), _ptr(out[1]), _ptr(out[2]),
                                        _ptr(out[3]), _ptr(status), _stream()), "grouter_plan_noalloc")
    return (*out, status)


def dense_gemm(A: torch.Tensor, a_mn_major: bool, B: torch.Tensor, b_mn_major: bool, M: int, N: int, K: int) -> torch.Tensor:
    """C[M,N] f32 = A*B on the tcgen05 core (component check).  A is [M,K] or, MN-major, [K,M]; B is [N,K] or [K,N]."""
    lib = load_library()
    C = torch.empty((M, N), dtype=torch.float32, device=A.device)
    status = torch.zeros(1, dtype=torch.int32, device=A.device)
    _check(lib.grouter_dense_gemm(_ptr(A), int(a_mn_major), _ptr(B), int(b_mn_major), _ptr(C), M, N, K, _ptr(status), _stream()),
           "grouter_dense_gemm")
    torch.cuda.synchronize(A.device)
    if int(status.item()) != 0:
        raise GrouterError(-7, "grouter_dense_gemm device status")
    return C
