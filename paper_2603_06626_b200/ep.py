"""Expert-parallel form of the layer: experts split over ranks, routed rows exchanged with split sizes that are known
before the step (the routing comes from the cache, not from the layer).

Host-side wiring only: every step that touches tensor data runs in the CUDA library (plan, row dispatch / combine,
the experts' grouped GEMMs) or in the collective (an all-to-all over rows into the receiver's own memory).  The layer
is cut into phases so that the caller puts the exchanges between them; `run_step` does that with torch.distributed.

    forward   fwd_dispatch -> exchange -> fwd_expert -> exchange back -> fwd_combine
    backward  bwd_dispatch -> exchange -> bwd_expert -> exchange back -> bwd_combine
"""
from __future__ import annotations

from typing import Optional, Sequence

import numpy as np
import torch

from . import binding


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def relabel_experts(expert_rank: Sequence[int], world: int):
    """-> (relabel [E], first_expert [world+1]): new expert ids under which every rank owns a contiguous range."""
    lib = binding.load_library()
    owner = _i32(expert_rank)
    relabel = np.empty(owner.shape[0], dtype=np.int32)
    first = np.empty(world + 1, dtype=np.int32)
    rc = lib.grouter_ep_relabel_host(owner.shape[0], world, owner.ctypes.data, relabel.ctypes.data, first.ctypes.data)
    if rc != 0:
        raise binding.GrouterError(rc, "grouter_ep_relabel_host")
    return relabel, first


def exchange_layout(world: int, rank: int, first_expert, counts_all):
    """Per-peer row counts / offsets of `rank` from every rank's expert histogram (counts_all [world, E], new ids)."""
    lib = binding.load_library()
    first = _i32(first_expert)
    counts = _i32(counts_all)
    E = counts.shape[1]
    if not 0 <= rank < world or first.shape[0] != world + 1 or counts.shape[0] != world:
        raise binding.GrouterError(-1, "grouter_ep_layout_host")
    n_local = max(int(first[rank + 1] - first[rank]), 0)
    out = dict(send_counts=np.empty(world, np.int32), send_offsets=np.empty(world + 1, np.int32),
               recv_counts=np.empty(world, np.int32), recv_offsets=np.empty(world + 1, np.int32),
               recv_seg_offsets=np.empty(world * n_local + 1, np.int32))
    rc = lib.grouter_ep_layout_host(world, rank, E, first.ctypes.data, counts.ctypes.data, out["send_counts"].ctypes.data,
                                    out["send_offsets"].ctypes.data, out["recv_counts"].ctypes.data, out["recv_offsets"].ctypes.data,
                                    out["recv_seg_offsets"].ctypes.data)
    if rc != 0:
        raise binding.GrouterError(rc, "grouter_ep_layout_host")
    out["n_local"] = n_local
    out["first_local"] = int(first[rank])
    return out


def place_samples(idx: torch.Tensor, E: int, seq_len: int, expert_rank, world: int):
    """Sample placement of Algorithm 1 for expert parallelism: every sample (run of seq_len tokens of the routing table
    `idx`, a device tensor) goes to the rank that owns at least one kept expert of most of its tokens.
    -> (best_rank [S] int32, local_tokens [S, world] int32), both on the host; computed by grouter_routing_stats."""
    node = torch.from_numpy(_i32(expert_rank)).to(idx.device)
    out = binding.routing_stats(idx, E, seq_len, node, world)
    if out["status"] != 0:
        raise binding.GrouterError(-6, "grouter_routing_stats device status")
    return out["best_node"].cpu().numpy(), out["local_tokens"].cpu().numpy()


def rows_crossing_ranks(idx: np.ndarray, expert_rank, sample_rank, seq_len: int) -> int:
    """Routed rows whose expert lives on another rank than their token, for a given sample -> rank assignment (a
    statistic of a routing table for reporting, host side: these are the rows an expert-parallel step must transfer)."""
    tok_rank = np.repeat(np.asarray(sample_rank), seq_len)
    return int((np.asarray(expert_rank)[np.asarray(idx).astype(np.int64)] != tok_rank[:, None]).sum())


class ExpertParallelRank:
    """One rank of the expert-parallel layer: its T tokens (source side) and its experts (expert side)."""

    def __init__(self, rank: int, world: int, T: int, d: int, ffn: int, E_src: int, E_tgt: int, k: int, first_expert,
                 device: str = "cuda:0", idx_dtype: int = binding.IDX_U8, gate_dtype: int = binding.GATE_BF16,
                 max_recv_rows: Optional[int] = None):
        self.rank, self.world, self.T, self.d, self.ffn, self.k = rank, world, T, d, ffn, k
        self.E_tgt = E_tgt
        self.first_expert = _i32(first_expert)
        self.device = torch.device(device)
        # source side: the plan over this rank's tokens and the row dispatch / combine (no GEMM runs on this context)
        self.src = binding.GrouterLayer(T, d, ffn, E_src, k, E_tgt=E_tgt, idx_dtype=idx_dtype, gate_dtype=gate_dtype, device=device,
                                        plan_only=True)
        self.R = T * k
        self.send_rows = torch.empty((self.R, d), dtype=torch.bfloat16, device=self.device)     # dispatched rows (fwd: X, bwd: g*dY)
        self.back_rows = torch.empty((self.R, d), dtype=torch.bfloat16, device=self.device)     # returned rows (fwd: O, bwd: dX rows)
        self.fwd_back = torch.empty((self.R, d), dtype=torch.bfloat16, device=self.device)      # the forward's returned rows, kept for dgates
        self.layout = None
        self.exp = None
        # With max_recv_rows the expert side is laid out once for that many received rows and serves every routing
        # table that sends this rank no more (grouter_set_active_tokens per table); without it, it is rebuilt per table.
        self.max_recv_rows = max_recv_rows
        self.n_local = int(self.first_expert[rank + 1] - self.first_expert[rank])
        self.exp_active = None
        if max_recv_rows is not None:
            self._build_expert_side(max_recv_rows)

    def close(self):
        self.src.close()
        if self.exp is not None:
            self.exp.close()

    def _build_expert_side(self, rows: int) -> None:
        dev = self.device
        i8 = self.n_local <= 256
        self.recv_rows = torch.empty((max(rows, 1), self.d), dtype=torch.bfloat16, device=dev)    # what the experts receive
        self.recv_rows2 = torch.empty((max(rows, 1), self.d), dtype=torch.bfloat16, device=dev)   # ... in the backward pass
        self.out_rows = torch.empty((max(rows, 1), self.d), dtype=torch.bfloat16, device=dev)     # what the experts send back
        if rows == 0 or self.n_local == 0:
            return
        self.exp = binding.GrouterLayer(rows, self.d, self.ffn, self.n_local, 1, idx_dtype=binding.IDX_U8 if i8 else binding.IDX_I32,
                                        gate_dtype=binding.GATE_BF16, device=str(dev))
        self.exp_ids = torch.empty((rows, 1), dtype=torch.uint8 if i8 else torch.int32, device=dev)
        self.unit_gates = torch.ones((rows, 1), dtype=torch.bfloat16, device=dev)
        self.exp_dgates = torch.empty((rows, 1), dtype=torch.float32, device=dev)

    def set_tokens(self, T: int) -> None:
        """This rank brings T tokens (at most what it was created for) to the next routing table."""
        self.src.set_active_tokens(T)
        self.T = T

    # ---- set-up per routing table (all of it is known before the step) ----
    def plan(self, idx: torch.Tensor, fold_map: Optional[torch.Tensor]):
        """Plan over this rank's tokens; fold_map must already map to the relabelled expert ids.  -> counts (device)."""
        return self.src.plan(idx, fold_map)[0]

    def set_counts(self, counts_all) -> None:
        """counts_all [world, E]: every rank's plan counts (from the routing cache, or gathered ahead of the step)."""
        lay = exchange_layout(self.world, self.rank, self.first_expert, counts_all)
        self.layout = lay
        n_recv = int(lay["recv_offsets"][-1])
        self.n_recv = n_recv
        dev = self.device
        if self.max_recv_rows is None:
            if self.exp is not None:
                self.exp.close()
                self.exp = None
            self._build_expert_side(n_recv)
        elif n_recv > self.max_recv_rows:
            raise ValueError(f"{n_recv} rows arrive at rank {self.rank}, more than the {self.max_recv_rows} it was laid out for")
        self.exp_active = self.exp if n_recv > 0 else None
        if self.exp_active is None:
            return
        n_local = lay["n_local"]
        i8 = n_local <= 256
        self.exp.set_active_tokens(n_recv)
        seg = torch.from_numpy(lay["recv_seg_offsets"]).to(dev)
        with torch.cuda.device(dev):
            rc = self.src.lib.grouter_ep_expand_ids(seg.data_ptr(), self.world * n_local, n_local, n_recv,
                                                    binding.IDX_U8 if i8 else binding.IDX_I32, self.exp_ids.data_ptr(),
                                                    torch.cuda.current_stream().cuda_stream)
        if rc != 0:
            raise binding.GrouterError(rc, "grouter_ep_expand_ids")
        self.exp.plan(self.exp_ids)

    # ---- phases ----
    def fwd_dispatch(self, X):
        return self.src.ep_dispatch_rows(X, None, self.send_rows)

    def fwd_expert(self, W_gu_local, W_d_local):
        """Runs this rank's experts on self.recv_rows -> self.out_rows."""
        if self.exp_active is not None:
            self.exp.forward(self.recv_rows, self.unit_gates, W_gu_local, W_d_local, self.out_rows)
        return self.out_rows

    def fwd_combine(self, gates, Y=None):
        """self.fwd_back (the returned expert outputs; kept for the backward pass's dgates) -> Y [T, d]."""
        Y = torch.empty((self.T, self.d), dtype=torch.bfloat16, device=self.device) if Y is None else Y
        self.src.ep_combine_rows(self.fwd_back, gates, out=Y)
        return Y

    def bwd_dispatch(self, dY, gates):
        return self.src.ep_dispatch_rows(dY, gates, self.send_rows)

    def bwd_expert(self, W_gu_local, W_d_local, dW_gu=None, dW_d=None):
        """Backward of this rank's experts: self.recv_rows2 (gate-scaled dY rows) -> self.out_rows (dX rows), dW of the local experts."""
        f32 = dict(dtype=torch.float32, device=self.device)
        dW_gu = torch.zeros(W_gu_local.shape, **f32) if dW_gu is None else dW_gu
        dW_d = torch.zeros(W_d_local.shape, **f32) if dW_d is None else dW_d
        if self.exp_active is not None:
            self.exp.backward(self.recv_rows2, self.recv_rows, self.unit_gates, W_gu_local, W_d_local, self.out_rows, dW_gu, dW_d,
                              self.exp_dgates)
        else:
            dW_gu.zero_()
            dW_d.zero_()
        return self.out_rows, dW_gu, dW_d

    def bwd_combine(self, dY, dX=None, dgates=None):
        """self.back_rows (returned input-gradient rows) -> dX; dgates from the forward's returned rows and dY."""
        dX = torch.empty((self.T, self.d), dtype=torch.bfloat16, device=self.device) if dX is None else dX
        dgates = torch.empty((self.T, self.k), dtype=torch.float32, device=self.device) if dgates is None else dgates
        self.src.ep_combine_rows(self.back_rows, None, out=dX)
        self.src.ep_combine_rows(self.fwd_back, None, out=None, dY=dY, dgates=dgates)
        return dX, dgates

    # ---- the exchange: an all-to-all over rows with split sizes known from the layout ----
    def exchange(self, send: torch.Tensor, recv: torch.Tensor, to_experts: bool, group=None) -> None:
        """to_experts: send = this rank's dispatched rows, recv = the rows for its experts; otherwise the way back."""
        import torch.distributed as dist
        lay = self.layout
        out_split = lay["send_counts"] if to_experts else lay["recv_counts"]
        in_split = lay["recv_counts"] if to_experts else lay["send_counts"]
        n_out, n_in = int(out_split.sum()), int(in_split.sum())
        if self.world == 1:
            recv[:n_in].copy_(send[:n_out])
            return
        dist.all_to_all_single(recv[:n_in], send[:n_out], output_split_sizes=[int(v) for v in in_split],
                               input_split_sizes=[int(v) for v in out_split], group=group)

    def run_step(self, X, dY, gates, W_gu_local, W_d_local, Y=None, dX=None, dgates=None, dW_gu=None, dW_d=None, group=None):
        """One forward + backward with the four exchanges (needs plan() and set_counts() first)."""
        self.fwd_dispatch(X)
        self.exchange(self.send_rows, self.recv_rows, True, group)
        self.fwd_expert(W_gu_local, W_d_local)
        self.exchange(self.out_rows, self.fwd_back, False, group)
        Y = self.fwd_combine(gates, Y)
        self.bwd_dispatch(dY, gates)
        self.exchange(self.send_rows, self.recv_rows2, True, group)
        _, dW_gu, dW_d = self.bwd_expert(W_gu_local, W_d_local, dW_gu, dW_d)
        self.exchange(self.out_rows, self.back_rows, False, group)
        dX, dgates = self.bwd_combine(dY, dX, dgates)
        return Y, dX, dgates, dW_gu, dW_d
