"""Expert-parallel bookkeeping on CPU: world-size-2 and -4 gloo ranks, one process each.

Every rank works out its per-peer send and receive row counts from the ranks' expert histograms alone (the C ABI's host
routines), then really exchanges row tags with an all-to-all using those sizes.  What arrives is compared with the
answer recomputed from the concatenated routing table by the oracle: exactly the rows of every source rank whose
expert lives here, ordered by (source rank, expert, slot).  The way back returns every row to its own place."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import grouter_oracle as orc
from paper_2603_06626_b200 import ep


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _routing(rank, T, k, E):
    rng = np.random.default_rng(100 + rank)
    p = 1.0 / np.arange(1, E + 1) ** 0.8
    return np.stack([rng.choice(E, size=k, replace=False, p=p / p.sum()) for _ in range(T)]).astype(np.uint8)


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        T, k, E = 200 + 17 * rank, 3, 12                              # ranks own different numbers of tokens
        owner = np.array([(5 * e + 1) % world for e in range(E)])       # an arbitrary expert -> rank assignment
        if world == 4:
            owner[owner == 3] = 2                                       # rank 3 owns no expert at all
        relabel, first = ep.relabel_experts(owner, world)
        assert sorted(relabel.tolist()) == list(range(E))
        for r in range(world):                                          # contiguous ownership, old order kept within a rank
            mine = [e for e in range(E) if owner[e] == r]
            assert [int(relabel[e]) for e in mine] == list(range(first[r], first[r + 1]))
        idx = _routing(rank, T, k, E)
        counts, offsets, row_to_slot, slot_to_row = orc.plan(idx, relabel, E)
        gathered = [None] * world
        dist.all_gather_object(gathered, (idx, counts))                 # stands for reading the routing cache
        counts_all = np.stack([g[1] for g in gathered])
        lay = ep.exchange_layout(world, rank, first, counts_all)
        # the rows for peer p are a contiguous range of this rank's expert-ordered rows
        for p in range(world):
            assert lay["send_offsets"][p] == offsets[first[p]] and lay["send_counts"][p] == offsets[first[p + 1]] - offsets[first[p]]
        assert lay["send_offsets"][world] == T * k

        # really exchange: a row's tag names its source rank and slot
        tags = torch.from_numpy((rank << 20) + row_to_slot.astype(np.int64))
        recv = torch.empty(int(lay["recv_offsets"][world]), dtype=torch.int64)
        dist.all_to_all_single(recv, tags, output_split_sizes=lay["recv_counts"].tolist(), input_split_sizes=lay["send_counts"].tolist())
        want, seg = [], [0]
        for q in range(world):                                          # recomputed from the concatenated routing table
            rid = relabel[gathered[q][0].astype(np.int64)].reshape(-1)
            for e in range(first[rank], first[rank + 1]):
                slots = np.nonzero(rid == e)[0]
                want += [(q << 20) + int(s) for s in slots]
                seg.append(len(want))
        assert recv.tolist() == want
        assert lay["recv_seg_offsets"].tolist() == seg
        assert lay["recv_offsets"].tolist() == [seg[q * lay["n_local"]] for q in range(world)] + [len(want)]
        # the way back: every row returns to the place it left
        back = torch.empty(T * k, dtype=torch.int64)
        dist.all_to_all_single(back, recv + 1, output_split_sizes=lay["send_counts"].tolist(), input_split_sizes=lay["recv_counts"].tolist())
        assert torch.equal(back, tags + 1)
        total = torch.tensor([recv.numel()])
        dist.all_reduce(total)
        assert int(total) == sum(200 + 17 * r for r in range(world)) * k   # nothing lost, nothing doubled
        if rank == 0:
            np.save(os.path.join(out_dir, "ok.npy"), np.array([1]))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 4])
def test_split_sizes_from_the_plan_route_every_row(world, tmp_path):
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    assert os.path.exists(tmp_path / "ok.npy")


def test_layout_rejects_inconsistent_input():
    from paper_2603_06626_b200 import binding
    with pytest.raises(binding.GrouterError):
        ep.relabel_experts([0, 1, 5], 2)                                # owner out of range
    relabel, first = ep.relabel_experts([1, 0, 1, 0], 2)
    assert relabel.tolist() == [2, 0, 3, 1] and first.tolist() == [0, 2, 4]
    counts = np.array([[1, 2, 3, 4], [5, 6, 7, 8]])
    lay = ep.exchange_layout(2, 1, first, counts)
    assert lay["send_counts"].tolist() == [11, 15] and lay["recv_counts"].tolist() == [7, 15]
    assert lay["recv_seg_offsets"].tolist() == [0, 3, 7, 14, 22]
    with pytest.raises(binding.GrouterError):
        ep.exchange_layout(2, 2, first, counts)                         # rank outside the world
    with pytest.raises(binding.GrouterError):
        ep.exchange_layout(2, 0, [0, 3, 2], counts)                     # ranges must tile [0, E)


def test_layout_against_brute_force_on_random_cases():
    """Host bookkeeping against the definition written out with numpy, over random worlds, owner maps and histograms
    (some ranks without experts, some experts without rows)."""
    rng = np.random.default_rng(2024)
    for _ in range(60):
        world = int(rng.integers(1, 9))
        E = int(rng.integers(1, 40))
        owner = rng.integers(0, world, size=E)
        relabel, first = ep.relabel_experts(owner, world)
        assert sorted(relabel.tolist()) == list(range(E))
        new_owner = np.empty(E, dtype=np.int64)
        new_owner[relabel] = owner                                   # owner of every new id: non-decreasing
        assert np.all(np.diff(new_owner) >= 0)
        assert [int((new_owner == r).sum()) for r in range(world)] == np.diff(first).tolist()
        counts = rng.integers(0, 50, size=(world, E)) * (rng.random((world, E)) < 0.7)
        for rank in range(world):
            lay = ep.exchange_layout(world, rank, first, counts)
            send = [int(counts[rank, new_owner == p].sum()) for p in range(world)]
            recv = [int(counts[q, new_owner == rank].sum()) for q in range(world)]
            assert lay["send_counts"].tolist() == send and lay["recv_counts"].tolist() == recv
            assert lay["send_offsets"].tolist() == np.concatenate([[0], np.cumsum(send)]).tolist()
            assert lay["recv_offsets"].tolist() == np.concatenate([[0], np.cumsum(recv)]).tolist()
            seg = counts[:, new_owner == rank].reshape(-1)           # (source rank, local expert), source outermost
            assert lay["recv_seg_offsets"].tolist() == np.concatenate([[0], np.cumsum(seg)]).astype(int).tolist()
        # what every rank sends to p is what p receives
        lays = [ep.exchange_layout(world, r, first, counts) for r in range(world)]
        for p in range(world):
            assert [int(lays[q]["send_counts"][p]) for q in range(world)] == lays[p]["recv_counts"].tolist()
