"""Host logic of the sequence-parallel exchange with more than one rank, on the CPU: the split sizes that
ExchangePlan hands to the two all-to-alls must route the reference permutations (oracle side) so that every rank
ends up with the head shard of the full tensors, and gets back exactly its token rows.  gloo, world sizes 2 and 3
(ragged shards)."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, total, heads, D, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    from oracle import exchange_oracle as xo
    from paper_2609_35110_b200.sequence_parallel import ExchangePlan
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        g = torch.Generator().manual_seed(5)
        full = [torch.randint(-30000, 30000, (total, heads, D), generator=g, dtype=torch.int32) for _ in range(3)]
        xp = ExchangePlan(total, heads, D, world, rank, out_record_bytes=4 * D)
        a, b = xp.first_token, xp.first_token + xp.n_local
        hl = heads // world
        # forward exchange: reference pack of the local shard, one all-to-all with the plan's splits
        send = xo.pack_qkv_reference(full[0][a:b], full[1][a:b], full[2][a:b], world)       # [G, n_local, 3, hl, D]
        recv = torch.empty((total, 3, hl, D), dtype=torch.int32)
        dist.all_to_all_single(recv.view(-1), send.view(-1), xp.qkv_recv_splits, xp.qkv_send_splits)
        for w in range(3):
            assert torch.equal(recv[:, w], full[w][:, rank * hl:(rank + 1) * hl]), f"rank {rank}: head shard of tensor {w}"
        # "attention" = q + 2k - v on the shard (elementwise, so the expected full result is known)
        out_shard = (recv[:, 0] + 2 * recv[:, 1] - recv[:, 2]).contiguous()                 # [total, hl, D]
        back = torch.empty((world, xp.n_local, hl, D), dtype=torch.int32)
        dist.all_to_all_single(back.view(-1), out_shard.view(-1), xp.out_recv_splits, xp.out_send_splits)
        merged = xo.merge_heads_reference(back)
        want = (full[0] + 2 * full[1] - full[2])[a:b]
        assert torch.equal(merged, want), f"rank {rank}: returned rows"
        assert xp.tok_begin[rank] == a and xp.tok_begin[-1] == total
        # one head group of every shard (here: the last head of each): same routing with the group's split sizes
        if hl > 1:
            gs, gr, _, _ = xp.splits(1)
            sel = torch.tensor([r * hl + hl - 1 for r in range(world)])
            send_g = xo.pack_qkv_reference(full[0][a:b][:, sel], full[1][a:b][:, sel], full[2][a:b][:, sel], world)
            recv_g = torch.empty((total, 3, 1, D), dtype=torch.int32)
            dist.all_to_all_single(recv_g.view(-1), send_g.contiguous().view(-1), gr, gs)
            for w in range(3):
                assert torch.equal(recv_g[:, w, 0], full[w][:, rank * hl + hl - 1])
        open(os.path.join(out_dir, f"ok{rank}"), "w").write("ok")
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world,total,heads", [(2, 13, 4), (3, 10, 6), (2, 1, 2)])
def test_split_sizes_route_the_exchange(tmp_path, world, total, heads):
    port = 31000 + (os.getpid() % 2000) + world * 7 + total
    mp.spawn(_worker, args=(world, port, total, heads, 8, str(tmp_path)), nprocs=world, join=True)
    for r in range(world):
        assert (tmp_path / f"ok{r}").exists()


def test_exchange_plan_rejects_bad_shapes():
    from paper_2609_35110_b200.sequence_parallel import ExchangePlan, shard_ranges
    with pytest.raises(ValueError):
        ExchangePlan(100, 6, 64, 4, 0, 128)          # heads not divisible
    with pytest.raises(ValueError):
        ExchangePlan(100, 8, 64, 16, 0, 128)         # more ranks than the library addresses
    with pytest.raises(ValueError):
        ExchangePlan(100, 8, 64, 4, 4, 128)          # rank out of range
    xp = ExchangePlan(111856, 40, 128, 8, 7, 128)
    assert sum(xp.qkv_recv_splits) == 111856 * 3 * 5 * 128 and len(xp.out_send_splits) == 8
    assert sum(xp.out_send_splits) == 111856 * 5 * 128 and xp.out_recv_splits == [xp.n_local * 5 * 128] * 8
    assert xp.n_local == 111856 - 7 * 13982 and shard_ranges(111856, 8)[7] == (97874, 111856)
