"""world_size-2 checks of the multi-GPU host logic on CPU (gloo): sequence
sharding needs no exchange; sharding one sequence by KV range needs exactly
one all-gather of partial results followed by the log-sum-exp merge."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2609_37062_b200 import sharding
from paper_2609_37062_b200 import workloads as wl


def test_shard_ranges_partition_everything():
    for n in (0, 1, 7, 64, 257):
        for world in (1, 2, 3, 8):
            spans = [sharding.shard_range(n, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
            sizes = [e - b for b, e in spans]
            assert max(sizes) - min(sizes) <= 1
    assert sharding.shard_kv_range(100, 16, 2, 0) == (0, 64) and sharding.shard_kv_range(100, 16, 2, 1) == (64, 100)
    assert sharding.shard_kv_range(10, 16, 4, 3) == (10, 10)          # more ranks than pages: empty range


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, result_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # ---- sequence sharding: each rank attends its own sequences, nothing is exchanged
        w = wl.config_short_chat(batch=6)
        mine = sharding.shard_sequences(w.batch, world, rank)
        sub = wl.make_workload("shard", [int(w.seq_lens[i]) for i in mine], w.num_q_heads, w.num_kv_heads, w.head_dim,
                               seed=2, seq_uids=mine)
        out, _ = oracle.paged_decode_attention(oracle.PagedInputs.from_workload(sub), num_threads=2)
        np.save(os.path.join(result_dir, f"seq_{rank}.npy"), out)
        # ---- the timing reduction is a max over ranks
        assert sharding.max_over_ranks(1.0 + rank) == float(world)
        # ---- context parallel: one sequence split by KV range, one all-gather, then the merge
        long = wl.config_long(context=1000)
        inp = oracle.PagedInputs.from_workload(long)
        t0, t1 = sharding.shard_kv_range(1000, 16, world, rank)
        Hq, D = long.num_q_heads, long.head_dim
        mine_rec = torch.zeros(Hq, D + 2, dtype=torch.float64)
        for h in range(Hq):
            o, m, l = oracle.partial_attention(inp, 0, h, t0, t1)
            mine_rec[h, :D] = torch.from_numpy(o)
            mine_rec[h, D], mine_rec[h, D + 1] = m, l
        gathered = [torch.zeros_like(mine_rec) for _ in range(world)]
        dist.all_gather(gathered, mine_rec)                              # the single exchange step
        full, full_lse = oracle.paged_decode_attention(inp, num_threads=2)
        for h in range(Hq):
            parts = torch.stack([g[h] for g in gathered]).numpy()        # rank order = ascending token order
            merged, lse = oracle.merge_partials(parts[:, :D], parts[:, D], parts[:, D + 1])
            assert np.max(np.abs(merged - full[0, h])) < 1e-12 and abs(lse - full_lse[0, h]) < 1e-12
        # ---- the same through the helpers the GPU path uses: local tables per rank, normalised
        # outputs with their log-sum-exp, one gather; the merge is the oracle's here (no GPU)
        mix = wl.make_workload("cp", [1000, 40, 16, 333], 8, 2, 64, seed=11)
        bt, lens = sharding.shard_kv_tables(mix.block_table, mix.seq_lens, 16, world, rank)
        import dataclasses
        local = dataclasses.replace(mix, block_table=bt, seq_lens=lens, max_pages_per_seq=bt.shape[1])
        o_loc, lse_loc = oracle.paged_decode_attention(oracle.PagedInputs.from_workload(local), num_threads=2)
        outs, lses = sharding.gather_shards(torch.from_numpy(o_loc), torch.from_numpy(lse_loc))
        assert outs.shape == (world, 4, 8, 64) and lses.shape == (world, 4, 8)
        ref, ref_lse = oracle.paged_decode_attention(oracle.PagedInputs.from_workload(mix), num_threads=2)
        for b in range(4):
            for h in range(8):
                merged, lse = oracle.merge_partials(outs[:, b, h].numpy(), lses[:, b, h].numpy(), np.ones(world))
                assert np.max(np.abs(merged - ref[b, h])) < 1e-12 and abs(lse - ref_lse[b, h]) < 1e-12
    finally:
        dist.destroy_process_group()


def test_two_ranks_gloo(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    w = wl.config_short_chat(batch=6)
    full, _ = oracle.paged_decode_attention(oracle.PagedInputs.from_workload(w))
    got = np.concatenate([np.load(os.path.join(tmp_path, f"seq_{r}.npy")) for r in range(world)])
    assert np.array_equal(got, full)          # same sequences, same bits, whatever rank holds them
