"""The multi-GPU path on CPU: sequences are sharded over ranks by summed context length, every rank
works on its own shard with no exchange on the data path, and timing is reduced with MAX over ranks.
Two gloo ranks; the oracle stands in for the per-rank compute."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import pdattn_oracle as orc
from paper_2607_09207_b200 import workloads as W


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, tmp):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = W.make_config(2, num_seqs=10, len_div=8)                 # same seeded batch on every rank
        shards = W.balanced_shards(w.context_lens_host, world)
        mine = w.shard(shards[rank])
        out = torch.from_numpy(orc.decode_workload(mine, num_threads=2))
        # reassemble on rank 0: pad to the largest shard, gather, scatter rows back to their places
        nmax = max(len(s) for s in shards)
        pad = torch.zeros(nmax, *out.shape[1:], dtype=out.dtype)
        pad[: out.shape[0]] = out
        bufs = [torch.zeros_like(pad) for _ in range(world)] if rank == 0 else None
        dist.gather(pad, bufs, dst=0)
        # per-rank "step time": the slowest rank defines the job's time
        t = torch.tensor([1.0 + rank], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        assert t.item() == float(world)
        loads = torch.tensor([float(mine.logical_tokens())], dtype=torch.float64)
        total = loads.clone()
        dist.all_reduce(total, op=dist.ReduceOp.SUM)
        assert total.item() == float(w.logical_tokens())
        if rank == 0:
            full = np.zeros((w.num_seqs, w.num_q_heads, w.head_dim))
            for r in range(world):
                full[shards[r]] = bufs[r][: len(shards[r])].numpy()
            ref = orc.decode_workload(w, num_threads=2)
            assert np.array_equal(full, ref)
            open(os.path.join(tmp, "ok"), "w").write("ok")
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(300)
def test_two_ranks_shard_sequences_without_exchange(tmp_path):
    port = _free_port()
    mp.spawn(_rank_main, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    assert (tmp_path / "ok").exists()


def test_shard_keeps_rows_and_pools():
    w = W.make_config(3, num_seqs=16, len_div=8)
    sh = w.shard([3, 9, 10])
    assert sh.num_seqs == 3 and sh.k_cache.data_ptr() == w.k_cache.data_ptr()
    assert sh.context_lens_host.tolist() == w.context_lens_host[[3, 9, 10]].tolist()
    ref = orc.decode_workload(w, num_threads=2)
    assert np.array_equal(orc.decode_workload(sh, num_threads=2), ref[[3, 9, 10]])
