"""The N>1 path on CPU: two gloo ranks verify their row blocks (the oracle stands in for the
kernels here) and the gathered result equals the unsharded one."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2502_05202_b200 import shard, workload as wl


def test_row_blocks_partition_the_batch():
    for B in (0, 1, 2, 7, 64, 255):
        for world in (1, 2, 3, 8):
            blocks = shard.row_blocks(B, world)
            assert blocks[0][0] == 0 and blocks[-1][1] == B
            assert all(blocks[i][1] == blocks[i + 1][0] for i in range(world - 1))
            sizes = [e - b for b, e in blocks]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        shard.row_block(4, 2, 2)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, B, out_path):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = wl.tiny_config(B=B, K=3, V_t=700, V_d=600, dtype=wl.BF16, f_mapped=0.6,
                         temperatures=(0.7, 1.0), greedy_rows="interleaved", seed=91)
    b, e = shard.row_block(B, rank, world)
    batch = wl.make_batch(cfg, rows=range(b, e), threads=1)
    o = oracle.verify(batch["target_logits"], batch["drafter_logits"], batch["id_map"], batch["draft_ids"],
                      batch["temperature"], batch["uniforms"])
    local = torch.from_numpy(np.stack([o["accepted"], o["next_token"]], axis=1))
    full = shard.gather_rows(local, B)
    if rank == 0:
        np.save(out_path, full.numpy())
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("B", [7, 8])
def test_two_ranks_match_one(tmp_path, B):
    out = str(tmp_path / "gathered.npy")
    mp.spawn(_worker, args=(2, _free_port(), B, out), nprocs=2, join=True)
    got = np.load(out)
    cfg = wl.tiny_config(B=B, K=3, V_t=700, V_d=600, dtype=wl.BF16, f_mapped=0.6,
                         temperatures=(0.7, 1.0), greedy_rows="interleaved", seed=91)
    batch = wl.make_batch(cfg)
    o = oracle.verify(batch["target_logits"], batch["drafter_logits"], batch["id_map"], batch["draft_ids"],
                      batch["temperature"], batch["uniforms"])
    np.testing.assert_array_equal(got[:, 0], o["accepted"])
    np.testing.assert_array_equal(got[:, 1], o["next_token"])
