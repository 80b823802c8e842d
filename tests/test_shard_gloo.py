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


# ---------------------------------------------------------------------------
# vocabulary shards: the exchange protocol of tli_shard_* on two gloo ranks
# ---------------------------------------------------------------------------
#
# No GPU here, so plain numpy (fp64) stands in for the four local calls; what is under test is the
# protocol around them: which sums cross shards, who owns a drafted token's logits, that every rank
# takes the same decisions from the gathered records, and that exactly one rank reports each token.

def test_vocab_slices_partition_the_ids():
    for V in (1, 5, 1000, 152064):
        for world in (1, 2, 3, 8):
            parts = [shard.vocab_slice(V, r, world) for r in range(world)]
            assert sum(c for _, c, _ in parts) == V
            assert all(parts[r][0] == min(V, r * parts[0][2]) for r in range(world))
            assert all(w == -(-V // world) for _, _, w in parts)


def _np_shard_worker(rank, world, port, out_path):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = wl.tiny_config(B=6, K=3, V_t=211, V_d=157, dtype=wl.F32, f_mapped=0.6, sigma_d=0.4,
                         temperatures=(0.7, 1.0), seed=93)
    batch = wl.make_batch(cfg, threads=1)
    B, K = cfg.B, cfg.K
    m = batch["id_map"]
    tau, u, draft = batch["temperature"].astype(np.float64), batch["uniforms"].astype(np.float64), batch["draft_ids"]
    tb, tc, wt = shard.vocab_slice(cfg.V_t, rank, world)
    db, dc, wd = shard.vocab_slice(cfg.V_d, rank, world)
    zt = batch["target_logits"][:, :, tb:tb + tc].astype(np.float64)
    zd = batch["drafter_logits"][:, :, db:db + dc].astype(np.float64)
    inside = m[db:db + dc] >= 0
    # step 1: this shard's record: (max, sum of exp around it) per row, and the drafted logits it owns
    rec = np.zeros((B, 2 * (2 * K + 1) + 2 * K))
    for b in range(B):
        for r in range(2 * K + 1):
            z = zt[b, r] if r <= K else zd[b, r - K - 1][inside]
            mx = z.max() if z.size else -np.inf
            rec[b, 2 * r] = mx
            rec[b, 2 * r + 1] = np.exp((z - mx) / tau[b]).sum() if z.size else 0.0
        for j in range(K):
            x = draft[b, j]
            t = m[x]
            if tb <= t < tb + tc:
                rec[b, 2 * (2 * K + 1) + j] = zt[b, j, t - tb]
            if t >= 0 and db <= x < db + dc:
                rec[b, 2 * (2 * K + 1) + K + j] = zd[b, j, x - db]
    recs = shard.all_gather_dist(torch.from_numpy(rec)).numpy()
    # step 2: the same decision on every rank
    mx = recs[:, :, 0:2 * (2 * K + 1):2].max(axis=0)                       # [B, rows]
    S = (recs[:, :, 1:2 * (2 * K + 1):2] * np.exp((recs[:, :, 0:2 * (2 * K + 1):2] - mx) / tau[None, :, None])).sum(axis=0)
    accepted = np.full(B, K)
    for b in range(B):
        for j in range(K):
            x = draft[b, j]; t = m[x]
            zt_j = recs[t // wt, b, 2 * (2 * K + 1) + j]
            zd_j = recs[x // wd, b, 2 * (2 * K + 1) + K + j]
            p = np.exp((zt_j - mx[b, j]) / tau[b]) / S[b, j]
            q = np.exp((zd_j - mx[b, K + 1 + j]) / tau[b]) / S[b, K + 1 + j]
            if not (u[b, j] < min(1.0, p / q)):
                accepted[b] = j
                break
    n = accepted
    rows = np.full((B, wd), -np.inf)
    for b in range(B):
        if n[b] < K:
            rows[b, :dc] = zd[b, n[b]]
    rows_all = shard.all_gather_dist(torch.from_numpy(rows)).numpy()           # [world, B, wd]
    # step 3: weights over this shard's target ids, q' from the gathered row
    inv = np.full(cfg.V_t, -1)
    inv[m[m >= 0]] = np.flatnonzero(m >= 0)
    w = np.zeros((B, tc))
    for b in range(B):
        p = np.exp((zt[b, n[b]] - mx[b, n[b]]) / tau[b]) / S[b, n[b]]
        if n[b] < K:
            x = inv[tb:tb + tc]
            zq = np.where(x >= 0, rows_all[np.maximum(x, 0) // wd, b, np.maximum(x, 0) % wd], -np.inf)
            q = np.exp((zq - mx[b, K + 1 + n[b]]) / tau[b]) / S[b, K + 1 + n[b]]
            p = np.maximum(0.0, p - q)
        w[b] = p
    masses = shard.all_gather_dist(torch.from_numpy(w.sum(axis=1))).numpy()   # [world, B]
    # step 4: the owner walks its slice
    token = np.full(B, -1, np.int64)
    for b in range(B):
        target = u[b, K] * masses[:, b].sum()
        cum = np.cumsum(masses[:, b])
        owner = int(np.searchsorted(cum, target, side="right"))
        if owner == rank:
            rem = target - (cum[owner - 1] if owner else 0.0)
            token[b] = tb + int(np.searchsorted(np.cumsum(w[b]), rem, side="right"))
    owners = torch.from_numpy((token >= 0).astype(np.int64))
    dist.all_reduce(owners)
    tok = torch.from_numpy(token.copy())
    dist.all_reduce(tok, op=dist.ReduceOp.MAX)
    if rank == 0:
        np.save(out_path, np.stack([accepted, tok.numpy(), owners.numpy()], axis=1))
    dist.barrier()
    dist.destroy_process_group()


def test_two_vocabulary_shards_agree_with_the_unsharded_oracle(tmp_path):
    out = str(tmp_path / "sharded.npy")
    mp.spawn(_np_shard_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    got = np.load(out)
    cfg = wl.tiny_config(B=6, K=3, V_t=211, V_d=157, dtype=wl.F32, f_mapped=0.6, sigma_d=0.4,
                         temperatures=(0.7, 1.0), seed=93)
    batch = wl.make_batch(cfg)
    o = oracle.verify(batch["target_logits"], batch["drafter_logits"], batch["id_map"], batch["draft_ids"],
                      batch["temperature"], batch["uniforms"])
    assert (got[:, 2] == 1).all()                          # exactly one rank reported each token
    np.testing.assert_array_equal(got[:, 0], o["accepted"])
    np.testing.assert_array_equal(got[:, 1], o["next_token"])
    assert 0 < o["accepted"].min() + 1 and o["accepted"].max() >= 1


def test_the_benchmark_split_covers_the_headline_batch_once():
    """bench.py --gpus N gives rank r the sequences shard.row_block(B, r, N) of the headline workload and
    builds only those (make_batch(rows=...)): the blocks partition the batch, and a block generated on
    its own holds the same bits as the same rows of the whole batch."""
    cfg = wl.tiny_config(B=11, K=3, V_t=900, V_d=700, dtype=wl.BF16, f_mapped=0.6, temperatures=(0.7, 1.0),
                         greedy_rows="interleaved", seed=95)
    full = wl.make_batch(cfg)
    for world in (2, 4, 8):
        seen = []
        for rank in range(world):
            b0, b1 = shard.row_block(cfg.B, rank, world)
            seen += list(range(b0, b1))
            if b1 > b0:
                part = wl.make_batch(cfg, rows=list(range(b0, b1)))
                for k in ("target_logits", "drafter_logits", "draft_ids", "temperature", "uniforms"):
                    np.testing.assert_array_equal(part[k], full[k][b0:b1], err_msg=k)
                np.testing.assert_array_equal(part["id_map"], full["id_map"])
        assert seen == list(range(cfg.B))
    big = wl.config_by_name("cfg3")
    for world in (1, 2, 4, 8):
        sizes = [e - b for b, e in shard.row_blocks(big.B, world)]
        assert sum(sizes) * big.K == big.positions and max(sizes) - min(sizes) <= 1
