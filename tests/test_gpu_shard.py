"""Vocabulary-sharded verification (tli_shard_*): G slices of the same tensors verified on one GPU,
the exchanges replaced by stacks of the shards' buffers, against the oracle on the unsharded inputs
with the rule of the parity tests.  Algorithm 4's sum over the intersection and Algorithm 5's
residual normaliser are the two quantities that cross shards."""
import numpy as np
import pytest
import torch

from paper_2502_05202_b200 import shard, tli, workload as wl
from parity_util import compare, run_oracle, to_device

pytestmark = pytest.mark.gpu


def bf16(x):
    return wl.f32_to_bf16_bits(np.asarray(x, np.float32))


def run_sharded(batch, G):
    """The batch verified as G vocabulary shards on one device; returns host arrays like run_gpu()."""
    dev = to_device(batch)
    zt, zd = dev["target_logits"], dev["drafter_logits"]
    V_t, V_d = zt.shape[2], zd.shape[2]
    shards = [shard.ShardedVerifier(V_t, V_d, batch["id_map"], G, g) for g in range(G)]
    zts, zds = [], []
    for g, s in enumerate(shards):
        i = s.info
        assert (i["t_begin"], i["t_count"], i["t_width"]) == shard.vocab_slice(V_t, g, G)
        assert (i["d_begin"], i["d_count"], i["d_width"]) == shard.vocab_slice(V_d, g, G)
        # views into the full tensors: rows of a slice start wherever the slice starts (no alignment)
        zts.append(zt[:, :, i["t_begin"]: i["t_begin"] + i["t_count"]] if i["t_count"] else zt[:, :, :1])
        zds.append(zd[:, :, i["d_begin"]: i["d_begin"] + i["d_count"]] if i["d_count"] else zd[:, :, :1])
    out = shard.verify_on_one_device(shards, zts, zds, dev["draft_ids"], dev["temperature"], dev["uniforms"])
    torch.cuda.synchronize()
    res = {k: out[k].cpu().numpy() for k in ("accepted", "next_token", "row_status", "p_draft", "q_draft")}
    # every shard took the same decisions; exactly one of them reports each sampled token
    for st in out["per_shard"][1:]:
        for k in ("accepted", "row_status", "p_draft", "q_draft"):
            np.testing.assert_array_equal(st[k].cpu().numpy(), res[k], err_msg=k)
    tokens = np.stack([st["next_token"].cpu().numpy() for st in out["per_shard"]])
    sampled = (batch["temperature"] > 0) & (res["row_status"] & (tli.TLI_ROW_NONFINITE | tli.TLI_ROW_BAD_TEMPERATURE) == 0)
    assert ((tokens[:, sampled] >= 0).sum(axis=0) == 1).all()
    assert (tokens[:, ~sampled] == tokens[:1, ~sampled]).all()
    for s in shards:
        s.close()
    return res


def check_sharded(batch, G):
    rep = compare(batch, run_sharded(batch, G))
    assert rep.ok(), "G=%d: %s" % (G, rep)
    return rep


@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
@pytest.mark.parametrize("G", [2, 4])
def test_shards_of_the_same_tensors_match_the_oracle(dtype, G):
    """Random maps: most mapped pairs have their drafter id and their target id on different shards."""
    cfg = wl.tiny_config(B=10, K=4, V_t=3 * 8192 + 131, V_d=2 * 8192 + 77, dtype=dtype, f_mapped=0.6, sigma_d=0.5,
                         temperatures=(0.6, 1.0), greedy_rows="interleaved", seed=401)
    batch = wl.make_batch(cfg)
    m = batch["id_map"]
    x = np.flatnonzero(m >= 0)
    wt, wd = -(-cfg.V_t // G), -(-cfg.V_d // G)
    assert ((x // wd) != (m[x] // wt)).mean() > 0.3          # pairs that straddle two shards
    rep = check_sharded(batch, G)
    assert rep.exact >= cfg.B - 2


def test_a_workload_at_full_width():
    cfg = wl.config_by_name("cfg2")
    batch = wl.make_batch(cfg, rows=list(range(16)))
    check_sharded(batch, 4)


@pytest.mark.parametrize("G", [2, 4])
def test_tiny_vocabularies_leave_shards_empty(G):
    """V_t = 5 and V_d = 3 over four shards: trailing shards hold no ids at all."""
    rng = np.random.default_rng(402)
    B, K, V_t, V_d = 7, 3, 5, 3
    batch = {"target_logits": rng.normal(0, 1.5, (B, K + 1, V_t)).astype(np.float32),
             "drafter_logits": rng.normal(0, 1.5, (B, K, V_d)).astype(np.float32),
             "id_map": np.array([4, -1, 0], np.int32),
             "draft_ids": rng.choice([0, 2], size=(B, K)).astype(np.int32),
             "temperature": np.array([1.0, 0.7, 0.0, 1.0, 0.5, 0.0, 1.0], np.float32),
             "uniforms": (rng.integers(0, 1 << 24, (B, K + 1)) / float(1 << 24)).astype(np.float32)}
    check_sharded(batch, G)


def test_a_shard_without_any_of_the_intersection():
    """Every mapped drafter id lies on shard 0 and every mapped target id on the last shard: the other
    shards add nothing to Algorithm 4's denominator, and q'_T is zero on all but the last."""
    cfg = wl.tiny_config(B=6, K=3, V_t=4000, V_d=3000, dtype=wl.BF16, f_mapped=0.5, temperatures=(0.8, 1.0), seed=403)
    batch = wl.make_batch(cfg)
    G = 3
    wt, wd = -(-cfg.V_t // G), -(-cfg.V_d // G)
    rng = np.random.default_rng(403)
    m = np.full(cfg.V_d, -1, np.int32)
    xs = rng.choice(wd, size=400, replace=False)
    m[xs] = 2 * wt + rng.choice(cfg.V_t - 2 * wt, size=400, replace=False)
    batch["id_map"] = m
    batch["draft_ids"] = rng.choice(xs, size=batch["draft_ids"].shape).astype(np.int32)
    check_sharded(batch, G)


def test_arg_max_ties_across_a_shard_edge():
    """Temperature 0: equal maxima on both sides of a shard boundary; the lowest global id must win."""
    V_t, V_d, K, B, G = 1000, 600, 2, 4, 4
    wt = -(-V_t // G)
    zt = np.zeros((B, K + 1, V_t), np.float32)
    pairs = [(wt - 1, wt), (wt + 3, 2 * wt), (2 * wt - 1, 3 * wt + 5), (5, 3 * wt)]
    for b, (lo, hi) in enumerate(pairs):
        zt[b, :, hi] = 7.0
        zt[b, :, lo] = 7.0
    id_map = np.full(V_d, -1, np.int32)
    id_map[:500] = np.arange(500) * 2
    inv = {int(t): x for x, t in enumerate(id_map) if t >= 0}
    draft = np.zeros((B, K), np.int32)
    for b, (lo, hi) in enumerate(pairs):
        draft[b, 0] = inv.get(lo, 1)
    batch = {"target_logits": bf16(zt), "drafter_logits": bf16(np.zeros((B, K, V_d), np.float32)), "id_map": id_map,
             "draft_ids": draft, "temperature": np.zeros(B, np.float32),
             "uniforms": np.full((B, K + 1), 0.5, np.float32)}
    res = run_sharded(batch, G)
    orc = run_oracle(batch)
    np.testing.assert_array_equal(res["next_token"], orc["next_token"])
    np.testing.assert_array_equal(res["accepted"], orc["accepted"])
    for b, (lo, hi) in enumerate(pairs):
        assert res["next_token"][b] == lo


def test_zero_residual_and_bad_rows_take_the_same_path_on_every_shard():
    """The exactly-zero residual (fall-back to p, decided from the exchanged totals), a draft outside
    the vocabulary, an invalid temperature."""
    V, K, B, G = 4096, 2, 5, 4
    batch = {"target_logits": np.zeros((B, K + 1, V), np.float32), "drafter_logits": np.zeros((B, K, V), np.float32),
             "id_map": np.arange(V, dtype=np.int32),
             "draft_ids": np.array([[V, 0], [-1, 3], [2, V + 5], [1, 2], [7, 9]], np.int32),
             "temperature": np.array([1.0, 1.0, 1.0, 1.0, -1.0], np.float32),
             "uniforms": np.array([[0.5, 0.5, 0.30], [0.1, 0.2, 0.99], [0.9, 0.1, 0.0625], [0.3, 0.3, 0.5],
                                   [0.999, 0.0, 0.124]], np.float32)}
    res = run_sharded(batch, G)
    fb = tli.TLI_ROW_DRAFT_RANGE | tli.TLI_ROW_FALLBACK
    assert res["row_status"].tolist() == [fb, fb, fb, 0, tli.TLI_ROW_BAD_TEMPERATURE]
    assert res["next_token"][:4].tolist() == [int(np.floor(float(v) * V)) for v in batch["uniforms"][:4, K]]
    assert res["accepted"].tolist() == [0, 0, 1, 2, 0]


def test_argument_errors():
    cfg = wl.tiny_config(B=2, K=2, V_t=300, V_d=200, seed=404)
    batch = wl.make_batch(cfg)
    with pytest.raises(tli.TLIError):
        tli.tli_shard_create(0, cfg.V_t, cfg.V_d, batch["id_map"], 0, 0)
    with pytest.raises(tli.TLIError):
        tli.tli_shard_create(0, cfg.V_t, cfg.V_d, batch["id_map"], 2, 2)
    s = shard.ShardedVerifier(cfg.V_t, cfg.V_d, batch["id_map"], 2, 1)
    dev = to_device(batch)
    out = torch.empty(2, dtype=torch.int32, device="cuda")
    args = tli.make_args(dev["target_logits"], dev["drafter_logits"], dev["draft_ids"], dev["temperature"], dev["uniforms"],
                         out, out.clone(), torch.empty(256, dtype=torch.uint8, device="cuda"))
    with pytest.raises(tli.TLIError) as e:                   # the unsharded call refuses a shard's context
        tli.tli_verify(s.ctx, args)
    assert e.value.code == tli.TLI_ERR_ARG
    with pytest.raises(tli.TLIError) as e:                   # scratch too small
        tli.tli_shard_stats(s.ctx, args, torch.empty(64, dtype=torch.float64, device="cuda"))
    assert e.value.code == tli.TLI_ERR_WORKSPACE
    s.close()
