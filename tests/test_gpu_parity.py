"""Parity of the CUDA library with the fp64 oracle, element by element, through the C ABI."""
import ctypes
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2502_05202_b200 import tli, workload as wl
from parity_util import check, compare, run_gpu, run_oracle, to_device

pytestmark = pytest.mark.gpu


def bf16(x):
    return wl.f32_to_bf16_bits(np.asarray(x, np.float32))


# --------------------------------------------------------------------------
# small and medium sizes: several tiles, ragged tails, both storage types
# --------------------------------------------------------------------------

@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
@pytest.mark.parametrize("V_t,V_d,K,B", [(3, 4, 1, 5), (11, 13, 3, 9), (64, 50, 2, 7), (257, 300, 5, 6),
                                         (1000, 999, 4, 4)])
def test_tiny_vocabularies(dtype, V_t, V_d, K, B):
    cfg = wl.tiny_config(B=B, K=K, V_t=V_t, V_d=V_d, dtype=dtype, f_mapped=0.6,
                         temperatures=(0.5, 1.0, 1.3), seed=11 + V_t)
    rep = check(wl.make_batch(cfg))
    assert rep.exact + rep.excused_sampler + rep.excused_threshold >= B


@pytest.mark.parametrize("dtype,V_t,V_d", [
    (wl.F32, 3 * 4096 + 37, 2 * 4096 + 5),      # 16 KB chunks of fp32: three full + ragged
    (wl.BF16, 2 * 8192 + 13, 8192 + 8191),      # odd lengths: bf16 rows start off 16-byte alignment
    (wl.BF16, 20001, 9999),
    (wl.F32, 4096, 8192),                       # exact multiples
])
def test_several_tiles_and_ragged_tails(dtype, V_t, V_d):
    cfg = wl.tiny_config(B=6, K=3, V_t=V_t, V_d=V_d, dtype=dtype, f_mapped=0.5,
                         temperatures=(0.7, 1.0), greedy_rows="interleaved", seed=5)
    rep = check(wl.make_batch(cfg))
    print(rep)


@pytest.mark.parametrize("mode", ["intersection", "raw"])
def test_draft_modes_and_low_overlap(mode):
    cfg = wl.tiny_config(B=16, K=6, V_t=5000, V_d=7001, dtype=wl.BF16, f_mapped=0.12, sigma_d=0.5,
                         temperatures=(0.8, 1.0), seed=21)
    batch = wl.make_batch(cfg, draft_mode=mode)
    rep = check(batch)
    if mode == "raw":
        assert (run_oracle(batch)["flags"] & oracle.FLAG_DRAFT_UNMAPPED).any()


def test_strided_and_offset_inputs():
    """Rows padded to odd strides and a base pointer one element into the buffer."""
    cfg = wl.tiny_config(B=5, K=3, V_t=4100, V_d=3001, dtype=wl.BF16, f_mapped=0.7, seed=31)
    batch = wl.make_batch(cfg)
    B, K = cfg.B, cfg.K
    dev = to_device(batch)
    big_t = torch.zeros(B, K + 2, cfg.V_t + 3, dtype=torch.bfloat16, device="cuda")
    big_d = torch.zeros(B, K + 1, cfg.V_d + 5, dtype=torch.bfloat16, device="cuda")
    big_t[:, :K + 1, 1:cfg.V_t + 1] = dev["target_logits"]
    big_d[:, :K, 1:cfg.V_d + 1] = dev["drafter_logits"]
    dev2 = dict(dev, target_logits=big_t[:, :K + 1, 1:cfg.V_t + 1], drafter_logits=big_d[:, :K, 1:cfg.V_d + 1])
    assert dev2["target_logits"].data_ptr() % 16 != 0
    gpu = run_gpu(batch, dev=dev2)
    rep = compare(batch, gpu)
    assert rep.ok(), str(rep)
    ref = run_gpu(batch)
    for k in ("accepted", "next_token", "row_status"):
        np.testing.assert_array_equal(gpu[k], ref[k])


# --------------------------------------------------------------------------
# the five workloads at full size, every row, in the benchmark's launch configuration
# --------------------------------------------------------------------------

@pytest.mark.parametrize("name", ["cfg0", "cfg1", "cfg2", "cfg3", "cfg4"])
def test_full_size_workloads(name):
    cfg = wl.config_by_name(name)
    batch = wl.make_batch(cfg)
    rep = check(batch)
    print(name, rep)
    assert rep.rows == cfg.B
    # near-ties are rare: almost every row must match exactly
    assert rep.exact >= cfg.B - max(2, cfg.B // 16)


@pytest.mark.parametrize("name", ["cfg0", "cfg1"])
def test_small_batches_with_the_portable_and_the_wide_cluster(name):
    """Clusters of 8 CTAs (portable) and, where the device places them, of 16: both against the oracle."""
    cfg = wl.config_by_name(name)
    batch = wl.make_batch(cfg)
    dt = tli.TLI_F32 if cfg.elt == 4 else tli.TLI_BF16
    widths = []
    for ctas in (8, 16):
        v = tli.Verifier(cfg.V_t, cfg.V_d, batch["id_map"])
        try:
            tli.tli_set_max_cluster(v.ctx, ctas)
        except tli.TLIError as e:
            assert ctas == 16 and e.code == tli.TLI_ERR_UNSUPPORTED
            v.close()
            continue
        plan = tli.tli_verify_plan(v.ctx, cfg.B, cfg.K, dt)
        assert plan["cluster"] == ctas, plan
        rep = check(batch, verifier=v)
        assert rep.rows == cfg.B
        widths.append(ctas)
        v.close()
    assert 8 in widths
    with pytest.raises(tli.TLIError):
        v = tli.Verifier(cfg.V_t, cfg.V_d, batch["id_map"])
        try:
            tli.tli_set_max_cluster(v.ctx, 12)
        finally:
            v.close()


def test_interleaved_greedy_rows_and_raw_drafts_on_cfg4_shape():
    cfg = dataclasses.replace(wl.config_by_name("cfg4"), B=8, K=6, greedy_rows="interleaved", seed=77)
    rep = check(wl.make_batch(cfg, draft_mode="raw"))
    print(rep)


# --------------------------------------------------------------------------
# degenerate cases of the method
# --------------------------------------------------------------------------

def test_empty_intersection_rejects_everything():
    cfg = wl.tiny_config(B=6, K=3, V_t=700, V_d=500, f_mapped=0.0, seed=3)
    batch = wl.make_batch(cfg)
    assert (batch["id_map"] < 0).all()
    gpu = run_gpu(batch)
    assert (gpu["accepted"] == 0).all()
    assert (gpu["row_status"] == (tli.TLI_ROW_DRAFT_UNMAPPED | tli.TLI_ROW_FALLBACK)).all()
    assert compare(batch, gpu).ok()


def test_identity_map_with_equal_logits_accepts_everything():
    rng = np.random.default_rng(0)
    V, K, B = 9000, 4, 5
    zt = rng.normal(0, 3, (B, K + 1, V)).astype(np.float32)
    batch = {"target_logits": zt, "drafter_logits": zt[:, :K].copy(), "id_map": np.arange(V, dtype=np.int32),
             "draft_ids": rng.integers(0, V, (B, K)).astype(np.int32), "temperature": np.ones(B, np.float32),
             "uniforms": np.full((B, K + 1), 1 - 2.0 ** -24, np.float32)}
    gpu = run_gpu(batch)
    assert (gpu["accepted"] == K).all()
    assert compare(batch, gpu).ok()


def test_zero_residual_falls_back_to_target_distribution():
    """p == q' bit for bit and a draft id out of range: rejected, residual mass exactly 0, sample from p.

    The oracle forms q' as q / M with M = 1 +- 1e-16, so its own residual is rounding noise instead of 0;
    the expected token is therefore the oracle's sample from p_0 (same logits, empty intersection)."""
    rng = np.random.default_rng(1)
    V, K, B = 5000, 2, 4
    zt = rng.normal(0, 2, (B, K + 1, V)).astype(np.float32)
    d = rng.integers(0, V, (B, K)).astype(np.int32)
    d[:, 0] = V + 3
    d[1, 0] = -1
    batch = {"target_logits": zt, "drafter_logits": zt[:, :K].copy(), "id_map": np.arange(V, dtype=np.int32),
             "draft_ids": d, "temperature": np.full(B, 0.9, np.float32),
             "uniforms": rng.random((B, K + 1)).astype(np.float32)}
    gpu = run_gpu(batch)
    assert (gpu["accepted"] == 0).all()
    assert (gpu["row_status"] == (tli.TLI_ROW_DRAFT_RANGE | tli.TLI_ROW_FALLBACK)).all()
    from_p = run_oracle(dict(batch, id_map=np.full(V, -1, np.int32), draft_ids=np.zeros((B, K), np.int32)))
    assert (from_p["accepted"] == 0).all()
    np.testing.assert_array_equal(gpu["next_token"], from_p["next_token"])


def test_minus_infinity_logits_are_zero_probability_tokens():
    cfg = wl.tiny_config(B=6, K=3, V_t=6000, V_d=5000, dtype=wl.F32, f_mapped=0.5, seed=41)
    batch = wl.make_batch(cfg)
    rng = np.random.default_rng(2)
    kill_t = rng.random(batch["target_logits"].shape) < 0.3
    kill_d = rng.random(batch["drafter_logits"].shape) < 0.3
    # keep the drafted tokens alive on both sides
    for b in range(cfg.B):
        for j in range(cfg.K):
            x = batch["draft_ids"][b, j]
            kill_d[b, j, x] = False
            kill_t[b, j, batch["id_map"][x]] = False
    gpu_in = dict(batch, target_logits=np.where(kill_t, -np.inf, batch["target_logits"]).astype(np.float32),
                  drafter_logits=np.where(kill_d, -np.inf, batch["drafter_logits"]).astype(np.float32))
    ref_in = dict(batch, target_logits=np.where(kill_t, -1e30, batch["target_logits"]).astype(np.float32),
                  drafter_logits=np.where(kill_d, -1e30, batch["drafter_logits"]).astype(np.float32))
    gpu = run_gpu(gpu_in)
    assert (gpu["row_status"] == 0).all()
    rep = compare(ref_in, gpu)
    assert rep.ok(), str(rep)
    dead = kill_t[np.arange(cfg.B), gpu["accepted"], gpu["next_token"]]
    assert not dead.any()


def test_nan_and_plus_infinity_flag_the_row():
    cfg = wl.tiny_config(B=6, K=3, V_t=6000, V_d=5000, dtype=wl.BF16, f_mapped=0.5, seed=42)
    batch = wl.make_batch(cfg)
    zt = wl.bf16_bits_to_f32(batch["target_logits"]).copy()
    zd = wl.bf16_bits_to_f32(batch["drafter_logits"]).copy()
    zt[1, 2, 4097] = np.nan
    zt[3, 0, 17] = np.inf
    mapped = np.flatnonzero(batch["id_map"] >= 0)
    zd[4, 1, mapped[5]] = np.nan
    bad = dict(batch, target_logits=bf16(zt), drafter_logits=bf16(zd))
    gpu = run_gpu(bad)
    flagged = (gpu["row_status"] & tli.TLI_ROW_NONFINITE) != 0
    assert flagged.tolist() == [False, True, False, True, True, False]
    assert (gpu["accepted"][flagged] == 0).all() and (gpu["next_token"][flagged] == 0).all()
    clean = run_gpu(batch)
    for k in ("accepted", "next_token"):
        np.testing.assert_array_equal(gpu[k][~flagged], clean[k][~flagged])


def test_non_finite_logits_where_the_oracle_and_the_header_say_they_count():
    """The rule of tli.h, case by case, against the oracle: a NaN in the bonus row counts only when every
    draft was accepted; at a drafter id outside the intersection it is not examined (the oracle, which
    forms the softmax over all of D, is given a finite value there); in a temperature-0 row a NaN past
    the first element is never the arg-max on either side."""
    cfg = wl.tiny_config(B=6, K=3, V_t=5000, V_d=4000, dtype=wl.F32, f_mapped=0.5, sigma_d=0.3,
                         temperatures=(1.0,), seed=47)
    batch = wl.make_batch(cfg)
    batch["temperature"] = np.array([1.0, 1.0, 1.0, 1.0, 0.0, 0.0], np.float32)
    clean = run_oracle(batch)
    K = cfg.K
    rejected = [b for b in range(4) if clean["accepted"][b] < K]
    accepted_all = [b for b in range(4) if clean["accepted"][b] == K]
    zt, zd = batch["target_logits"].copy(), batch["drafter_logits"].copy()
    unmapped = np.flatnonzero(batch["id_map"] < 0)
    for b in range(4):
        zt[b, K, 123] = np.nan                       # bonus row of every sampled sequence
    zd_orc = zd.copy()
    zd[0, 0, unmapped[3]] = np.nan                   # outside the intersection: not examined by the GPU
    zd[1, 1, unmapped[7]] = np.inf
    zt[4, 1, 2500] = np.nan                          # temperature 0: never the arg-max
    zt[5, 0, 77] = np.nan
    gpu = run_gpu(dict(batch, target_logits=zt, drafter_logits=zd))
    orc = run_oracle(dict(batch, target_logits=zt, drafter_logits=zd_orc))
    assert rejected, "the case needs a sequence with a rejected draft"
    for b in rejected:
        assert orc["flags"][b] == 0 and gpu["row_status"][b] == 0
    for b in accepted_all:
        assert orc["flags"][b] == oracle.FLAG_NONFINITE and gpu["row_status"][b] == tli.TLI_ROW_NONFINITE
    rep = compare(dict(batch, target_logits=zt, drafter_logits=zd_orc), gpu, orc=orc)
    assert rep.ok(), str(rep)
    tiled = run_gpu(dict(batch, target_logits=zt, drafter_logits=zd), tiled=True)
    rep = compare(dict(batch, target_logits=zt, drafter_logits=zd_orc), tiled, orc=orc)
    assert rep.ok(), "tile kernels: " + str(rep)


def test_exactly_zero_residual_falls_back_to_the_target_distribution():
    """p = q' = 2^-k exactly (identity map, equal logits, power-of-two vocabulary): a draft outside the
    vocabulary leaves a residual of exactly zero, the fall-back flag, and a token drawn from p --
    the same on the oracle (pinned on the CPU side) and on both forms of the GPU call."""
    for dtype in (wl.F32, wl.BF16):
        V, K, B = 4096, 2, 6
        zt = np.zeros((B, K + 1, V), np.float32)
        zd = np.zeros((B, K, V), np.float32)
        if dtype == wl.BF16:
            zt, zd = bf16(zt), bf16(zd)
        batch = {"target_logits": zt, "drafter_logits": zd, "id_map": np.arange(V, dtype=np.int32),
                 "draft_ids": np.array([[V, 0], [-1, 3], [2, V + 5], [1, 2], [7, -9], [0, 0]], np.int32),
                 "temperature": np.ones(B, np.float32),
                 "uniforms": np.array([[0.5, 0.5, 0.30], [0.1, 0.2, 0.99], [0.9, 0.1, 0.0625], [0.3, 0.3, 0.5],
                                       [0.999, 0.0, 0.124], [0.2, 0.4, 0.9999]], np.float32)}
        rep = check(batch)
        assert rep.exact == B and rep.excused_sampler == 0, str(rep)
        gpu = run_gpu(batch)
        fb = tli.TLI_ROW_DRAFT_RANGE | tli.TLI_ROW_FALLBACK
        assert gpu["row_status"].tolist() == [fb, fb, fb, 0, fb, 0]
        assert gpu["next_token"].tolist() == [int(np.floor(float(v) * V)) for v in batch["uniforms"][:, K]]


def test_reset_brings_the_counters_back():
    """tli_reset() zeroes the context's counters in stream order; calls before and after agree."""
    cfg = wl.tiny_config(B=4, K=3, V_t=9000, V_d=7000, dtype=wl.BF16, f_mapped=0.5, seed=48)
    batch = wl.make_batch(cfg)
    v = tli.Verifier(cfg.V_t, cfg.V_d, batch["id_map"])
    before = run_gpu(batch, v)
    tli.tli_reset(v.ctx)
    after = run_gpu(batch, v)
    for k in before:
        np.testing.assert_array_equal(before[k], after[k])
    assert tli.load().tli_reset(None, None) == tli.TLI_ERR_ARG
    v.close()


def test_bad_temperature_flags_the_row():
    cfg = wl.tiny_config(B=5, K=2, V_t=500, V_d=400, seed=43)
    batch = wl.make_batch(cfg)
    batch["temperature"] = np.array([1.0, -0.5, np.nan, np.inf, 0.0], np.float32)
    gpu = run_gpu(batch)
    assert gpu["row_status"].tolist()[1:4] == [tli.TLI_ROW_BAD_TEMPERATURE] * 3
    assert (gpu["accepted"][1:4] == 0).all()
    orc = run_oracle(dict(batch, temperature=np.array([1.0, 1.0, 1.0, 1.0, 0.0], np.float32)))
    for b in (0, 4):
        assert gpu["accepted"][b] == orc["accepted"][b] and gpu["next_token"][b] == orc["next_token"][b]


def test_greedy_ties_are_bit_exact():
    """bf16 logits tie often; the lowest index must win in every reduction step."""
    rng = np.random.default_rng(5)
    V_t, V_d, K, B = 3 * 8192 + 100, 30000, 4, 12
    zt = np.round(rng.normal(0, 1, (B, K + 1, V_t))).astype(np.float32)     # few distinct values -> many ties
    zd = rng.normal(0, 1, (B, K, V_d)).astype(np.float32)
    cfgm = wl.tiny_config(V_t=V_t, V_d=V_d, f_mapped=0.8, seed=9)
    id_map = wl.make_id_map(cfgm)
    first_max = zt.argmax(axis=2)
    inv = np.full(V_t, -1)
    inv[id_map[id_map >= 0]] = np.flatnonzero(id_map >= 0)
    d = np.where(inv[first_max[:, :K]] >= 0, inv[first_max[:, :K]], 0).astype(np.int32)
    d[::3, 1] = (d[::3, 1] + 1) % V_d
    batch = {"target_logits": bf16(zt), "drafter_logits": bf16(zd), "id_map": id_map, "draft_ids": d,
             "temperature": np.zeros(B, np.float32), "uniforms": np.zeros((B, K + 1), np.float32)}
    gpu = run_gpu(batch)
    orc = run_oracle(batch)
    np.testing.assert_array_equal(gpu["accepted"], orc["accepted"])
    np.testing.assert_array_equal(gpu["next_token"], orc["next_token"])
    assert gpu["accepted"].max() == K


@pytest.mark.parametrize("B,K", [(1, 1), (1, 64), (300, 1)])
def test_extreme_batch_and_draft_counts(B, K):
    cfg = wl.tiny_config(B=B, K=K, V_t=2000, V_d=1500, dtype=wl.BF16, f_mapped=0.6, sigma_d=0.3, seed=50 + K)
    check(wl.make_batch(cfg))


def test_most_sequences_in_one_call():
    """B at the library's limit (65535 sequences of a small vocabulary)."""
    rng = np.random.default_rng(61)
    B, K, V_t, V_d = tli.TLI_MAX_B, 2, 96, 80
    zt = rng.normal(0, 2, (B, K + 1, V_t)).astype(np.float32)
    id_map = np.full(V_d, -1, np.int32)
    inside = rng.choice(V_d, 56, replace=False)
    id_map[inside] = rng.permutation(V_t)[:56]
    zd = rng.normal(-2, 1, (B, K, V_d)).astype(np.float32)
    zd[:, :, inside] = zt[:, :K, id_map[inside]] + rng.normal(0, 0.3, (B, K, 56)).astype(np.float32)
    batch = {"target_logits": zt, "drafter_logits": zd, "id_map": id_map,
             "draft_ids": inside[rng.integers(0, 56, (B, K))].astype(np.int32),
             "temperature": rng.choice(np.array([0.0, 0.7, 1.0], np.float32), B),
             "uniforms": rng.integers(0, 1 << 24, (B, K + 1)).astype(np.float32) / np.float32(1 << 24)}
    rep = check(batch, threads=16)
    assert rep.rows == B and rep.exact >= B - 50


def test_large_vocabulary_near_the_limit():
    cfg = wl.tiny_config(B=2, K=1, V_t=tli.TLI_MAX_V, V_d=tli.TLI_MAX_V - 7, dtype=wl.F32, f_mapped=0.5, seed=60)
    check(wl.make_batch(cfg))


def test_repeated_calls_reuse_the_context():
    cfg = wl.tiny_config(B=7, K=3, V_t=9000, V_d=7000, dtype=wl.BF16, f_mapped=0.6, seed=61)
    batch = wl.make_batch(cfg)
    v = tli.Verifier(cfg.V_t, cfg.V_d, batch["id_map"])
    first = run_gpu(batch, v)
    for _ in range(3):
        again = run_gpu(batch, v)
        for k in first:
            np.testing.assert_array_equal(first[k], again[k])
    small = wl.make_batch(dataclasses.replace(cfg, B=2, K=2))      # same seed: same id map
    assert compare(small, run_gpu(small, v)).ok()
    v.close()


# --------------------------------------------------------------------------
# host-detectable argument errors
# --------------------------------------------------------------------------

def test_argument_errors_are_reported_not_launched():
    cfg = wl.tiny_config(B=2, K=2, V_t=300, V_d=200, seed=70)
    batch = wl.make_batch(cfg)
    v = tli.Verifier(cfg.V_t, cfg.V_d, batch["id_map"])
    dev = to_device(batch)
    acc = torch.zeros(2, dtype=torch.int32, device="cuda")
    nxt = torch.zeros(2, dtype=torch.int32, device="cuda")
    ws = v.workspace(2, 2, tli.TLI_F32)
    good = lambda: tli.make_args(dev["target_logits"], dev["drafter_logits"], dev["draft_ids"], dev["temperature"],
                                 dev["uniforms"], acc, nxt, ws)
    lib = tli.load()
    call = lambda a: lib.tli_verify(v.ctx, ctypes.byref(a), None)
    a = good(); a.workspace_bytes = 16
    assert call(a) == tli.TLI_ERR_WORKSPACE
    a = good(); a.workspace = None
    assert call(a) == tli.TLI_ERR_WORKSPACE
    a = good(); a.K = 0
    assert call(a) == tli.TLI_ERR_ARG
    a = good(); a.K = tli.TLI_MAX_K + 1
    assert call(a) == tli.TLI_ERR_UNSUPPORTED
    a = good(); a.dtype = 7
    assert call(a) == tli.TLI_ERR_ARG
    a = good(); a.uniforms = None
    assert call(a) == tli.TLI_ERR_ARG
    assert lib.tli_verify(None, ctypes.byref(good()), None) == tli.TLI_ERR_ARG
    assert tli.tli_workspace_bytes(v.ctx, 0, 1, 0) == 0
    assert call(good()) == tli.TLI_OK
    torch.cuda.synchronize()
    v.close()


def test_many_tiles_use_the_separate_selection_kernel():
    """B x tiles >= 4096: the CDF inversions run as their own kernel; same results required."""
    cfg = wl.tiny_config(B=300, K=1, V_t=60001, V_d=3000, dtype=wl.F32, f_mapped=0.5, sigma_d=0.7,
                         temperatures=(0.8, 1.0), seed=81)
    rep = check(wl.make_batch(cfg))
    assert rep.rows == 300


def test_profile_hook_reports_three_positive_durations_and_the_same_results():
    cfg = wl.tiny_config(B=6, K=3, V_t=20000, V_d=15000, dtype=wl.BF16, f_mapped=0.5, seed=82)
    batch = wl.make_batch(cfg)
    v = tli.Verifier(cfg.V_t, cfg.V_d, batch["id_map"])
    dev = to_device(batch)
    ref = run_gpu(batch, v, dev)
    acc = torch.full((6,), -1, dtype=torch.int32, device="cuda")
    nxt = torch.full((6,), -1, dtype=torch.int32, device="cuda")
    args = tli.make_args(dev["target_logits"], dev["drafter_logits"], dev["draft_ids"], dev["temperature"],
                         dev["uniforms"], acc, nxt, v.workspace(6, 3, tli.TLI_BF16))
    ms = tli.tli_verify_profile(v.ctx, args)
    assert len(ms) == 3 and all(m > 0 for m in ms)
    np.testing.assert_array_equal(acc.cpu().numpy(), ref["accepted"])
    np.testing.assert_array_equal(nxt.cpu().numpy(), ref["next_token"])
    v.close()


def test_calls_recorded_in_a_cuda_graph_replay_to_the_same_results():
    """tli_verify() only launches kernels: captured into a graph (two calls, two dtypes of batch) and replayed."""
    cfg = wl.tiny_config(B=9, K=4, V_t=70001, V_d=33000, dtype=wl.F32, f_mapped=0.6, temperatures=(0.0, 0.7, 1.0), seed=84)
    batch = wl.make_batch(cfg)
    v = tli.Verifier(cfg.V_t, cfg.V_d, batch["id_map"])
    dev = to_device(batch)
    ref = run_gpu(batch, v, dev)
    outs = [{k: torch.full((9,), -7, dtype=torch.int32, device="cuda") for k in ("acc", "nxt", "st")} for _ in range(2)]
    ws = v.workspace(9, 4, tli.TLI_F32)
    args = [tli.make_args(dev["target_logits"], dev["drafter_logits"], dev["draft_ids"], dev["temperature"],
                          dev["uniforms"], o["acc"], o["nxt"], ws, o["st"]) for o in outs]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        for a in args:
            tli.tli_verify(v.ctx, a, torch.cuda.current_stream().cuda_stream)
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(3):
        for o in outs:
            for t in o.values():
                t.fill_(-7)
        g.replay()
        torch.cuda.synchronize()
        for o in outs:
            np.testing.assert_array_equal(o["acc"].cpu().numpy(), ref["accepted"])
            np.testing.assert_array_equal(o["nxt"].cpu().numpy(), ref["next_token"])
            np.testing.assert_array_equal(o["st"].cpu().numpy(), ref["row_status"])
    del g
    v.close()


def test_host_buffer_entry_point_gives_the_same_results():
    """tli_verify_host(): pinned host tensors in and out through a caller's device buffer."""
    cfg = wl.tiny_config(B=7, K=3, V_t=30011, V_d=20011, dtype=wl.BF16, f_mapped=0.5, temperatures=(0.0, 0.9), seed=86)
    batch = wl.make_batch(cfg)
    v = tli.Verifier(cfg.V_t, cfg.V_d, batch["id_map"])
    ref = run_gpu(batch, v)
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    zt, zd = pin(batch["target_logits"]).view(torch.bfloat16), pin(batch["drafter_logits"]).view(torch.bfloat16)
    acc, nxt, st = (torch.full((7,), -5, dtype=torch.int32).pin_memory() for _ in range(3))
    need = tli.tli_verify_host_buffer_bytes(v.ctx, 7, 3, tli.TLI_BF16)
    assert need > zt.numel() * 2 + zd.numel() * 2
    buf = torch.empty(need, dtype=torch.uint8, device="cuda")
    args = tli.make_host_args(zt, zd, pin(batch["draft_ids"]), pin(batch["temperature"]), pin(batch["uniforms"]),
                              acc, nxt, buf, st)
    tli.tli_verify_host(v.ctx, args)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(acc.numpy(), ref["accepted"])
    np.testing.assert_array_equal(nxt.numpy(), ref["next_token"])
    np.testing.assert_array_equal(st.numpy(), ref["row_status"])
    args.device_buffer_bytes = need - 1
    with pytest.raises(tli.TLIError) as e:
        tli.tli_verify_host(v.ctx, args)
    assert e.value.code == tli.TLI_ERR_WORKSPACE
    assert tli.tli_verify_host_buffer_bytes(v.ctx, 0, 3, tli.TLI_BF16) == 0
    v.close()


@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
def test_per_sequence_draft_counts(dtype):
    """draft_lengths: only the first m_b drafts of a sequence count, the bonus position is row m_b, later
    rows are never read (they hold NaN here)."""
    cfg = wl.tiny_config(B=14, K=6, V_t=40013, V_d=33001, dtype=dtype, f_mapped=0.6, sigma_d=0.4,
                         temperatures=(0.0, 0.7, 1.0), seed=85)
    batch = wl.make_batch(cfg)
    lengths = np.array([0, 1, 2, 3, 4, 5, 6, 6, 3, 0, 2, 5, 1, 4], np.int32)
    nan = np.float32(np.nan) if dtype == wl.F32 else np.uint16(0x7fc0)
    for b, m in enumerate(lengths):
        batch["target_logits"][b, m + 1:] = nan
        batch["drafter_logits"][b, m:] = nan
        batch["draft_ids"][b, m:] = -12345
    batch["draft_lengths"] = lengths
    rep = check(batch)
    gpu = run_gpu(batch)
    assert (gpu["accepted"] <= lengths).all() and (gpu["row_status"] == 0).all()
    assert gpu["accepted"].max() >= 2 and ((gpu["accepted"] == lengths) & (lengths > 0)).sum() >= 2   # bonus rows below K were sampled
    for b, m in enumerate(lengths):
        assert (gpu["p_draft"][b, m:] == 0).all() and (gpu["q_draft"][b, m:] == 0).all()


def test_one_context_through_changing_shapes():
    """Calls of different batch sizes, draft counts and temperature mixes on one context, in turn and again:
    the context's buffer of partial results is back in its empty state after every call, whatever rows the
    call before used (temperature 0 sequences have no drafter rows, short sequences fewer rows)."""
    V_t, V_d = 40013, 33001
    base = wl.tiny_config(B=9, K=5, V_t=V_t, V_d=V_d, dtype=wl.BF16, f_mapped=0.6, sigma_d=0.4,
                          temperatures=(0.0, 0.7, 1.0), seed=91)
    first = wl.make_batch(base)
    v = tli.Verifier(V_t, V_d, first["id_map"])
    shapes = [dict(B=9, K=5), dict(B=3, K=2), dict(B=14, K=7), dict(B=1, K=1), dict(B=9, K=5)]      # the id map comes from the seed alone
    for rnd in range(2):
        for i, sh in enumerate(shapes):
            cfg = dataclasses.replace(base, **sh)
            batch = wl.make_batch(cfg)
            np.testing.assert_array_equal(batch["id_map"], first["id_map"])
            if i % 2 == 1:
                batch["draft_lengths"] = (np.arange(cfg.B, dtype=np.int32) * 3) % (cfg.K + 1)
            rep = check(batch, verifier=v)
            assert rep.rows == cfg.B, (rnd, sh, rep)
    plan = tli.tli_verify_plan(v.ctx, 9, 5, tli.TLI_BF16)
    assert plan["launches"] == 2 and plan["cluster"] >= 1         # the form that uses that buffer
    v.close()


def test_a_wait_that_nothing_completes_gives_up_and_leaves_the_context_usable():
    """The kernels' waits are bounded: run the same wait code on a barrier nobody will complete."""
    cfg = wl.tiny_config(B=3, K=2, V_t=9000, V_d=7000, dtype=wl.F32, f_mapped=0.5, seed=83)
    batch = wl.make_batch(cfg)
    v = tli.Verifier(cfg.V_t, cfg.V_d, batch["id_map"])
    before = run_gpu(batch, v)
    assert tli.tli_selftest_bounded_wait(v.ctx, polls=2000)
    after = run_gpu(batch, v)
    for k in before:
        np.testing.assert_array_equal(before[k], after[k])
    assert (after["row_status"] & tli.TLI_ROW_TIMEOUT == 0).all()     # the self-test keeps its own error word
    with pytest.raises(tli.TLIError):
        tli.tli_selftest_bounded_wait(v.ctx, polls=0)
    v.close()


def test_the_plan_follows_the_size_rule():
    """tli_verify_plan(): two launches (one cluster per sequence) where the drafter row fits a CTA's shared
    memory and the batch is moderate, the tile kernels otherwise; tli_set_tiled forces the latter."""
    expect = {"cfg0": (2, 8), "cfg1": (2, 8), "cfg2": (2, 4), "cfg3": (4, 0), "cfg4": (2, 4)}
    for name, (launches, cluster) in expect.items():
        cfg = wl.config_by_name(name)
        v = tli.Verifier(cfg.V_t, cfg.V_d, wl.make_id_map(cfg))
        dt = tli.TLI_F32 if cfg.elt == 4 else tli.TLI_BF16
        plan = tli.tli_verify_plan(v.ctx, cfg.B, cfg.K, dt)
        wide = 16 if name in ("cfg0", "cfg1") else cluster       # where the driver places clusters of 16, small batches get them
        assert plan["launches"] == launches and plan["cluster"] in (cluster, wide), (name, plan)
        assert plan["stats_ctas"] >= 1 and plan["segment_bytes"] % plan["stage_bytes"] in (0, plan["segment_bytes"])
        big = tli.tli_verify_plan(v.ctx, 4096, cfg.K, dt)                # far more CTAs than eight per SM
        assert big["cluster"] == 0 and big["launches"] >= 3
        tli.tli_set_tiled(v.ctx, True)
        assert tli.tli_verify_plan(v.ctx, cfg.B, cfg.K, dt)["cluster"] == 0
        v.close()
    with pytest.raises(tli.TLIError):
        tli.tli_verify_plan(0, 1, 1, 0)
