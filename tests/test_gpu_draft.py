"""Parity of tli_draft_sample() (drawing the draft ids from q') with the fp64 drafting oracle.

Rule, per row of drafter logits: the id must be identical, except that a difference is excused --
and counted -- when the GPU's id has positive weight in the oracle's q' and v lies within 1e-6 of
the oracle's normalised CDF interval of that id.  q_draft within 1e-5 absolute; temperature-0 rows
and the status bits get no excuses."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2502_05202_b200 import tli, workload as wl

pytestmark = pytest.mark.gpu

TOL_U = 1e-6
TOL_P = 1e-5


def dev_logits(z):
    t = torch.from_numpy(np.ascontiguousarray(z))
    if t.dtype == torch.uint16:
        t = t.view(torch.bfloat16)
    return t.cuda()


def run_gpu(zd, id_map, tau, u, V_t=None, verifier=None, zd_dev=None):
    B, R, V_d = zd.shape
    own = verifier is None
    v = verifier or tli.Verifier(int(id_map.max()) + 1 if V_t is None else V_t, V_d, id_map)
    z = dev_logits(zd) if zd_dev is None else zd_dev
    t = torch.from_numpy(np.asarray(tau, np.float32)).cuda()
    uu = torch.from_numpy(np.asarray(u, np.float32).reshape(B, R)).cuda()
    out = v.draft(z, t, uu)
    torch.cuda.synchronize()
    res = {k: x.cpu().numpy() for k, x in out.items()}
    again = v.draft(z, t, uu)                               # tickets came back to zero
    torch.cuda.synchronize()
    for k in res:
        np.testing.assert_array_equal(res[k], again[k].cpu().numpy(), err_msg="repeat call differs: " + k)
    if own:
        v.close()
    return res


def compare(zd, id_map, tau, u, gpu, threads=8):
    B, R, _ = zd.shape
    tau = np.asarray(tau, np.float32)
    u = np.asarray(u, np.float32).reshape(B, R)
    orc = oracle.draft(zd, id_map, tau, u, probe_id=gpu["draft_ids"], threads=threads)
    assert not (orc["flags"] & oracle.FLAG_SELFCHECK).any()
    oflags = orc["flags"] & ~oracle.FLAG_SELFCHECK
    row_or = np.bitwise_or.reduce(gpu["draft_status"], axis=1)
    np.testing.assert_array_equal(row_or, oflags)
    sampled = (tau > 0) & (oflags == 0)
    excused = 0
    for b in range(B):
        for r in range(R):
            g, o = int(gpu["draft_ids"][b, r]), int(orc["draft_ids"][b, r])
            if g == o:
                continue
            assert sampled[b], "row (%d,%d): gpu %d oracle %d without a sampled distribution" % (b, r, g, o)
            v = float(u[b, r])
            ok = orc["probe_w"][b, r] > 0 and orc["probe_lo"][b, r] - TOL_U <= v <= orc["probe_hi"][b, r] + TOL_U
            assert ok, "row (%d,%d): gpu %d oracle %d, v=%.9f gpu-id interval [%.9f, %.9f] w=%.3e" % (
                b, r, g, o, v, orc["probe_lo"][b, r], orc["probe_hi"][b, r], orc["probe_w"][b, r])
            excused += 1
    if sampled.any():
        same = (gpu["draft_ids"] == orc["draft_ids"]) & sampled[:, None]
        err = np.abs(gpu["q_draft"].astype(np.float64) - orc["q_draft"])[same]
        assert err.size == 0 or err.max() <= TOL_P, err.max()
    greedy = (tau == 0) & (oflags == 0)
    assert (gpu["q_draft"][greedy] == 1.0).all()
    return excused, orc


def make(B, R, V_d, dtype, f_mapped, seed, taus=(0.0, 0.6, 1.0), V_t=None, sigma=2.0):
    rng = np.random.default_rng(seed)
    z = rng.normal(0, sigma, (B, R, V_d)).astype(np.float32)
    z -= 1.2 * np.log1p(rng.permutation(V_d)).astype(np.float32)          # a rank bias, as in the workloads
    if dtype == wl.BF16:
        z = wl.f32_to_bf16_bits(z)
    V_t = V_t or V_d + 13
    id_map = np.full(V_d, -1, np.int32)
    mapped = rng.random(V_d) < f_mapped
    id_map[mapped] = rng.permutation(V_t)[:int(mapped.sum())]
    tau = rng.choice(np.array(taus, np.float32), B)
    u = rng.integers(0, 1 << 24, (B, R)).astype(np.float32) / np.float32(1 << 24)
    return z, id_map, tau, u, V_t


@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
@pytest.mark.parametrize("B,R,V_d", [(5, 1, 3), (4, 3, 13), (6, 2, 257), (3, 4, 4099), (2, 2, 8192), (3, 1, 33001)])
def test_small_and_ragged_vocabularies(dtype, B, R, V_d):
    z, id_map, tau, u, V_t = make(B, R, V_d, dtype, 0.6, seed=100 + V_d)
    gpu = run_gpu(z, id_map, tau, u, V_t)
    compare(z, id_map, tau, u, gpu)
    ids = gpu["draft_ids"]
    assert ((ids >= 0) & (ids < V_d)).all() and (id_map[ids] >= 0).all()       # always inside the intersection


@pytest.mark.parametrize("name", ["cfg0", "cfg1", "cfg2", "cfg3", "cfg4"])
def test_drafter_rows_of_the_five_workloads(name):
    """The drafter logits of each workload at full width and full batch (all K rows of every sequence)."""
    cfg = wl.config_by_name(name)
    batch = wl.make_batch(cfg)
    zd = batch["drafter_logits"]
    B, K, _ = zd.shape
    u = batch["uniforms"][:, :K]
    gpu = run_gpu(zd, batch["id_map"], batch["temperature"], u, cfg.V_t)
    excused, orc = compare(zd, batch["id_map"], batch["temperature"], u, gpu)
    assert excused <= 4
    assert (orc["flags"] == 0).all()


def test_drawn_ids_feed_the_verification_call():
    """Draft on the GPU, verify on the GPU, both against the oracle pipeline."""
    cfg = wl.tiny_config(B=6, K=4, V_t=30011, V_d=21001, dtype=wl.BF16, f_mapped=0.5, temperatures=(0.0, 0.8, 1.0), seed=131)
    batch = wl.make_batch(cfg)
    v = tli.Verifier(cfg.V_t, cfg.V_d, batch["id_map"])
    zt, zd = dev_logits(batch["target_logits"]), dev_logits(batch["drafter_logits"])
    tau = torch.from_numpy(batch["temperature"]).cuda()
    u = torch.from_numpy(batch["uniforms"]).cuda()
    d = v.draft(zd, tau, u[:, :cfg.K].contiguous())
    out = v.verify(zt, zd, d["draft_ids"], tau, u)
    torch.cuda.synchronize()
    ids = d["draft_ids"].cpu().numpy()
    od = oracle.draft(batch["drafter_logits"], batch["id_map"], batch["temperature"], batch["uniforms"][:, :cfg.K])
    np.testing.assert_array_equal(ids, od["draft_ids"])                          # no boundary cases with this seed
    ov = oracle.verify(batch["target_logits"], batch["drafter_logits"], batch["id_map"], ids,
                       batch["temperature"], batch["uniforms"])
    np.testing.assert_array_equal(out["accepted"].cpu().numpy(), ov["accepted"])
    np.testing.assert_array_equal(out["next_token"].cpu().numpy(), ov["next_token"])
    sampled = batch["temperature"] > 0
    np.testing.assert_allclose(out["q_draft"].cpu().numpy()[sampled], d["q_draft"].cpu().numpy()[sampled], atol=2e-6)
    v.close()


def test_strided_and_offset_rows():
    rng = np.random.default_rng(140)
    B, R, V_d = 5, 3, 6007
    big = torch.from_numpy(rng.normal(0, 2, (B, R + 2, V_d + 9)).astype(np.float32)).to(torch.bfloat16).cuda()
    view = big[:, 1:R + 1, 3:3 + V_d]                                            # odd element offset: rows not 16-byte aligned
    zd = view.contiguous().view(torch.uint16).cpu().numpy()
    _, id_map, tau, u, V_t = make(B, R, V_d, wl.BF16, 0.4, seed=141)
    gpu = run_gpu(zd, id_map, tau, u, V_t, zd_dev=view)
    compare(zd, id_map, tau, u, gpu)


def test_empty_intersection_bad_temperature_and_nonfinite_rows():
    z, id_map, tau, u, V_t = make(4, 2, 5000, wl.F32, 0.5, seed=150, taus=(1.0,))
    none = run_gpu(z, np.full(5000, -1, np.int32), [1.0, 0.0, 0.5, 2.0], u, V_t)
    np.testing.assert_array_equal(none["draft_ids"], -1)
    assert (none["draft_status"] == tli.TLI_ROW_FALLBACK).all() and (none["q_draft"] == 0).all()
    bad = run_gpu(z, id_map, [-1.0, np.nan, np.inf, 1.0], u, V_t)
    np.testing.assert_array_equal(bad["draft_ids"][:3], -1)
    assert (bad["draft_status"][:3] == tli.TLI_ROW_BAD_TEMPERATURE).all() and (bad["draft_status"][3] == 0).all()
    inside, outside = np.flatnonzero(id_map >= 0), np.flatnonzero(id_map < 0)
    ref = run_gpu(z, id_map, tau, u, V_t)
    z2 = z.copy()
    z2[1, 0, inside[7]] = np.nan
    z2[2, 1, inside[-1]] = np.inf
    z2[0, 0, outside[3]] = np.nan             # outside the intersection: does not enter q', is not examined
    z2[3, 1, outside[-1]] = np.inf
    for t in (tau, np.zeros(4, np.float32)):
        nf = run_gpu(z2, id_map, t, u, V_t)
        assert nf["draft_ids"][1, 0] == -1 and nf["draft_status"][1, 0] == tli.TLI_ROW_NONFINITE
        assert nf["draft_ids"][2, 1] == -1 and nf["draft_status"][2, 1] == tli.TLI_ROW_NONFINITE
        ok = np.ones((4, 2), bool)
        ok[1, 0] = ok[2, 1] = False
        assert (nf["draft_status"][ok] == 0).all()
        if t is tau:
            np.testing.assert_array_equal(nf["draft_ids"][ok], ref["draft_ids"][ok])


def test_minus_infinity_is_a_token_of_probability_zero():
    z, id_map, tau, u, V_t = make(3, 2, 9001, wl.F32, 0.7, seed=160, taus=(0.0, 1.0))
    hole = np.random.default_rng(161).random(z.shape) < 0.3
    z_inf = np.where(hole, -np.inf, z).astype(np.float32)
    z_big = np.where(hole, -1e30, z).astype(np.float32)
    gpu = run_gpu(z_inf, id_map, tau, u, V_t)
    assert (gpu["draft_status"] == 0).all()
    compare(z_big, id_map, tau, u, gpu)


def test_temperature_zero_ties_take_the_lowest_id_inside_the_intersection():
    V_d = 20000
    z = np.zeros((2, 1, V_d), np.float32)
    z[:, 0, [17, 4100, 4101, 19999]] = 3.0
    id_map = np.arange(V_d, dtype=np.int32)
    id_map[17] = -1
    for dtype in (wl.F32, wl.BF16):
        zz = z if dtype == wl.F32 else wl.f32_to_bf16_bits(z)
        gpu = run_gpu(zz, id_map, [0.0, 0.0], [[0.1], [0.9]], V_d)
        np.testing.assert_array_equal(gpu["draft_ids"], 4100)


def test_argument_errors_are_reported_not_launched():
    z, id_map, tau, u, V_t = make(2, 2, 1000, wl.F32, 0.5, seed=170)
    v = tli.Verifier(V_t, 1000, id_map)
    zd = dev_logits(z)
    ids = torch.empty(2, 2, dtype=torch.int32, device="cuda")
    ws = torch.empty(tli.tli_draft_workspace_bytes(v.ctx, 2, 2, tli.TLI_F32), dtype=torch.uint8, device="cuda")
    t = torch.from_numpy(tau).cuda()
    uu = torch.from_numpy(u).cuda()
    good = tli.make_draft_args(zd, t, uu, ids, ws)
    tli.tli_draft_sample(v.ctx, good)
    for field, value, code in (("B", 0, tli.TLI_ERR_ARG), ("R", 0, tli.TLI_ERR_ARG), ("dtype", 7, tli.TLI_ERR_ARG),
                               ("drafter_logits", None, tli.TLI_ERR_ARG), ("draft_ids", None, tli.TLI_ERR_ARG),
                               ("workspace_bytes", 16, tli.TLI_ERR_WORKSPACE), ("B", 40000, tli.TLI_ERR_UNSUPPORTED)):
        a = tli.make_draft_args(zd, t, uu, ids, ws)
        setattr(a, field, value)
        with pytest.raises(tli.TLIError) as e:
            tli.tli_draft_sample(v.ctx, a)
        assert e.value.code == code, field
    assert tli.tli_draft_workspace_bytes(v.ctx, 0, 1, tli.TLI_F32) == 0
    assert tli.tli_draft_workspace_bytes(v.ctx, 70000, 1, tli.TLI_F32) == 0
    torch.cuda.synchronize()
    v.close()


def test_largest_vocabulary_and_most_rows():
    """V_d at the library's limit (fp32: 257 tiles, 2056 strips per row) and B * R at its limit."""
    V_d = 1 << 20
    z, id_map, tau, u, V_t = make(1, 2, V_d, wl.F32, 0.3, seed=180, taus=(0.9,), V_t=V_d)
    gpu = run_gpu(z, id_map, [0.9], u, V_t)
    compare(z, id_map, [0.9], u, gpu)
    gpu0 = run_gpu(z, id_map, [0.0], u, V_t)
    compare(z, id_map, [0.0], u, gpu0)
    B = 65535
    z, id_map, tau, u, V_t = make(B, 1, 40, wl.BF16, 0.5, seed=181)
    many = run_gpu(z, id_map, tau, u, V_t)
    compare(z, id_map, tau, u, many)
