"""Parity of tli_slem_verify() (Algorithm 2's exact-match verification) with its fp64 oracle.

Rule: every sampled token t'_j (j <= m_b) must be identical to the oracle's, except that a difference
is excused -- and counted -- when the GPU's token has positive weight in the oracle's p_j and the
uniform lies within 1e-6 of the oracle's normalised CDF interval of that token.  accepted and
next_token must follow from the GPU's own sampled tokens by definition (first mismatch), and equal
the oracle's wherever no excuse was used.  Temperature-0 rows and status bits get no excuses."""
import numpy as np
import pytest
import torch

import oracle
from paper_2502_05202_b200 import tli, workload as wl

pytestmark = pytest.mark.gpu

TOL_U = 1e-6


def dev_logits(z):
    t = torch.from_numpy(np.ascontiguousarray(z))
    if t.dtype == torch.uint16:
        t = t.view(torch.bfloat16)
    return t.cuda()


def run_gpu(zt, cand, tau, u, lengths=None, zt_dev=None, verifier=None):
    B, M1, V_t = zt.shape
    own = verifier is None
    v = verifier or tli.Verifier(V_t, 8, np.full(8, -1, np.int32))        # the id map plays no part
    z = dev_logits(zt) if zt_dev is None else zt_dev
    c = torch.from_numpy(np.asarray(cand, np.int32).reshape(B, M1 - 1)).cuda()
    t = torch.from_numpy(np.asarray(tau, np.float32)).cuda()
    uu = torch.from_numpy(np.asarray(u, np.float32).reshape(B, M1)).cuda()
    ln = None if lengths is None else torch.from_numpy(np.asarray(lengths, np.int32)).cuda()
    out = v.slem(z, c, t, uu, ln)
    torch.cuda.synchronize()
    res = {k: x.cpu().numpy() for k, x in out.items()}
    again = v.slem(z, c, t, uu, ln)
    torch.cuda.synchronize()
    for k in res:
        np.testing.assert_array_equal(res[k], again[k].cpu().numpy(), err_msg="repeat call differs: " + k)
    if own:
        v.close()
    return res


def compare(zt, cand, tau, u, gpu, lengths=None, threads=8):
    B, M1, V_t = zt.shape
    M = M1 - 1
    cand = np.asarray(cand, np.int32).reshape(B, M)
    tau = np.asarray(tau, np.float32)
    u = np.asarray(u, np.float32).reshape(B, M1)
    m = np.full(B, M, np.int32) if lengths is None else np.asarray(lengths, np.int32)
    orc = oracle.slem(zt, cand, tau, u, lengths=lengths, probe_token=np.clip(gpu["sampled"], 0, V_t - 1), threads=threads)
    np.testing.assert_array_equal(gpu["row_status"], orc["flags"])
    excused = 0
    for b in range(B):
        if orc["flags"][b]:
            assert gpu["accepted"][b] == 0 and gpu["next_token"][b] == 0 and (gpu["sampled"][b] == -1).all()
            continue
        used = False
        for j in range(M1):
            g, o = int(gpu["sampled"][b, j]), int(orc["sampled"][b, j])
            if j > m[b]:
                assert g == -1
                continue
            if g == o:
                continue
            assert tau[b] > 0, "row (%d,%d): temperature 0, gpu %d oracle %d" % (b, j, g, o)
            v = float(u[b, j])
            ok = orc["probe_w"][b, j] > 0 and orc["probe_lo"][b, j] - TOL_U <= v <= orc["probe_hi"][b, j] + TOL_U
            assert ok, "row (%d,%d): gpu %d oracle %d, v=%.9f interval [%.9f, %.9f] w=%.3e" % (
                b, j, g, o, v, orc["probe_lo"][b, j], orc["probe_hi"][b, j], orc["probe_w"][b, j])
            excused += 1
            used = True
        n = 0
        while n < m[b] and gpu["sampled"][b, n] == cand[b, n]:
            n += 1
        assert gpu["accepted"][b] == n and gpu["next_token"][b] == gpu["sampled"][b, n]
        if not used:
            assert gpu["accepted"][b] == orc["accepted"][b] and gpu["next_token"][b] == orc["next_token"][b]
    return excused, orc


def make(B, M, V_t, dtype, seed, taus=(0.0, 0.6, 1.0), hit=0.7):
    """Target rows with a rank bias; candidates = what the oracle samples, with mismatches planted."""
    rng = np.random.default_rng(seed)
    z = rng.normal(0, 2.0, (B, M + 1, V_t)).astype(np.float32)
    z -= 1.2 * np.log1p(rng.permutation(V_t)).astype(np.float32)
    if dtype == wl.BF16:
        z = wl.f32_to_bf16_bits(z)
    tau = rng.choice(np.array(taus, np.float32), B)
    u = rng.integers(0, 1 << 24, (B, M + 1)).astype(np.float32) / np.float32(1 << 24)
    own = oracle.slem(z, np.zeros((B, M), np.int32), tau, u)["sampled"][:, :M]
    miss = rng.random((B, M)) > hit
    cand = np.where(miss, (own + 1 + rng.integers(0, V_t - 1, (B, M))) % V_t, own).astype(np.int32)
    return z, cand, tau, u


@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
@pytest.mark.parametrize("B,M,V_t", [(5, 0, 3), (4, 3, 13), (6, 2, 257), (3, 4, 4099), (2, 2, 8192), (3, 1, 33001)])
def test_small_and_ragged_vocabularies(dtype, B, M, V_t):
    z, cand, tau, u = make(B, M, V_t, dtype, seed=200 + V_t)
    gpu = run_gpu(z, cand, tau, u)
    compare(z, cand, tau, u, gpu)


@pytest.mark.parametrize("name", ["cfg0", "cfg1", "cfg2", "cfg3", "cfg4"])
def test_target_rows_of_the_five_workloads(name):
    """The target logits of each workload (up to 48 sequences); candidates = the drafts carried to target ids."""
    cfg = wl.config_by_name(name)
    rows = list(range(min(cfg.B, 48)))
    batch = wl.make_batch(cfg, rows=rows)
    zt = batch["target_logits"]
    cand = batch["id_map"][batch["draft_ids"]].astype(np.int32)
    lengths = (np.arange(len(rows)) % (cfg.K + 1)).astype(np.int32) if name == "cfg2" else None
    gpu = run_gpu(zt, cand, batch["temperature"], batch["uniforms"], lengths)
    excused, orc = compare(zt, cand, batch["temperature"], batch["uniforms"], gpu, lengths)
    assert excused <= 2 and (orc["flags"] == 0).all()


def test_ragged_lengths_and_planted_mismatches():
    z, cand, tau, u = make(9, 5, 20011, wl.BF16, seed=230, hit=0.85)
    lengths = np.array([0, 1, 2, 3, 4, 5, 5, 2, 0], np.int32)
    gpu = run_gpu(z, cand, tau, u, lengths)
    excused, orc = compare(z, cand, tau, u, gpu, lengths)
    assert (gpu["accepted"] <= lengths).all()
    assert len(set(gpu["accepted"].tolist())) > 2                          # both matches and mismatches occurred


def test_strided_and_offset_rows():
    rng = np.random.default_rng(240)
    B, M, V_t = 4, 3, 7001
    big = torch.from_numpy(rng.normal(0, 2, (B, M + 3, V_t + 9)).astype(np.float32)).to(torch.bfloat16).cuda()
    view = big[:, 1:M + 2, 5:5 + V_t]
    zt = view.contiguous().view(torch.uint16).cpu().numpy()
    tau = np.array([1.0, 0.0, 0.7, 1.0], np.float32)
    u = rng.random((B, M + 1)).astype(np.float32)
    cand = oracle.slem(zt, np.zeros((B, M), np.int32), tau, u)["sampled"][:, :M].copy()
    cand[2, 1] += 1
    gpu = run_gpu(zt, cand, tau, u, zt_dev=view)
    compare(zt, cand, tau, u, gpu)


def test_bad_temperature_and_nonfinite_rows():
    z, cand, tau, u = make(5, 3, 6000, wl.F32, seed=250, taus=(1.0,))
    bad = run_gpu(z, cand, [-1.0, np.nan, np.inf, 1.0, 0.0], u)
    assert (bad["row_status"][:3] == tli.TLI_ROW_BAD_TEMPERATURE).all() and (bad["row_status"][3:] == 0).all()
    assert (bad["accepted"][:3] == 0).all() and (bad["sampled"][:3] == -1).all()
    z2 = z.copy()
    z2[1, 2, 100] = np.nan
    z2[3, 0, 5999] = np.inf
    z2[4, 3, 7] = np.nan                                                   # beyond m_4 = 1: never read
    lengths = np.array([3, 3, 3, 3, 1], np.int32)
    for t in (tau, np.zeros(5, np.float32)):
        gpu = run_gpu(z2, cand, t, u, lengths)
        compare(z2, cand, t, u, gpu, lengths)
        assert gpu["row_status"].tolist() == [0, tli.TLI_ROW_NONFINITE, 0, tli.TLI_ROW_NONFINITE, 0]


def test_minus_infinity_is_a_token_of_probability_zero():
    z, cand, tau, u = make(3, 2, 9001, wl.F32, seed=260, taus=(0.0, 1.0))
    hole = np.random.default_rng(261).random(z.shape) < 0.3
    gpu = run_gpu(np.where(hole, -np.inf, z).astype(np.float32), cand, tau, u)
    assert (gpu["row_status"] == 0).all()
    compare(np.where(hole, -1e30, z).astype(np.float32), cand, tau, u, gpu)


def test_argument_errors_are_reported_not_launched():
    z, cand, tau, u = make(2, 2, 1000, wl.F32, seed=270)
    v = tli.Verifier(1000, 8, np.full(8, -1, np.int32))
    zt = dev_logits(z)
    acc = torch.empty(2, dtype=torch.int32, device="cuda")
    nxt = torch.empty(2, dtype=torch.int32, device="cuda")
    ws = torch.empty(tli.tli_slem_workspace_bytes(v.ctx, 2, 2, tli.TLI_F32), dtype=torch.uint8, device="cuda")
    c, t, uu = torch.from_numpy(cand).cuda(), torch.from_numpy(tau).cuda(), torch.from_numpy(u).cuda()
    tli.tli_slem_verify(v.ctx, tli.make_slem_args(zt, c, t, uu, acc, nxt, ws))
    for field, value, code in (("B", 0, tli.TLI_ERR_ARG), ("M", -1, tli.TLI_ERR_ARG), ("dtype", 9, tli.TLI_ERR_ARG),
                               ("target_logits", None, tli.TLI_ERR_ARG), ("candidates", None, tli.TLI_ERR_ARG),
                               ("accepted", None, tli.TLI_ERR_ARG), ("workspace_bytes", 16, tli.TLI_ERR_WORKSPACE),
                               ("M", 65, tli.TLI_ERR_UNSUPPORTED), ("B", 40000, tli.TLI_ERR_UNSUPPORTED)):
        a = tli.make_slem_args(zt, c, t, uu, acc, nxt, ws)
        setattr(a, field, value)
        with pytest.raises(tli.TLIError) as e:
            tli.tli_slem_verify(v.ctx, a)
        assert e.value.code == code, field
    assert tli.tli_slem_workspace_bytes(v.ctx, 0, 1, tli.TLI_F32) == 0
    torch.cuda.synchronize()
    v.close()


def test_largest_vocabulary_and_most_rows():
    """V_t at the library's limit (fp32: 257 tiles, 2056 strips per row) and B * (M+1) at its limit."""
    z, cand, tau, u = make(1, 1, 1 << 20, wl.F32, seed=280, taus=(0.0, 0.9))
    for t in ([0.9], [0.0]):
        gpu = run_gpu(z, cand, t, u)
        compare(z, cand, t, u, gpu)
    z, cand, tau, u = make(21845, 2, 50, wl.BF16, seed=281)
    gpu = run_gpu(z, cand, tau, u)
    compare(z, cand, tau, u, gpu)
