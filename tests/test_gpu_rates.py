"""Parity of tli_acceptance_rates() (the paper's expected acceptance rates per draft position) with
its fp64 oracle: mass, alpha_union, alpha_tli within 1e-5 absolute; temperature-0 positions (0 or 1)
and the status bits exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2502_05202_b200 import tli, workload as wl

pytestmark = pytest.mark.gpu

TOL = 1e-5


def dev_logits(z):
    t = torch.from_numpy(np.ascontiguousarray(z))
    if t.dtype == torch.uint16:
        t = t.view(torch.bfloat16)
    return t.cuda()


def run_gpu(zt, zd, id_map, tau, V_t=None, zt_dev=None, zd_dev=None):
    v = tli.Verifier(zt.shape[2] if V_t is None else V_t, zd.shape[2], id_map)
    a = dev_logits(zt) if zt_dev is None else zt_dev
    d = dev_logits(zd) if zd_dev is None else zd_dev
    t = torch.from_numpy(np.asarray(tau, np.float32)).cuda()
    out = v.rates(a, d, t)
    torch.cuda.synchronize()
    res = {k: x.cpu().numpy() for k, x in out.items()}
    again = v.rates(a, d, t)
    torch.cuda.synchronize()
    for k in res:
        np.testing.assert_array_equal(res[k], again[k].cpu().numpy(), err_msg="repeat call differs: " + k)
    v.close()
    return res


def compare(zt, zd, id_map, tau, gpu, threads=8):
    tau = np.asarray(tau, np.float32)
    orc = oracle.rates(zt, zd, id_map, tau, threads=threads)
    np.testing.assert_array_equal(np.bitwise_or.reduce(gpu["position_status"], axis=1), orc["flags"])
    flagged = gpu["position_status"] != 0                    # the oracle leaves zeros at a flagged position too
    for k in ("mass", "alpha_union", "alpha_tli"):
        err = np.abs(gpu[k].astype(np.float64) - orc[k])
        assert err.max() <= TOL, (k, err.max())
        cold = tau == 0
        np.testing.assert_array_equal(gpu[k][cold], orc[k][cold].astype(np.float32))
        assert (gpu[k][flagged] == 0).all()
    assert (gpu["alpha_union"] <= gpu["alpha_tli"] + 1e-6).all()               # Theorem 4.1 on the GPU's own numbers
    return orc


@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
@pytest.mark.parametrize("B,K,V_t,V_d", [(3, 1, 3, 4), (4, 2, 13, 11), (5, 3, 300, 257), (3, 2, 4099, 5000),
                                          (2, 2, 33001, 8192), (2, 1, 9000, 40001)])
def test_small_and_ragged_vocabularies(dtype, B, K, V_t, V_d):
    cfg = wl.tiny_config(B=B, K=K, V_t=V_t, V_d=V_d, dtype=dtype, f_mapped=0.6, sigma_d=0.8,
                         temperatures=(0.0, 0.6, 1.0), seed=300 + V_t)
    b = wl.make_batch(cfg)
    gpu = run_gpu(b["target_logits"], b["drafter_logits"], b["id_map"], b["temperature"])
    compare(b["target_logits"], b["drafter_logits"], b["id_map"], b["temperature"], gpu)


@pytest.mark.parametrize("name", ["cfg0", "cfg1", "cfg2", "cfg3", "cfg4"])
def test_positions_of_the_five_workloads(name):
    cfg = wl.config_by_name(name)
    batch = wl.make_batch(cfg, rows=list(range(min(cfg.B, 24))))
    gpu = run_gpu(batch["target_logits"], batch["drafter_logits"], batch["id_map"], batch["temperature"])
    orc = compare(batch["target_logits"], batch["drafter_logits"], batch["id_map"], batch["temperature"], gpu)
    sampled = batch["temperature"] > 0
    assert (orc["flags"] == 0).all() and (orc["alpha_tli"][sampled] >= orc["alpha_union"][sampled]).all()


def test_strided_rows_and_the_worked_example():
    rng = np.random.default_rng(340)
    B, K, V_t, V_d = 4, 3, 6007, 5003
    bt = torch.from_numpy(rng.normal(0, 2, (B, K + 3, V_t + 9)).astype(np.float32)).to(torch.bfloat16).cuda()
    bd = torch.from_numpy(rng.normal(0, 2, (B, K + 1, V_d + 5)).astype(np.float32)).to(torch.bfloat16).cuda()
    vt, vd = bt[:, 1:K + 2, 3:3 + V_t], bd[:, 1:K + 1, 1:1 + V_d]
    zt = vt.contiguous().view(torch.uint16).cpu().numpy()
    zd = vd.contiguous().view(torch.uint16).cpu().numpy()
    id_map = np.full(V_d, -1, np.int32)
    inside = rng.random(V_d) < 0.5
    id_map[inside] = rng.permutation(V_t)[:int(inside.sum())]
    tau = np.array([1.0, 0.0, 0.7, 1.3], np.float32)
    gpu = run_gpu(zt, zd, id_map, tau, zt_dev=vt, zd_dev=vd)
    compare(zt, zd, id_map, tau, gpu)
    # q = 1/3,1/3,1/3 on {a,b,c}, T = {a,b}, p = 1/2,1/2: M = 2/3, alpha_union = 2/3, alpha_tli = 1
    ex = run_gpu(np.zeros((1, 1, 2), np.float32), np.zeros((1, 1, 3), np.float32), np.array([0, 1, -1], np.int32), [1.0])
    assert ex["mass"][0, 0] == pytest.approx(2 / 3, abs=1e-6) and ex["alpha_union"][0, 0] == pytest.approx(2 / 3, abs=1e-6)
    assert ex["alpha_tli"][0, 0] == pytest.approx(1.0, abs=1e-6)


def test_flags_and_degenerate_maps():
    cfg = wl.tiny_config(B=5, K=2, V_t=7001, V_d=6001, dtype=wl.F32, f_mapped=0.5, temperatures=(1.0,), seed=350)
    b = wl.make_batch(cfg)
    zt, zd = b["target_logits"], b["drafter_logits"]
    none = run_gpu(zt, zd, np.full(cfg.V_d, -1, np.int32), [1.0, 0.0, 0.5, 1.0, 2.0], V_t=cfg.V_t)
    assert (none["position_status"] == tli.TLI_ROW_FALLBACK).all()
    for k in ("mass", "alpha_union", "alpha_tli"):
        assert (none[k] == 0).all()
    bad = run_gpu(zt, zd, b["id_map"], [-1.0, np.nan, np.inf, 1.0, 1.0])
    assert (bad["position_status"][:3] == tli.TLI_ROW_BAD_TEMPERATURE).all() and (bad["position_status"][3:] == 0).all()
    z2t, z2d = zt.copy(), zd.copy()
    z2t[1, 0, 17] = np.nan
    z2d[3, 1, 6000] = np.inf
    for tau in ([1.0] * 5, [0.0] * 5):
        nf = run_gpu(z2t, z2d, b["id_map"], tau)
        compare(z2t, z2d, b["id_map"], tau, nf)
        assert nf["position_status"][1, 0] == tli.TLI_ROW_NONFINITE and nf["position_status"][3, 1] == tli.TLI_ROW_NONFINITE
        assert nf["position_status"].sum() == 2 * tli.TLI_ROW_NONFINITE
    ident = run_gpu(zt[:, :, :6001].copy(), zt[:, :2, :6001].copy(), np.arange(6001, dtype=np.int32), [1.0] * 5)
    for k in ("mass", "alpha_union", "alpha_tli"):
        np.testing.assert_allclose(ident[k], 1.0, atol=2e-6)                 # q = p on T = D


def test_argument_errors_are_reported_not_launched():
    cfg = wl.tiny_config(B=2, K=2, V_t=900, V_d=800, dtype=wl.F32, f_mapped=0.5, seed=360)
    b = wl.make_batch(cfg)
    v = tli.Verifier(cfg.V_t, cfg.V_d, b["id_map"])
    zt, zd = dev_logits(b["target_logits"]), dev_logits(b["drafter_logits"])
    t = torch.from_numpy(b["temperature"]).cuda()
    outs = [torch.empty(2, 2, dtype=torch.float32, device="cuda") for _ in range(3)]
    ws = torch.empty(tli.tli_rates_workspace_bytes(v.ctx, 2, 2, tli.TLI_F32), dtype=torch.uint8, device="cuda")
    tli.tli_acceptance_rates(v.ctx, tli.make_rates_args(zt, zd, t, *outs, ws))
    for field, value, code in (("B", 0, tli.TLI_ERR_ARG), ("K", 0, tli.TLI_ERR_ARG), ("dtype", 5, tli.TLI_ERR_ARG),
                               ("target_logits", None, tli.TLI_ERR_ARG), ("mass", None, tli.TLI_ERR_ARG),
                               ("workspace_bytes", 8, tli.TLI_ERR_WORKSPACE), ("B", 20000, tli.TLI_ERR_UNSUPPORTED)):
        a = tli.make_rates_args(zt, zd, t, *outs, ws)
        setattr(a, field, value)
        with pytest.raises(tli.TLIError) as e:
            tli.tli_acceptance_rates(v.ctx, a)
        assert e.value.code == code, field
    assert tli.tli_rates_workspace_bytes(v.ctx, 0, 1, tli.TLI_F32) == 0
    torch.cuda.synchronize()
    v.close()
