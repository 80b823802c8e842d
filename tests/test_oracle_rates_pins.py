"""Pins of the expected-acceptance-rate oracle (the paper's table of expected acceptance rates:
sum over the intersection of min{p, q} when drafting from q, of min{p, q'} when drafting from q')."""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def softmax(z, tau):
    z = np.asarray(z, np.float64)
    e = np.exp((z - z.max()) / tau)
    return e / e.sum()


def random_case(rng, B, K, V_t, V_d, n_in):
    zt = rng.normal(0, 1.5, (B, K + 1, V_t)).astype(np.float32)
    zd = rng.normal(0, 1.5, (B, K, V_d)).astype(np.float32)
    id_map = np.full(V_d, -1, np.int32)
    id_map[rng.choice(V_d, n_in, replace=False)] = rng.permutation(V_t)[:n_in]
    return zt, zd, id_map


def test_worked_example_of_the_paper():
    """q = 1/3,1/3,1/3 on {a,b,c}, T = {a,b}: M = 2/3, q' = 1/2,1/2; with p = 1/2,1/2 every draft from q'
    is accepted (rate 1) while drafting from q accepts with 1/3 + 1/3."""
    rows = [l.split() for l in open(os.path.join(GOLDEN, "qprime_worked_example.txt")) if l.strip() and l[0] != "#"]
    in_T = np.array([int(r[1]) for r in rows])
    id_map = np.where(in_T == 1, np.arange(len(rows)), -1).astype(np.int32)
    out = oracle.rates(np.zeros((1, 1, 2), np.float32), np.zeros((1, 1, 3), np.float32), id_map, [1.0])
    assert out["mass"][0, 0] == pytest.approx(2 / 3, abs=1e-15)
    assert out["alpha_union"][0, 0] == pytest.approx(2 / 3, abs=1e-15)
    assert out["alpha_tli"][0, 0] == pytest.approx(1.0, abs=1e-15)


@pytest.mark.parametrize("seed", range(4))
def test_direct_evaluation_and_theorem_4_1(seed):
    rng = np.random.default_rng(seed)
    B, K, V_t, V_d = 3, 2, 9, 11
    zt, zd, id_map = random_case(rng, B, K, V_t, V_d, 6)
    tau = np.array([0.6, 1.0, 1.4], np.float32)
    out = oracle.rates(zt, zd, id_map, tau)
    inside = np.flatnonzero(id_map >= 0)
    for b in range(B):
        for j in range(K):
            p, q = softmax(zt[b, j], float(tau[b])), softmax(zd[b, j], float(tau[b]))
            M = q[inside].sum()
            au = np.minimum(p[id_map[inside]], q[inside]).sum()
            at = np.minimum(p[id_map[inside]], q[inside] / M).sum()
            assert out["mass"][b, j] == pytest.approx(M, rel=1e-12)
            assert out["alpha_union"][b, j] == pytest.approx(au, rel=1e-12)
            assert out["alpha_tli"][b, j] == pytest.approx(at, rel=1e-12)
    assert (out["alpha_union"] <= out["alpha_tli"] + 1e-15).all()              # Theorem 4.1
    assert (out["alpha_tli"] <= 1 + 1e-15).all() and (out["mass"] <= 1 + 1e-15).all()


def test_identity_and_disjoint_vocabularies():
    rng = np.random.default_rng(9)
    V = 12
    zt = rng.normal(0, 1, (2, 3, V)).astype(np.float32)
    same = oracle.rates(zt, zt[:, :2].copy(), np.arange(V, dtype=np.int32), [1.0, 0.7])     # q = p, T = D
    np.testing.assert_allclose(same["mass"], 1.0, atol=1e-12)
    np.testing.assert_allclose(same["alpha_union"], 1.0, atol=1e-12)
    np.testing.assert_allclose(same["alpha_tli"], 1.0, atol=1e-12)
    none = oracle.rates(zt, zt[:, :2].copy(), np.full(V, -1, np.int32), [1.0, 0.7])
    for k in ("mass", "alpha_union", "alpha_tli"):
        np.testing.assert_array_equal(none[k], 0.0)
    assert (none["flags"] & oracle.FLAG_FALLBACK).all()


def test_monte_carlo_acceptance_of_the_drafting_and_verification_oracles_matches_alpha_tli():
    """Draw d ~ q' with the drafting oracle, verify with the verification oracle: the frequency of
    accepting the first draft is alpha_tli (and drafting from q would give alpha_union)."""
    rng = np.random.default_rng(10)
    V_t, V_d, N = 8, 10, 200_000
    zt1, zd1, id_map = random_case(rng, 1, 1, V_t, V_d, 6)
    tau = np.float32(0.9)
    want = oracle.rates(zt1, zd1, id_map, [tau])
    zt = np.broadcast_to(zt1, (N, 2, V_t))
    zd = np.broadcast_to(zd1, (N, 1, V_d))
    u = rng.integers(0, 1 << 24, (N, 2)).astype(np.float32) / np.float32(1 << 24)
    ud = rng.integers(0, 1 << 24, (N, 1)).astype(np.float32) / np.float32(1 << 24)
    taus = np.full(N, tau, np.float32)
    d = oracle.draft(zd, id_map, taus, ud, threads=4)
    v = oracle.verify(zt, zd, id_map, d["draft_ids"], taus, u, threads=4)
    freq = (v["accepted"] == 1).mean()
    a = want["alpha_tli"][0, 0]
    assert abs(freq - a) < 5 * np.sqrt(a * (1 - a) / N), (freq, a)
    # drafting from q itself (ids outside the intersection are rejected): alpha_union
    q = softmax(zd1[0, 0], float(tau))
    raw = np.searchsorted(np.cumsum(q), rng.random(N) * q.sum(), side="right").clip(0, V_d - 1).astype(np.int32)
    p = softmax(zt1[0, 0], float(tau))
    acc = np.where(id_map[raw] >= 0, rng.random(N) < np.minimum(1, p[np.maximum(id_map[raw], 0)] / q[raw]), False)
    au = want["alpha_union"][0, 0]
    assert abs(acc.mean() - au) < 5 * np.sqrt(au * (1 - au) / N), (acc.mean(), au)


def test_temperature_zero_is_the_one_hot_limit():
    rng = np.random.default_rng(11)
    B, K, V_t, V_d = 6, 2, 30, 40
    zt, zd, id_map = random_case(rng, B, K, V_t, V_d, 20)
    cold = oracle.rates(zt, zd, id_map, np.zeros(B, np.float32))
    nearly = oracle.rates(zt, zd, id_map, np.full(B, 1e-4, np.float32))
    for k in ("mass", "alpha_union", "alpha_tli"):
        assert set(np.unique(cold[k])) <= {0.0, 1.0}
        np.testing.assert_allclose(cold[k], nearly[k], atol=1e-6)


def test_flags_bf16_and_threads():
    from paper_2502_05202_b200 import workload as wl
    rng = np.random.default_rng(12)
    zt, zd, id_map = random_case(rng, 5, 3, 50, 60, 30)
    bt, bd = wl.f32_to_bf16_bits(zt), wl.f32_to_bf16_bits(zd)
    tau = np.array([1.0, 0.5, 0.0, 1.0, 0.8], np.float32)
    a = oracle.rates(bt, bd, id_map, tau)
    b = oracle.rates(wl.bf16_bits_to_f32(bt), wl.bf16_bits_to_f32(bd), id_map, tau, threads=3)
    for k in a:
        np.testing.assert_array_equal(a[k], b[k])
    bad = oracle.rates(zt, zd, id_map, [-1.0, np.nan, np.inf, 1.0, 1.0])
    assert (bad["flags"][:3] == oracle.FLAG_BAD_TEMPERATURE).all() and (bad["flags"][3:] == 0).all()
    zt[3, 1, 7] = np.nan
    assert oracle.rates(zt, zd, id_map, tau)["flags"][3] == oracle.FLAG_NONFINITE
