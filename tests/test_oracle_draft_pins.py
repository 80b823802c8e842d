"""Pins of the drafting oracle (Algorithm 4's q' as the sampling distribution of Algorithm 5's
drafting step) against what the paper and the mathematics fix -- none of them calls the
oracle's own formula for q' or its CDF walk."""
import os

import numpy as np
import pytest
from scipy import stats

import oracle
from paper_2502_05202_b200 import workload as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def f32(x):
    return float(np.float32(x))


def masked_softmax(z, mask, tau):
    """q restricted to the intersection and renormalised: softmax(z/tau) / its mass on the mask."""
    z = np.asarray(z, np.float64)
    q = np.exp((z - z.max()) / tau)
    q /= q.sum()
    qp = np.where(mask, q, 0.0)
    return qp / qp.sum()


def test_worked_example_from_the_paper_drives_the_draws():
    """Motivating example of Algorithm 4: q = 1/3,1/3,1/3 on {a,b,c}, T = {a,b} -> q' = 1/2,1/2,0."""
    rows = [l.split() for l in open(os.path.join(GOLDEN, "qprime_worked_example.txt")) if l.strip() and l[0] != "#"]
    in_T = np.array([int(r[1]) for r in rows])
    qprime = np.array([float(r[3]) for r in rows])
    id_map = np.where(in_T == 1, np.arange(len(rows)), -1).astype(np.int32)
    zd = np.zeros((1, 1, len(rows)), np.float32)                    # equal logits: q = 1/3 each
    edges = np.concatenate([[0.0], np.cumsum(qprime)])
    for v in np.arange(0, 1, 1 / 64):
        out = oracle.draft(zd, id_map, [1.0], [[v]])
        want = int(np.searchsorted(edges, v, side="right") - 1)
        assert out["draft_ids"][0, 0] == want
        assert out["q_draft"][0, 0] == pytest.approx(qprime[want], abs=1e-15)
        assert out["draft_ids"][0, 0] != 2                           # c is outside T: never drawn
    assert out["flags"][0] == 0


@pytest.mark.parametrize("V_d,n_mapped,tau,seed", [(12, 7, 1.0, 1), (16, 5, 0.6, 2), (9, 9, 1.3, 3)])
def test_draws_follow_qprime_chi_square(V_d, n_mapped, tau, seed):
    rng = np.random.default_rng(seed)
    z = rng.normal(0, 1.5, V_d).astype(np.float32)
    mapped = np.zeros(V_d, bool)
    mapped[rng.choice(V_d, n_mapped, replace=False)] = True
    id_map = np.where(mapped, np.arange(V_d), -1).astype(np.int32)   # any injective image will do
    N = 400_000
    u = (rng.integers(0, 1 << 24, N).astype(np.float32) / np.float32(1 << 24)).reshape(1, N)
    zd = np.broadcast_to(z, (1, N, V_d))
    out = oracle.draft(zd, id_map, [f32(tau)], u)
    ids = out["draft_ids"][0]
    assert (ids >= 0).all() and mapped[ids].all()
    want = masked_softmax(z, mapped, f32(tau))
    counts = np.bincount(ids, minlength=V_d)
    keep = want > 0
    chi2 = ((counts[keep] - N * want[keep]) ** 2 / (N * want[keep])).sum()
    pval = stats.chi2.sf(chi2, keep.sum() - 1)
    assert pval > 1e-4, (chi2, pval)


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_cdf_boundaries_by_brute_force(seed):
    """Weights 1..V through logits ln(k): the drawn id changes where the cumulative weights say."""
    rng = np.random.default_rng(seed)
    V_d = 8
    k = rng.permutation(np.arange(1, V_d + 1)).astype(np.float64)
    mapped = np.ones(V_d, bool)
    mapped[rng.choice(V_d, 3, replace=False)] = False
    id_map = np.where(mapped, np.arange(V_d)[::-1], -1).astype(np.int32)
    z = np.log(k).astype(np.float32)
    w = np.where(mapped, np.exp(z.astype(np.float64)), 0.0)
    edges = np.concatenate([[0.0], np.cumsum(w) / w.sum()])
    grid = np.arange(0, 1 << 12, dtype=np.float32) / np.float32(1 << 12)
    out = oracle.draft(np.broadcast_to(z, (1, len(grid), V_d)), id_map, [1.0], grid.reshape(1, -1))
    for v, d, lo, hi in zip(grid, out["draft_ids"][0], out["cdf_lo"][0], out["cdf_hi"][0]):
        want = int(np.searchsorted(edges, v, side="right") - 1)
        if min(abs(v - edges)) > 1e-9:
            assert d == want
        assert lo - 1e-12 <= v < hi + 1e-12
        assert mapped[d]


def test_full_intersection_is_a_plain_softmax_sampler():
    """Every drafter id in T: q' = q, and the draw is numpy's cumulative-sum search on softmax(z/tau)."""
    rng = np.random.default_rng(5)
    B, R, V_d = 6, 5, 301
    zd = rng.normal(0, 2, (B, R, V_d)).astype(np.float32)
    tau = np.array([0.5, 0.7, 1.0, 1.0, 1.5, 2.0], np.float32)
    u = rng.integers(0, 1 << 24, (B, R)).astype(np.float32) / np.float32(1 << 24)
    id_map = rng.permutation(V_d).astype(np.int32)
    out = oracle.draft(zd, id_map, tau, u)
    for b in range(B):
        for r in range(R):
            z = zd[b, r].astype(np.float64)
            q = np.exp((z - z.max()) / float(tau[b]))
            q /= q.sum()
            c = np.cumsum(q)
            want = int(np.searchsorted(c, float(u[b, r]) * c[-1], side="right"))
            near = np.min(np.abs(c / c[-1] - float(u[b, r]))) < 1e-12
            assert near or out["draft_ids"][b, r] == want
            assert out["q_draft"][b, r] == pytest.approx(q[out["draft_ids"][b, r]], rel=1e-12)


def test_temperature_zero_is_the_masked_argmax_and_the_cold_limit():
    rng = np.random.default_rng(6)
    B, R, V_d = 4, 3, 200
    zd = rng.normal(0, 3, (B, R, V_d)).astype(np.float32)
    mapped = rng.random(V_d) < 0.4
    id_map = np.where(mapped, np.arange(V_d), -1).astype(np.int32)
    u = rng.random((B, R)).astype(np.float32)
    cold = oracle.draft(zd, id_map, np.zeros(B, np.float32), u)
    want = np.where(mapped, zd, -np.inf).argmax(axis=2)
    np.testing.assert_array_equal(cold["draft_ids"], want)
    np.testing.assert_array_equal(cold["q_draft"], 1.0)
    nearly = oracle.draft(zd, id_map, np.full(B, 1e-3, np.float32), np.minimum(u, 0.999).astype(np.float32))
    np.testing.assert_array_equal(nearly["draft_ids"], want)           # gaps >> 1e-3 with these logits
    # ties: the lowest id wins, ids outside the intersection do not count
    z = np.zeros((1, 1, 10), np.float32)
    z[0, 0, [1, 4, 7]] = 5.0
    m = np.arange(10, dtype=np.int32)
    m[1] = -1
    assert oracle.draft(z, m, [0.0], [[0.3]])["draft_ids"][0, 0] == 4


def test_drawn_ids_are_always_accepted_when_the_target_equals_qprime():
    """Algorithm 5 run with p = q' accepts every draft: the drafting oracle feeds the verification oracle."""
    rng = np.random.default_rng(7)
    B, K, V_d = 5, 4, 120
    zd = rng.normal(0, 2, (B, K, V_d)).astype(np.float32)
    mapped = rng.random(V_d) < 0.5
    V_t = int(mapped.sum())
    id_map = np.full(V_d, -1, np.int32)
    id_map[mapped] = rng.permutation(V_t)
    inv = np.empty(V_t, np.int64)
    inv[id_map[mapped]] = np.flatnonzero(mapped)
    tau = np.array([0.7, 1.0, 1.0, 1.3, 0.9], np.float32)
    u = rng.integers(0, (1 << 24) - 8, (B, K + 1)).astype(np.float32) / np.float32(1 << 24)
    d = oracle.draft(zd, id_map, tau, u[:, :K])
    zt = np.ascontiguousarray(np.concatenate([zd[:, :, inv], zd[:, :1, inv]], axis=1))   # p_j = q'_j carried to target ids
    v = oracle.verify(zt, zd, id_map, d["draft_ids"], tau, u)
    np.testing.assert_array_equal(v["accepted"], K)
    np.testing.assert_allclose(v["q_draft"], d["q_draft"], rtol=0, atol=1e-15)
    np.testing.assert_allclose(v["thr"], 1.0, atol=1e-12)


def test_no_id_when_nothing_can_be_drawn():
    zd = np.random.default_rng(8).normal(0, 1, (3, 2, 40)).astype(np.float32)
    u = np.full((3, 2), 0.5, np.float32)
    empty = oracle.draft(zd, np.full(40, -1, np.int32), [1.0, 0.0, 0.5], u)
    np.testing.assert_array_equal(empty["draft_ids"], -1)
    assert (empty["flags"] & oracle.FLAG_FALLBACK).all()
    m = np.arange(40, dtype=np.int32)
    bad = oracle.draft(zd, m, [-1.0, np.nan, np.inf], u)
    np.testing.assert_array_equal(bad["draft_ids"], -1)
    assert (bad["flags"] & oracle.FLAG_BAD_TEMPERATURE).all()
    zd[1, 1, 3] = np.nan
    nf = oracle.draft(zd, m, [1.0, 1.0, 1.0], u)
    assert nf["flags"][1] & oracle.FLAG_NONFINITE and nf["draft_ids"][1, 1] == -1
    assert nf["flags"][0] == 0 and nf["flags"][2] == 0 and (nf["draft_ids"][[0, 2]] >= 0).all()


def test_bf16_strides_threads_and_probe():
    rng = np.random.default_rng(9)
    B, R, V_d = 7, 3, 500
    big = wl.f32_to_bf16_bits(rng.normal(0, 2, (B, R + 2, V_d + 11)).astype(np.float32))
    zd = big[:, 1:R + 1, 5:5 + V_d]                                    # strided view, odd offsets
    id_map = np.where(rng.random(V_d) < 0.6, np.arange(V_d), -1).astype(np.int32)
    tau = rng.choice([0.0, 0.5, 1.0], B).astype(np.float32)
    u = rng.random((B, R)).astype(np.float32)
    a = oracle.draft(zd, id_map, tau, u)
    b = oracle.draft(np.ascontiguousarray(zd), id_map, tau, u, threads=4)
    for k in a:
        np.testing.assert_array_equal(a[k], b[k])
    wide = oracle.draft(wl.bf16_bits_to_f32(np.ascontiguousarray(zd)), id_map, tau, u)
    np.testing.assert_array_equal(a["draft_ids"], wide["draft_ids"])   # bf16 widens exactly
    pr = oracle.draft(zd, id_map, tau, u, probe_id=a["draft_ids"])
    sampled = tau > 0
    np.testing.assert_allclose(pr["probe_lo"][sampled], a["cdf_lo"][sampled], atol=1e-15)
    np.testing.assert_allclose(pr["probe_hi"][sampled], a["cdf_hi"][sampled], atol=1e-15)
    np.testing.assert_allclose(pr["probe_w"][sampled], a["q_draft"][sampled], rtol=1e-12)


def test_the_chi_square_pin_catches_a_drafter_that_forgets_the_intersection():
    """Sensitivity of the pin above: ids drawn from q (no renormalisation onto the intersection) fail it."""
    rng = np.random.default_rng(21)
    V_d, N, tau = 12, 400_000, 1.0
    z = rng.normal(0, 1.5, V_d).astype(np.float32)
    mapped = np.zeros(V_d, bool)
    mapped[rng.choice(V_d, 7, replace=False)] = True
    want = masked_softmax(z, mapped, tau)
    q = np.exp((z.astype(np.float64) - z.max()) / tau)
    q /= q.sum()
    wrong = rng.choice(V_d, N, p=q)                                   # a sampler that ignores the mask
    kept = wrong[mapped[wrong]]                                       # even after dropping the ids outside it ...
    counts = np.bincount(kept, minlength=V_d)
    n = len(kept)
    chi2 = ((counts[mapped] - n * want[mapped]) ** 2 / (n * want[mapped])).sum()
    assert stats.chi2.sf(chi2, mapped.sum() - 1) > 1e-4                # ... the conditional law is q' (rejection sampling),
    assert (~mapped[wrong]).mean() > 0.05                             # but a share of the draws lies outside T: the pin's
    # first assertion (every id inside the intersection) is what such a drafter fails.
    off_by_one = np.searchsorted(np.cumsum(want), rng.random(N), side="left") + 1      # a CDF walk shifted by one id
    counts = np.bincount(np.clip(off_by_one, 0, V_d - 1), minlength=V_d)
    keep = want > 0
    chi2 = ((counts[keep] - N * want[keep]) ** 2 / (N * want[keep])).sum()
    assert stats.chi2.sf(chi2, keep.sum() - 1) < 1e-4                  # the chi-square rejects it
