"""Pins for the fp64 oracle: every check here compares it with something the
paper or the mathematics fixes, computed without the oracle's own formulas
(scipy's softmax, numpy's cumsum/searchsorted, exact enumeration, chi-square).
"""
import os

import numpy as np
import pytest
import scipy.special
import scipy.stats

import oracle
from paper_2502_05202_b200 import workload as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
ONE_M = np.float32(1.0 - 2.0 ** -24)   # the largest uniform the ABI allows


def softmax(z, tau):
    return scipy.special.softmax(np.asarray(z, np.float64) / tau, axis=-1)


def random_map(rng, V_d, V_t, n):
    m = np.full(V_d, -1, np.int32)
    xs = rng.permutation(V_d)[:n]
    ts = rng.permutation(V_t)[:n]
    m[xs] = ts
    return m


def qprime_def(q, id_map):
    """Algorithm 4: renormalise q on the intersection (computed here by definition)."""
    inside = id_map >= 0
    qp = np.where(inside, q, 0.0)
    return qp / qp.sum()


def bcast(z, B):
    """[rows, V] logits -> [B, rows, V] view with batch stride 0."""
    z = np.ascontiguousarray(z)
    return np.lib.stride_tricks.as_strided(z, (B,) + z.shape, (0,) + z.strides)


# --------------------------------------------------------------------------
# Algorithm 4: the renormalisation
# --------------------------------------------------------------------------

def test_qprime_worked_example_from_paper():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "qprime_worked_example.txt"))
            if l.strip() and not l.startswith("#")]
    in_T = [int(r[1]) for r in rows]
    q = np.array([float(r[2]) for r in rows])
    qp_expected = np.array([float(r[3]) for r in rows])
    V_d = len(rows)
    id_map = np.full(V_d, -1, np.int32)
    t = 0
    for x in range(V_d):
        if in_T[x]:
            id_map[x] = t
            t += 1
    V_t = t
    zd = np.log(q).astype(np.float32)[None, None, :]          # softmax(log q) = q
    zt = np.zeros((1, 2, V_t), np.float32)
    tau = np.ones(1, np.float32)
    p, qT = oracle.distributions(zt, zd, id_map, tau, 0, 0)
    np.testing.assert_allclose(qT, qp_expected[:V_t], atol=1e-7)   # float32 log(1/3) inputs
    np.testing.assert_allclose(p, [0.5, 0.5], atol=1e-15)
    # the same through the verifier: q'(d) of each draft, and the draft outside T is rejected
    for x in range(V_d):
        out = oracle.verify(zt, zd, id_map, [[x]], tau, [[0.0, 0.0]])
        if in_T[x]:
            assert abs(out["q_draft"][0, 0] - qp_expected[x]) < 1e-7
            assert out["thr"][0, 0] == pytest.approx(1.0)      # p = 1/2 = q'
            assert out["accepted"][0] == 1
        else:
            assert out["thr"][0, 0] == 0.0 and out["accepted"][0] == 0
            assert out["flags"][0] & oracle.FLAG_DRAFT_UNMAPPED


@pytest.mark.parametrize("seed", range(6))
def test_qprime_matches_definition(seed):
    rng = np.random.default_rng(seed)
    V_t, V_d = int(rng.integers(2, 9)), int(rng.integers(2, 9))
    n = int(rng.integers(1, min(V_t, V_d) + 1))
    id_map = random_map(rng, V_d, V_t, n)
    tau = np.array([rng.choice([0.5, 1.0, 1.7])], np.float32)
    zt = rng.normal(0, 2, (1, 2, V_t)).astype(np.float32)
    zd = rng.normal(0, 2, (1, 1, V_d)).astype(np.float32)
    p, qT = oracle.distributions(zt, zd, id_map, tau, 0, 0)
    np.testing.assert_allclose(p, softmax(zt[0, 0], float(tau[0])), atol=1e-14)
    qp = qprime_def(softmax(zd[0, 0], float(tau[0])), id_map)
    expect = np.zeros(V_t)
    expect[id_map[id_map >= 0]] = qp[id_map >= 0]
    np.testing.assert_allclose(qT, expect, atol=1e-14)
    assert abs(qT.sum() - 1.0) < 1e-13


# --------------------------------------------------------------------------
# Algorithm 5 with (p, q'): exact enumeration on tiny vocabularies
# --------------------------------------------------------------------------

def enumerate_output_distribution(zt, zd, id_map, tau):
    """P(first emitted token = t) with the draft x ~ q', from the oracle's
    thresholds and residual weights; K = 1."""
    V_t, V_d = zt.shape[-1], zd.shape[-1]
    tau_f = float(tau)
    qp = qprime_def(softmax(zd, tau_f), id_map) if (id_map >= 0).any() else np.zeros(V_d)
    zt2 = np.stack([zt, zt]).astype(np.float32)                # K+1 = 2 rows
    zd2 = zd.astype(np.float32)[None, :]
    out_dist = np.zeros(V_t)
    alpha = 0.0
    for x in range(V_d):
        if id_map[x] < 0:
            continue
        # threshold of draft x
        o = oracle.verify(zt2[None], zd2[None], id_map, [[x]], [tau], [[0.0, 0.0]])
        a = o["thr"][0, 0]
        alpha += qp[x] * a
        out_dist[id_map[x]] += qp[x] * a
        if a < 1.0:
            # force a rejection and read the residual weight of every target token
            B = V_t
            o = oracle.verify(bcast(zt2, B), bcast(zd2, B), id_map, np.full((B, 1), x, np.int32),
                              np.full(B, tau, np.float32), np.tile([ONE_M, 0.5], (B, 1)).astype(np.float32),
                              probe_token=np.arange(V_t, dtype=np.int32))
            assert (o["accepted"] == 0).all()
            r = o["probe_w"]
            assert abs(r.sum() - 1.0) < 1e-12
            out_dist += qp[x] * (1.0 - a) * r
    return out_dist, alpha


@pytest.mark.parametrize("seed", range(12))
def test_losslessness_by_enumeration(seed):
    """Theorem 4.1: the emitted token is distributed as p (exact, V <= 8)."""
    rng = np.random.default_rng(100 + seed)
    V_t, V_d = int(rng.integers(2, 9)), int(rng.integers(2, 9))
    n = int(rng.integers(1, min(V_t, V_d) + 1))
    id_map = random_map(rng, V_d, V_t, n)
    tau = float(np.float32(rng.choice([0.5, 1.0, 1.7])))
    zt = rng.normal(0, 1.5, V_t).astype(np.float32)
    zd = rng.normal(0, 1.5, V_d).astype(np.float32)
    dist, alpha = enumerate_output_distribution(zt, zd, id_map, tau)
    p = softmax(zt, tau)
    np.testing.assert_allclose(dist, p, atol=1e-12)
    # expected acceptance rate (table of expected acceptance rates, TLI row) and Theorem 4.1's ordering
    q = softmax(zd, tau)
    qp = qprime_def(q, id_map)
    inside = id_map >= 0
    alpha_tli = np.minimum(p[id_map[inside]], qp[inside]).sum()
    alpha_union = np.minimum(p[id_map[inside]], q[inside]).sum()
    assert abs(alpha - alpha_tli) < 1e-12
    assert alpha_union <= alpha_tli + 1e-15


@pytest.mark.parametrize("case", ["T=ab,D=b", "T=a,D=ab", "T=ab,D=abc"])
def test_subset_vocabularies_stay_lossless(case):
    """The motivating examples' subset vocabularies."""
    id_map = {"T=ab,D=b": np.array([1], np.int32),
              "T=a,D=ab": np.array([0, -1], np.int32),
              "T=ab,D=abc": np.array([0, 1, -1], np.int32)}[case]
    V_t = {"T=ab,D=b": 2, "T=a,D=ab": 1, "T=ab,D=abc": 2}[case]
    rng = np.random.default_rng(5)
    zt = rng.normal(0, 1, V_t).astype(np.float32)
    zd = rng.normal(0, 1, len(id_map)).astype(np.float32)
    dist, _ = enumerate_output_distribution(zt, zd, id_map, 1.0)
    np.testing.assert_allclose(dist, softmax(zt, 1.0), atol=1e-12)


def test_residual_mass_identity():
    """sum_t max(0, p - q'_T) = 1 - sum_{T cap D} min(p, q') (the denominator of r)."""
    rng = np.random.default_rng(3)
    for _ in range(10):
        V_t, V_d = int(rng.integers(3, 40)), int(rng.integers(3, 40))
        id_map = random_map(rng, V_d, V_t, int(rng.integers(1, min(V_t, V_d) + 1)))
        tau = float(np.float32(rng.choice([0.6, 1.0])))
        zt = rng.normal(0, 2, (1, 2, V_t)).astype(np.float32)
        zd = rng.normal(0, 2, (1, 1, V_d)).astype(np.float32)
        x = int(np.flatnonzero(id_map >= 0)[0])
        o = oracle.verify(zt, zd, id_map, [[x]], [tau], [[ONE_M, 0.3]])
        p = softmax(zt[0, 0], tau)
        qp = qprime_def(softmax(zd[0, 0], tau), id_map)
        inside = id_map >= 0
        expect = 1.0 - np.minimum(p[id_map[inside]], qp[inside]).sum()
        if o["accepted"][0] == 0:
            assert abs(o["total"][0] - expect) < 1e-12


# --------------------------------------------------------------------------
# inverse CDF
# --------------------------------------------------------------------------

@pytest.mark.parametrize("seed", range(4))
def test_inverse_cdf_boundaries(seed):
    """Sweep v over a fine grid: the token changes where numpy's cumulative sum says."""
    rng = np.random.default_rng(200 + seed)
    V_t, V_d = 7, 6
    id_map = random_map(rng, V_d, V_t, 4)
    tau = 1.0
    zt = rng.normal(0, 1.5, (2, V_t)).astype(np.float32)
    zd = rng.normal(0, 1.5, (1, V_d)).astype(np.float32)
    x = int(np.flatnonzero(id_map >= 0)[0])
    G = 4096
    v = (np.arange(G) / G).astype(np.float32)
    p0 = softmax(zt[0], tau)
    qp = qprime_def(softmax(zd[0], tau), id_map)
    qT = np.zeros(V_t)
    qT[id_map[id_map >= 0]] = qp[id_map >= 0]
    for reject in (True, False):
        u = np.stack([np.full(G, ONE_M if reject else 0.0, np.float32), v], axis=1)
        o = oracle.verify(bcast(zt, G), bcast(zd, G), id_map, np.full((G, 1), x, np.int32),
                          np.full(G, tau, np.float32), u)
        if reject:
            if o["thr"][0, 0] >= 1.0:
                continue
            w = np.maximum(0.0, p0 - qT)
            assert (o["accepted"] == 0).all()
        else:
            if o["thr"][0, 0] <= 0.0:
                continue
            w = softmax(zt[1], tau)            # bonus row
            assert (o["accepted"] == 1).all()
        C = np.cumsum(w) / w.sum()
        expect = np.searchsorted(C, v.astype(np.float64), side="right")
        near = np.min(np.abs(C[None, :] - v[:, None].astype(np.float64)), axis=1) < 1e-9
        got = o["next_token"]
        assert (got[~near] == expect[~near]).all()
        assert (w[got] > 0).all()                  # zero-weight ids are never returned
        np.testing.assert_allclose(o["cdf_hi"], C[got], atol=1e-12)


# --------------------------------------------------------------------------
# Reduction to single-vocabulary speculative decoding (Algorithm 5)
# --------------------------------------------------------------------------

def single_vocab_sd(zt, zq, d, tau, u):
    """Algorithm 5 for one sequence with a shared vocabulary, written with numpy only."""
    K = len(d)
    n = K
    for j in range(K):
        p = softmax(zt[j], tau)
        q = softmax(zq[j], tau)
        if not (u[j] < min(1.0, p[d[j]] / q[d[j]])):
            n = j
            break
    p = softmax(zt[n], tau)
    if n < K:
        q = softmax(zq[n], tau)
        r = p - np.minimum(p, q)
        r = r / r.sum()
    else:
        r = p
    t = int(np.searchsorted(np.cumsum(r), float(u[K]), side="right"))
    return n, min(t, len(r) - 1)


def test_identity_map_reduces_to_standard_sd():
    rng = np.random.default_rng(11)
    V, K, B = 23, 4, 300
    id_map = np.arange(V, dtype=np.int32)
    zt = rng.normal(0, 2, (B, K + 1, V)).astype(np.float32)
    zq = (zt[:, :K] + rng.normal(0, 0.7, (B, K, V))).astype(np.float32)
    tau = rng.choice([0.7, 1.0], B).astype(np.float32)
    d = rng.integers(0, V, (B, K)).astype(np.int32)
    u = (rng.integers(0, 1 << 24, (B, K + 1)) * 2.0 ** -24).astype(np.float32)
    o = oracle.verify(zt, zq, id_map, d, tau, u)
    for b in range(B):
        n, t = single_vocab_sd(zt[b], zq[b], d[b], float(tau[b]), u[b])
        assert (o["accepted"][b], o["next_token"][b]) == (n, t)


def test_q_equals_p_accepts_everything():
    """alpha_SD = sum min(p, p) = 1 when the drafter equals the target."""
    rng = np.random.default_rng(12)
    V, K, B = 31, 5, 50
    zt = rng.normal(0, 3, (B, K + 1, V)).astype(np.float32)
    d = rng.integers(0, V, (B, K)).astype(np.int32)
    u = np.full((B, K + 1), ONE_M, np.float32)
    o = oracle.verify(zt, zt[:, :K].copy(), np.arange(V, dtype=np.int32), d, np.ones(B, np.float32), u)
    assert (o["accepted"] == K).all()
    np.testing.assert_allclose(o["thr"], 1.0, atol=1e-12)


def test_disjoint_vocabularies_reject_everything():
    """Empty intersection: acceptance rate zero, the emitted token still follows p."""
    rng = np.random.default_rng(13)
    V_t, V_d, K, B = 9, 6, 3, 200
    id_map = np.full(V_d, -1, np.int32)
    zt = rng.normal(0, 1, (B, K + 1, V_t)).astype(np.float32)
    zd = rng.normal(0, 1, (B, K, V_d)).astype(np.float32)
    d = rng.integers(0, V_d, (B, K)).astype(np.int32)
    u = (rng.integers(0, 1 << 24, (B, K + 1)) * 2.0 ** -24).astype(np.float32)
    o = oracle.verify(zt, zd, id_map, d, np.ones(B, np.float32), u)
    assert (o["accepted"] == 0).all()
    assert (o["flags"] & oracle.FLAG_DRAFT_UNMAPPED).all()
    for b in range(B):
        C = np.cumsum(softmax(zt[b, 0], 1.0))
        assert o["next_token"][b] == np.searchsorted(C, float(u[b, K]), side="right")


def test_strict_threshold_comparison():
    """accept iff u < min(1, p/q'): thr = 1/2 exactly when p = (1/2, 1/2) and q' = (1)."""
    zt = np.zeros((1, 2, 2), np.float32)
    zd = np.zeros((1, 1, 1), np.float32)
    id_map = np.array([0], np.int32)
    for u0, expect in ((0.5, 0), (0.5 - 2.0 ** -24, 1), (0.0, 1)):
        o = oracle.verify(zt, zd, id_map, [[0]], [1.0], [[u0, 0.25]])
        assert o["thr"][0, 0] == 0.5
        assert o["accepted"][0] == expect
    # rejected: residual is max(0, p - q'_T) = (0, 1/2) -> always token 1
    o = oracle.verify(zt, zd, id_map, [[0]], [1.0], [[0.75, 0.0]])
    assert o["accepted"][0] == 0 and o["next_token"][0] == 1 and o["total"][0] == 0.5


# --------------------------------------------------------------------------
# Losslessness by chi-square
# --------------------------------------------------------------------------

@pytest.mark.parametrize("K,V_t,V_d,seed", [(1, 6, 8, 0), (2, 12, 9, 1), (3, 16, 16, 2)])
def test_losslessness_chi_square(K, V_t, V_d, seed):
    """Conditioned on reaching position j, the token emitted there follows p_j; >= 1e6 trials."""
    rng = np.random.default_rng(300 + seed)
    N = 1_000_000
    id_map = random_map(rng, V_d, V_t, min(V_t, V_d) - 2)
    tau = float(np.float32(0.9))
    zt = rng.normal(0, 1.0, (K + 1, V_t)).astype(np.float32)
    zd = rng.normal(0, 1.0, (K, V_d)).astype(np.float32)
    d = np.empty((N, K), np.int32)
    for j in range(K):
        qp = qprime_def(softmax(zd[j], tau), id_map)
        d[:, j] = rng.choice(V_d, size=N, p=qp)
    u = (rng.integers(0, 1 << 24, (N, K + 1)) * 2.0 ** -24).astype(np.float32)
    o = oracle.verify(bcast(zt, N), bcast(zd, N), id_map, d, np.full(N, tau, np.float32), u, threads=8)
    n, nxt = o["accepted"], o["next_token"]
    for j in range(K + 1):
        reached = n >= j
        emitted = np.where(n[reached] > j, id_map[d[reached, min(j, K - 1)]], nxt[reached])
        counts = np.bincount(emitted, minlength=V_t).astype(np.float64)
        expected = softmax(zt[j], tau) * reached.sum()
        assert expected.min() > 5
        pval = scipy.stats.chisquare(counts, expected).pvalue
        assert pval > 1e-4, (j, pval)


# --------------------------------------------------------------------------
# temperature 0
# --------------------------------------------------------------------------

def test_greedy_is_the_low_temperature_limit():
    rng = np.random.default_rng(21)
    V_t, V_d, K, B = 40, 37, 4, 200
    id_map = random_map(rng, V_d, V_t, 25)
    # well separated logits: distinct multiples of 0.5
    zt = np.stack([np.stack([rng.permutation(V_t) for _ in range(K + 1)]) for _ in range(B)]).astype(np.float32) * 0.5
    zd = np.stack([np.stack([rng.permutation(V_d) for _ in range(K)]) for _ in range(B)]).astype(np.float32) * 0.5
    # half the rows: drafter's best mapped token is the target's arg-max
    for b in range(0, B, 2):
        for j in range(K):
            xs = np.flatnonzero(id_map >= 0)
            xbest = xs[np.argmax(zd[b, j, xs])]
            t = id_map[xbest]
            a = np.argmax(zt[b, j])
            zt[b, j, [t, a]] = zt[b, j, [a, t]]
    masked = np.where(id_map[None, None, :] >= 0, zd, -np.inf)
    d = np.argmax(masked, axis=2).astype(np.int32)       # what a temperature-0 TLI drafter emits
    u = (rng.integers(1, 1 << 24, (B, K + 1)) * 2.0 ** -24).astype(np.float32)
    cold = oracle.verify(zt, zd, id_map, d, np.full(B, 0.01, np.float32), u)
    zero = oracle.verify(zt, zd, id_map, d, np.zeros(B, np.float32), u)
    assert (cold["accepted"] == zero["accepted"]).all()
    assert (cold["next_token"] == zero["next_token"]).all()
    assert zero["accepted"].max() == K and zero["accepted"].min() == 0


def test_greedy_ties_take_the_lowest_index():
    V_t = 10
    zt = np.zeros((1, 3, V_t), np.float32)
    zt[0, 0, [3, 7]] = 2.0          # tie -> 3
    zt[0, 1, [9, 4]] = 1.5          # tie -> 4
    zt[0, 2, :] = -1.0              # all equal -> 0
    id_map = np.array([3, 7, 4, 9, -1], np.int32)
    zd = np.zeros((1, 2, 5), np.float32)
    tau = np.zeros(1, np.float32)
    u = np.zeros((1, 3), np.float32)
    assert_out = lambda d, n, t: (
        lambda o: (o["accepted"][0], o["next_token"][0]) == (n, t))(oracle.verify(zt, zd, id_map, [d], tau, u))
    assert assert_out([0, 2], 2, 0)     # both match the lowest-index arg-max; bonus row all equal -> 0
    assert assert_out([1, 2], 0, 3)     # maps to 7, the other maximiser: not a match
    assert assert_out([0, 3], 1, 4)
    assert assert_out([4, 2], 0, 3)     # outside the intersection


# --------------------------------------------------------------------------
# storage formats, strides, harness hooks, flags
# --------------------------------------------------------------------------

def test_bf16_inputs_are_widened_exactly():
    rng = np.random.default_rng(31)
    V_t, V_d, K, B = 50, 45, 3, 20
    id_map = random_map(rng, V_d, V_t, 30)
    zt = rng.normal(0, 2, (B, K + 1, V_t)).astype(np.float32)
    zd = rng.normal(0, 2, (B, K, V_d)).astype(np.float32)
    zt_b = (zt.view(np.uint32) >> 16).astype(np.uint16)        # truncation: any bf16 pattern will do
    zd_b = (zd.view(np.uint32) >> 16).astype(np.uint16)
    zt_f = (zt_b.astype(np.uint32) << 16).view(np.float32)
    zd_f = (zd_b.astype(np.uint32) << 16).view(np.float32)
    d = rng.choice(np.flatnonzero(id_map >= 0), (B, K)).astype(np.int32)
    u = (rng.integers(0, 1 << 24, (B, K + 1)) * 2.0 ** -24).astype(np.float32)
    tau = np.full(B, 0.8, np.float32)
    a = oracle.verify(zt_b, zd_b, id_map, d, tau, u)
    b = oracle.verify(zt_f, zd_f, id_map, d, tau, u)
    for k in a:
        np.testing.assert_array_equal(a[k], b[k])


def test_strided_batches_and_threads():
    rng = np.random.default_rng(32)
    V_t, V_d, K, B = 33, 29, 2, 16
    id_map = random_map(rng, V_d, V_t, 20)
    big_t = rng.normal(0, 2, (B, K + 3, V_t + 5)).astype(np.float32)
    big_d = rng.normal(0, 2, (B, K + 1, V_d + 3)).astype(np.float32)
    zt, zd = big_t[:, :K + 1, :V_t], big_d[:, :K, :V_d]
    d = rng.choice(np.flatnonzero(id_map >= 0), (B, K)).astype(np.int32)
    u = (rng.integers(0, 1 << 24, (B, K + 1)) * 2.0 ** -24).astype(np.float32)
    tau = np.ones(B, np.float32)
    a = oracle.verify(zt, zd, id_map, d, tau, u)
    b = oracle.verify(np.ascontiguousarray(zt), np.ascontiguousarray(zd), id_map, d, tau, u, threads=4)
    for k in a:
        np.testing.assert_array_equal(a[k], b[k])


def test_force_accept_and_flags():
    rng = np.random.default_rng(33)
    V_t, V_d, K = 12, 10, 3
    id_map = random_map(rng, V_d, V_t, 6)
    zt = rng.normal(0, 1, (1, K + 1, V_t)).astype(np.float32)
    zd = rng.normal(0, 1, (1, K, V_d)).astype(np.float32)
    xin = np.flatnonzero(id_map >= 0)
    xout = np.flatnonzero(id_map < 0)
    d = np.array([[xin[0], xin[1], xin[2]]], np.int32)
    u = np.array([[0.0, 0.0, 0.0, 0.5]], np.float32)
    o = oracle.verify(zt, zd, id_map, d, [1.0], u)
    assert o["accepted"][0] == K
    o = oracle.verify(zt, zd, id_map, d, [1.0], u, force_accept=[[-1, 0, -1]])
    assert o["accepted"][0] == 1
    o = oracle.verify(zt, zd, id_map, [[xin[0], xout[0], xin[1]]], [1.0], u)
    assert o["accepted"][0] == 1 and o["flags"][0] == oracle.FLAG_DRAFT_UNMAPPED
    o = oracle.verify(zt, zd, id_map, [[V_d, xin[0], xin[1]]], [1.0], u)
    assert o["accepted"][0] == 0 and o["flags"][0] & oracle.FLAG_DRAFT_RANGE
    o = oracle.verify(zt, zd, id_map, d, [-1.0], u)
    assert o["flags"][0] == oracle.FLAG_BAD_TEMPERATURE
    bad = id_map.copy()
    bad[xout[0]] = id_map[xin[0]]                    # two drafter ids on one target id
    with pytest.raises(RuntimeError):
        oracle.verify(zt, zd, bad, d, [1.0], u)


def test_enumeration_pin_catches_a_forgotten_renormalisation():
    """The enumeration pin is sensitive where it matters.  Feed the oracle drafter logits whose softmax is
    the *unnormalised* q restricted to the intersection (so that its q' is right), then read its
    thresholds and residual while the drafts are assumed to come from q instead of q': the identity
    sum_x q(x) [a 1{map x = t} + (1 - a) r(t)] = p(t) must fail, by the mass q puts outside T."""
    rng = np.random.default_rng(41)
    V_t, V_d = 6, 7
    id_map = random_map(rng, V_d, V_t, 4)
    zt = rng.normal(0, 1.5, V_t).astype(np.float32)
    zd = rng.normal(0, 1.5, V_d).astype(np.float32)
    p = softmax(zt, 1.0)
    q = softmax(zd, 1.0)
    inside = np.flatnonzero(id_map >= 0)
    thr = np.zeros(V_d)
    for x in inside:                                   # the oracle's acceptance probability of every draft
        o = oracle.verify(zt[None, None].repeat(2, 1), zd[None, None], id_map, np.array([[x]], np.int32),
                          np.ones(1, np.float32), np.zeros((1, 2), np.float32))
        thr[x] = o["thr"][0, 0]
    # the oracle's residual, read off its CDF for a draft it rejects
    x0 = inside[np.argmin(thr[inside])]
    assert thr[x0] < 1.0
    r = np.zeros(V_t)
    for t in range(V_t):
        o = oracle.verify(zt[None, None].repeat(2, 1), zd[None, None], id_map, np.array([[x0]], np.int32),
                          np.ones(1, np.float32), np.array([[0.999999, 0.5]], np.float32),
                          probe_token=np.array([t], np.int32))
        assert o["accepted"][0] == 0
        r[t] = o["probe_w"][0]
    assert abs(r.sum() - 1) < 1e-12
    def emitted(proposal):
        dist = np.zeros(V_t)
        np.add.at(dist, id_map[inside], proposal[inside] * thr[inside])
        return dist + (proposal[inside] * (1 - thr[inside])).sum() * r
    # NB: r is the residual of the one draft position, which is the same for every x (it depends on p, q' only)
    assert np.abs(emitted(qprime_def(q, id_map)) - p).max() < 1e-12      # drafts from q': lossless
    assert np.abs(emitted(q) - p).max() > 1e-3                           # drafts from q: not


def test_exactly_zero_residual_falls_back_to_the_target_distribution():
    """Identity map, all logits equal on a power-of-two vocabulary: p = q' = 2^-k and the mass on the
    intersection is 1, all exactly, so a rejected draft leaves a residual of exactly zero everywhere.
    Only a draft outside the vocabulary can be rejected there; the oracle must then flag the fall-back
    and draw from p, i.e. return floor(v * V)."""
    V = 16
    K = 2
    zt = np.zeros((5, K + 1, V), np.float32)
    zd = np.zeros((5, K, V), np.float32)
    id_map = np.arange(V, dtype=np.int32)
    draft = np.array([[V, 0], [-1, 3], [2, V + 5], [1, 2], [7, -9]], np.int32)
    u = np.array([[0.5, 0.5, 0.30], [0.1, 0.2, 0.99], [0.9, 0.1, 0.0625], [0.3, 0.3, 0.5], [0.999, 0.0, 0.124]], np.float32)
    o = oracle.verify(zt, zd, id_map, draft, np.ones(5, np.float32), u)
    assert list(o["accepted"]) == [0, 0, 1, 2, 1]
    expect_flags = [oracle.FLAG_DRAFT_RANGE | oracle.FLAG_FALLBACK] * 3 + [0, oracle.FLAG_DRAFT_RANGE | oracle.FLAG_FALLBACK]
    assert list(o["flags"]) == expect_flags
    assert list(o["next_token"]) == [int(np.floor(float(v) * V)) for v in u[:, K]]
    assert np.all(o["total"] == 1.0)                   # the sum of sixteen times 2^-4, exactly


def test_ragged_draft_counts_equal_truncated_batches():
    """draft_lengths[b] = m: the result is that of the same sequence given with K = m drafts (rows and
    uniforms beyond m dropped, the last uniform kept); m = 0 is one draw from target row 0."""
    cfg = wl.tiny_config(B=12, K=5, V_t=60, V_d=50, dtype=wl.F32, f_mapped=0.7, sigma_d=0.3,
                         temperatures=(0.0, 0.8, 1.0), seed=77)
    b = wl.make_batch(cfg)
    lengths = np.array([0, 1, 2, 3, 4, 5, 5, 3, 0, 2, 1, 4], np.int32)
    rag = oracle.verify(b["target_logits"], b["drafter_logits"], b["id_map"], b["draft_ids"], b["temperature"],
                        b["uniforms"], draft_lengths=lengths)
    full = oracle.verify(b["target_logits"], b["drafter_logits"], b["id_map"], b["draft_ids"], b["temperature"],
                         b["uniforms"])
    assert (rag["accepted"] <= lengths).all() and rag["accepted"].max() >= 2
    for i, m in enumerate(lengths):
        u = np.concatenate([b["uniforms"][i:i + 1, :m], b["uniforms"][i:i + 1, -1:]], axis=1)
        if m == 0:
            one = oracle.slem(b["target_logits"][i:i + 1, :1], np.zeros((1, 0), np.int32), b["temperature"][i:i + 1], u)
            assert rag["accepted"][i] == 0 and rag["next_token"][i] == one["next_token"][0]
            continue
        sub = oracle.verify(b["target_logits"][i:i + 1, :m + 1], b["drafter_logits"][i:i + 1, :m], b["id_map"],
                            b["draft_ids"][i:i + 1, :m], b["temperature"][i:i + 1], u)
        assert sub["accepted"][0] == rag["accepted"][i] and sub["next_token"][0] == rag["next_token"][i]
        np.testing.assert_array_equal(sub["thr"][0], rag["thr"][i, :m])
        assert (rag["thr"][i, m:] == 0).all() and (rag["q_draft"][i, m:] == 0).all()
        if m == cfg.K:
            assert rag["accepted"][i] == full["accepted"][i] and rag["next_token"][i] == full["next_token"][i]
