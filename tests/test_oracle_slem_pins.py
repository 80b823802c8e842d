"""Pins of the exact-match verification oracle (Algorithm 2: sample t'_j from each of the m+1 target
rows, accept the re-tokenised drafts up to the first mismatch, emit t'_j there) against what the
paper and the mathematics fix."""
import itertools

import numpy as np
import pytest
from scipy import stats

import oracle
from paper_2502_05202_b200 import workload as wl


def softmax(z, tau):
    z = np.asarray(z, np.float64)
    e = np.exp((z - z.max()) / tau)
    return e / e.sum()


def uniforms(rng, shape):
    return rng.integers(0, 1 << 24, shape).astype(np.float32) / np.float32(1 << 24)


def test_sampled_tokens_follow_the_target_softmax_chi_square():
    """Every t'_j is a draw from p_j whatever the candidates are (that is why Algorithm 2 is lossless)."""
    rng = np.random.default_rng(1)
    V, M, N = 11, 2, 300_000
    z = rng.normal(0, 1.5, (M + 1, V)).astype(np.float32)
    tau = float(np.float32(0.8))
    zt = np.broadcast_to(z, (N, M + 1, V))
    out = oracle.slem(zt, rng.integers(0, V, (N, M)), np.full(N, tau, np.float32), uniforms(rng, (N, M + 1)), threads=4)
    for j in range(M + 1):
        want = softmax(z[j], tau)
        counts = np.bincount(out["sampled"][:, j], minlength=V)
        chi2 = ((counts - N * want) ** 2 / (N * want)).sum()
        assert stats.chi2.sf(chi2, V - 1) > 1e-4, (j, chi2)


def test_acceptance_is_a_run_of_matches_with_probability_p_of_the_candidate():
    """P(accept position j | reached) = p_j(t_j): the closed form of exact matching."""
    rng = np.random.default_rng(2)
    V, M, N = 6, 3, 400_000
    z = rng.normal(0, 1.0, (M + 1, V)).astype(np.float32)
    cand = np.array([2, 0, 5])
    zt = np.broadcast_to(z, (N, M + 1, V))
    out = oracle.slem(zt, np.broadcast_to(cand, (N, M)), np.ones(N, np.float32), uniforms(rng, (N, M + 1)), threads=4)
    pm = [softmax(z[j], 1.0)[cand[j]] for j in range(M)]
    want = [1 - pm[0], pm[0] * (1 - pm[1]), pm[0] * pm[1] * (1 - pm[2]), pm[0] * pm[1] * pm[2]]
    counts = np.bincount(out["accepted"], minlength=M + 1)
    chi2 = ((counts - N * np.array(want)) ** 2 / (N * np.array(want))).sum()
    assert stats.chi2.sf(chi2, M) > 1e-4, (counts / N, want)
    # the emitted token is t'_n: never the rejected candidate, and distributed as p_n given a mismatch
    n = out["accepted"]
    rej = n < M
    assert (out["next_token"][rej] != cand[n[rej]]).all()
    at0 = out["next_token"][n == 0]
    p0 = softmax(z[0], 1.0).copy()
    p0[cand[0]] = 0
    p0 /= p0.sum()
    c0 = np.bincount(at0, minlength=V)
    keep = p0 > 0
    chi2 = ((c0[keep] - len(at0) * p0[keep]) ** 2 / (len(at0) * p0[keep])).sum()
    assert stats.chi2.sf(chi2, keep.sum() - 1) > 1e-4


def test_each_draw_is_numpys_cumulative_sum_search():
    rng = np.random.default_rng(3)
    B, M, V = 5, 4, 257
    zt = rng.normal(0, 2, (B, M + 1, V)).astype(np.float32)
    tau = np.array([0.5, 0.8, 1.0, 1.0, 1.7], np.float32)
    u = uniforms(rng, (B, M + 1))
    out = oracle.slem(zt, np.zeros((B, M), np.int32), tau, u, lengths=None)
    # candidates of all zeros: force the comparison of every row by reading `sampled`
    full = oracle.slem(zt, out["sampled"][:, :M], tau, u)
    np.testing.assert_array_equal(full["accepted"], M)                         # its own samples always match
    np.testing.assert_array_equal(full["next_token"], full["sampled"][:, M])   # ... and the bonus token is t'_{m+1}
    for b in range(B):
        for j in range(M + 1):
            p = softmax(zt[b, j], float(tau[b]))
            c = np.cumsum(p)
            want = int(np.searchsorted(c, float(u[b, j]) * c[-1], side="right"))
            assert full["sampled"][b, j] == want or np.min(np.abs(c / c[-1] - float(u[b, j]))) < 1e-12


def test_brute_force_over_all_candidate_strings():
    """V = 3, M = 2: for every candidate string, n and the token follow from the sampled t' by definition."""
    rng = np.random.default_rng(4)
    V, M = 3, 2
    zt = rng.normal(0, 1, (1, M + 1, V)).astype(np.float32)
    for u in uniforms(rng, (20, M + 1)):
        base = oracle.slem(zt, [[0, 0]], [1.0], u[None])
        tp = base["sampled"][0]
        for cand in itertools.product(range(V), repeat=M):
            out = oracle.slem(zt, [list(cand)], [1.0], u[None])
            n = 0
            while n < M and tp[n] == cand[n]:
                n += 1
            assert out["accepted"][0] == n and out["next_token"][0] == tp[n]


def test_temperature_zero_agrees_with_tli_verification_under_an_identity_map():
    """Exact matching at tau = 0 is what the token-level oracle does at tau = 0 when T = D."""
    rng = np.random.default_rng(5)
    B, M, V = 8, 5, 64
    zt = rng.normal(0, 2, (B, M + 1, V)).astype(np.float32)
    best = zt.argmax(axis=2)
    cand = best[:, :M].copy()
    for b in range(B):
        if b % 2:
            cand[b, b % M] = (cand[b, b % M] + 1) % V                            # plant a mismatch
    tau = np.zeros(B, np.float32)
    u = uniforms(rng, (B, M + 1))
    a = oracle.slem(zt, cand, tau, u)
    v = oracle.verify(zt, np.zeros((B, M, V), np.float32), np.arange(V, dtype=np.int32), cand, tau, u)
    np.testing.assert_array_equal(a["accepted"], v["accepted"])
    np.testing.assert_array_equal(a["next_token"], v["next_token"])
    np.testing.assert_array_equal(a["sampled"], best)
    zt[0, 0, [3, 9]] = zt[0, 0].max() + 1                                        # a tie: the lowest id
    assert oracle.slem(zt, cand, tau, u)["sampled"][0, 0] == 3


def test_ragged_lengths_flags_bf16_and_threads():
    rng = np.random.default_rng(6)
    B, M, V = 6, 4, 300
    bits = wl.f32_to_bf16_bits(rng.normal(0, 2, (B, M + 1, V)).astype(np.float32))
    tau = rng.choice([0.0, 0.7, 1.0], B).astype(np.float32)
    u = uniforms(rng, (B, M + 1))
    first = oracle.slem(bits, np.zeros((B, M), np.int32), tau, u)["sampled"]
    lengths = np.array([0, 1, 2, 3, 4, 4], np.int32)
    out = oracle.slem(bits, first[:, :M], tau, u, lengths=lengths)
    np.testing.assert_array_equal(out["accepted"], lengths)                    # own samples match up to m_b
    for b in range(B):
        assert out["next_token"][b] == first[b, lengths[b]]
        assert (out["sampled"][b, lengths[b] + 1:] == -1).all() and (out["sampled"][b, :lengths[b] + 1] >= 0).all()
    wide = oracle.slem(wl.bf16_bits_to_f32(bits), first[:, :M], tau, u, lengths=lengths, threads=3)
    for k in ("sampled", "accepted", "next_token"):
        np.testing.assert_array_equal(out[k], wide[k])
    bad = oracle.slem(bits, first[:, :M], [-1, np.nan, np.inf, 1, 1, 1], u)
    assert (bad["flags"][:3] == oracle.FLAG_BAD_TEMPERATURE).all() and (bad["flags"][3:] == 0).all()
    assert (bad["accepted"][:3] == 0).all() and (bad["sampled"][:3] == -1).all()
    z = wl.bf16_bits_to_f32(bits).copy()
    z[4, 2, 17] = np.nan
    nf = oracle.slem(z, first[:, :M], np.ones(B, np.float32), u, lengths=np.array([4, 4, 4, 4, 4, 1], np.int32))
    assert nf["flags"][4] == oracle.FLAG_NONFINITE and nf["accepted"][4] == 0 and nf["next_token"][4] == 0
    z[5, 3, 0] = np.inf                                                       # beyond m_5 = 1: not sampled, not seen
    nf = oracle.slem(z, first[:, :M], np.ones(B, np.float32), u, lengths=np.array([4, 4, 4, 4, 4, 1], np.int32))
    assert nf["flags"][5] == 0
