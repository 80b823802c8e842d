"""The paper's central claim checked on the GPU path itself: drafting from q' and verifying with
Algorithm 5 (token level), or exact matching (Algorithm 2), emits tokens distributed as the target
softmax -- chi-square over tens of thousands of sequences that share their logits and differ in
their uniforms.  (Parity with the oracle is tested elsewhere; this does not use the oracle.)"""
import numpy as np
import pytest
import torch
from scipy import stats

from paper_2502_05202_b200 import tli

pytestmark = pytest.mark.gpu


def softmax(z, tau):
    z = np.asarray(z, np.float64)
    e = np.exp((z - z.max()) / tau)
    return e / e.sum()


def uniforms(rng, shape):
    return torch.from_numpy(rng.integers(0, 1 << 24, shape).astype(np.float32) / np.float32(1 << 24)).cuda()


def chi2_ok(tokens, want, what):
    n = len(tokens)
    counts = np.bincount(tokens, minlength=len(want)).astype(np.float64)
    keep = want > 0
    assert counts[~keep].sum() == 0, what
    chi2 = ((counts[keep] - n * want[keep]) ** 2 / (n * want[keep])).sum()
    p = stats.chi2.sf(chi2, keep.sum() - 1)
    assert p > 1e-4, (what, chi2, p)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("tau", [1.0, 0.6])
def test_token_level_intersection_is_lossless_on_the_gpu(dtype, tau):
    rng = np.random.default_rng(11)
    V_t, V_d, K, B = 9, 11, 3, 21000                                        # B * K rows in one drafting call
    id_map = np.array([4, -1, 0, 7, -1, 2, 8, -1, 5, 1, -1], np.int32)       # T and D overlap in 7 tokens
    zt1 = torch.from_numpy(rng.normal(0, 1.2, (1, K + 1, V_t)).astype(np.float32)).to(dtype).cuda()
    zd1 = torch.from_numpy(rng.normal(0, 1.2, (1, K, V_d)).astype(np.float32)).to(dtype).cuda()
    zt, zd = zt1.expand(B, K + 1, V_t), zd1.expand(B, K, V_d)                 # stride 0 over the batch
    t = torch.full((B,), tau, dtype=torch.float32, device="cuda")
    v = tli.Verifier(V_t, V_d, id_map)
    d = v.draft(zd, t, uniforms(rng, (B, K)))
    out = v.verify(zt, zd, d["draft_ids"], t, uniforms(rng, (B, K + 1)))
    torch.cuda.synchronize()
    ids = d["draft_ids"].cpu().numpy()
    n = out["accepted"].cpu().numpy()
    nxt = out["next_token"].cpu().numpy()
    assert (out["row_status"].cpu().numpy() == 0).all() and (id_map[ids] >= 0).all()
    zt_h = zt1.float().cpu().numpy()[0]
    for j in range(K + 1):
        reached = n >= j                                                     # sequences that emit a token at position j
        if j < K:
            tok = np.where(n[reached] > j, id_map[ids[reached, j]], nxt[reached])
        else:
            tok = nxt[reached]
        assert reached.sum() > 300
        chi2_ok(tok, softmax(zt_h[j], tau), "position %d" % j)
    v.close()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_exact_matching_is_lossless_on_the_gpu(dtype):
    rng = np.random.default_rng(12)
    V_t, M, B, tau = 10, 2, 21000, 0.8
    zt1 = torch.from_numpy(rng.normal(0, 1.0, (1, M + 1, V_t)).astype(np.float32)).to(dtype).cuda()
    zt = zt1.expand(B, M + 1, V_t)
    cand_h = rng.integers(0, V_t, (B, M)).astype(np.int32)
    cand_h[:, 0] = np.argmax(zt1.float().cpu().numpy()[0, 0])                 # a likely first candidate: some runs continue
    t = torch.full((B,), tau, dtype=torch.float32, device="cuda")
    v = tli.Verifier(V_t, 4, np.full(4, -1, np.int32))
    out = v.slem(zt, torch.from_numpy(cand_h).cuda(), t, uniforms(rng, (B, M + 1)))
    torch.cuda.synchronize()
    n = out["accepted"].cpu().numpy()
    nxt = out["next_token"].cpu().numpy()
    zt_h = zt1.float().cpu().numpy()[0]
    for j in range(M + 1):
        reached = n >= j
        tok = np.where(n[reached] > j, cand_h[reached, min(j, M - 1)], nxt[reached]) if j < M else nxt[reached]
        assert reached.sum() > 300
        chi2_ok(tok, softmax(zt_h[j], tau), "position %d" % j)
    v.close()


def test_a_whole_speculation_step_replays_from_a_cuda_graph():
    """Draft from q', verify, exact-match and acceptance rates recorded into one graph: every call only
    launches kernels, so the replay must reproduce the eager results bit for bit."""
    from paper_2502_05202_b200 import workload as wl
    cfg = wl.tiny_config(B=10, K=3, V_t=50021, V_d=30011, dtype=wl.BF16, f_mapped=0.6, sigma_d=0.5,
                         temperatures=(0.0, 0.8, 1.0), seed=91)
    b = wl.make_batch(cfg)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    zt, zd = dev(b["target_logits"]).view(torch.bfloat16), dev(b["drafter_logits"]).view(torch.bfloat16)
    tau, u = dev(b["temperature"]), dev(b["uniforms"])
    ud = u[:, :cfg.K].contiguous()
    idmap = dev(b["id_map"])
    v = tli.Verifier(cfg.V_t, cfg.V_d, b["id_map"])
    v._ws = torch.empty(64 << 20, dtype=torch.uint8, device="cuda")          # one scratch for all four calls

    def step():
        d = v.draft(zd, tau, ud)
        out = v.verify(zt, zd, d["draft_ids"], tau, u)
        cand = idmap[d["draft_ids"].long()].contiguous()
        s = v.slem(zt, cand, tau, u)
        r = v.rates(zt, zd, tau)
        return [d["draft_ids"], out["accepted"], out["next_token"], s["accepted"], s["next_token"], r["alpha_tli"]]

    eager = [t.clone() for t in step()]
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        outs = step()
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(3):
        for t in outs:
            t.zero_()
        g.replay()
        torch.cuda.synchronize()
        for a, e in zip(outs, eager):
            assert torch.equal(a, e)
    del g
    v.close()
