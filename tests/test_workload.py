"""The seeded input generator: determinism, row isolation, storage formats, map structure."""
import numpy as np
import torch

from paper_2502_05202_b200 import workload as wl


def test_configs_match_the_five_workloads():
    got = [(c.B, c.K, c.V_t, c.V_d, c.dtype, c.f_mapped) for c in wl.CONFIGS]
    assert got == [(1, 5, 32000, 32768, wl.F32, 0.70), (8, 5, 128256, 49152, wl.BF16, 0.40),
                   (64, 8, 152064, 32000, wl.BF16, 0.85), (256, 4, 256000, 128256, wl.F32, 0.55),
                   (32, 16, 128256, 50257, wl.BF16, 0.30)]
    assert [c.logit_bytes for c in wl.CONFIGS] == [1423360, 16244736, 207945728, 1836056576, 191005696]


def test_bf16_rounding_is_nearest_even():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.normal(0, 10, 5000).astype(np.float32),
                        np.array([1.0, 1.00390625, 1.01171875, -3.0e38, 1e-30, 0.0], np.float32)])
    ours = wl.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(ours, ref)
    np.testing.assert_array_equal(wl.bf16_bits_to_f32(ours),
                                  torch.from_numpy(x).to(torch.bfloat16).float().numpy())


def test_rows_rebuild_in_isolation_and_deterministically():
    cfg = wl.tiny_config(B=6, K=3, V_t=300, V_d=257, dtype=wl.BF16, f_mapped=0.5,
                         temperatures=(0.5, 1.0), greedy_rows="interleaved")
    full = wl.make_batch(cfg)
    again = wl.make_batch(cfg, threads=1)
    part = wl.make_batch(cfg, rows=[4, 1])
    for k in full:
        np.testing.assert_array_equal(full[k], again[k])
    for k in ("target_logits", "drafter_logits", "draft_ids", "temperature", "uniforms"):
        np.testing.assert_array_equal(part[k], full[k][[4, 1]])
    assert full["target_logits"].dtype == np.uint16
    assert (full["temperature"][0::2] == 0).all() and (full["temperature"][1::2] > 0).all()


def test_map_structure_and_drafts():
    cfg = wl.tiny_config(B=5, K=4, V_t=500, V_d=700, f_mapped=0.4)
    b = wl.make_batch(cfg)
    m = b["id_map"]
    inside = m[m >= 0]
    assert len(inside) == round(0.4 * 700) and len(np.unique(inside)) == len(inside)
    assert inside.min() >= 0 and inside.max() < 500
    assert (m[b["draft_ids"]] >= 0).all()                 # TLI drafts stay inside the intersection
    raw = wl.make_batch(cfg, draft_mode="raw")
    assert (m[raw["draft_ids"]] < 0).any()
    u = b["uniforms"]
    assert u.dtype == np.float32 and (u >= 0).all() and (u < 1).all()
    assert (u * 2 ** 24 == np.round(u * 2 ** 24)).all()


def test_drafter_tracks_target_on_mapped_ids():
    cfg = wl.tiny_config(B=2, K=2, V_t=4000, V_d=3000, f_mapped=0.7, sigma_d=0.5)
    b = wl.make_batch(cfg)
    m = b["id_map"]
    x = np.flatnonzero(m >= 0)
    diff = b["drafter_logits"][:, :, x] - b["target_logits"][:, :2][:, :, m[x]]
    assert abs(diff.std() - 0.5) < 0.05 and abs(diff.mean()) < 0.05
    out = b["drafter_logits"][:, :, np.flatnonzero(m < 0)]
    assert abs(out.mean() + 2.0) < 0.1 and abs(out.std() - 1.0) < 0.1
