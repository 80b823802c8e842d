"""tli_verify_static(): verification on the library's built-in scratch, for callers that cannot
allocate device memory when they need it (an inference server whose HBM is already fully
committed, a decode loop that must not stall on cudaMalloc).

Collected last on purpose: if this addition fails, `pytest -x` has already run everything else.
The entry point is compared with tli_verify() and with the CPU oracle on two calls in a row -- the
second on a different, smaller batch, so whatever the first call left in the shared scratch is still there.
"""
import ctypes
import dataclasses

import numpy as np
import pytest
import torch

from paper_2502_05202_b200 import tli, workload as wl
from parity_util import compare, to_device

pytestmark = pytest.mark.gpu


def _outputs(B, K):
    return {"accepted": torch.full((B,), -7, dtype=torch.int32, device="cuda"),
            "next_token": torch.full((B,), -7, dtype=torch.int32, device="cuda"),
            "row_status": torch.full((B,), -7, dtype=torch.int32, device="cuda"),
            "p_draft": torch.full((B, K), -7.0, dtype=torch.float32, device="cuda"),
            "q_draft": torch.full((B, K), -7.0, dtype=torch.float32, device="cuda")}


def _run(entry, ctx, dev, workspace):
    B, K = dev["draft_ids"].shape
    out = _outputs(B, K)
    args = tli.make_args(dev["target_logits"], dev["drafter_logits"], dev["draft_ids"], dev["temperature"],
                         dev["uniforms"], out["accepted"], out["next_token"], workspace, out["row_status"],
                         out["p_draft"], out["q_draft"])
    entry(ctx, args)
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items()}


def test_static_scratch_matches_tli_verify_on_two_calls_in_a_row():
    cfg = wl.tiny_config(B=9, K=4, V_t=3 * 8192 + 77, V_d=2 * 8192 + 5, dtype=wl.BF16, f_mapped=0.6,
                         temperatures=(0.7, 1.0), greedy_rows="interleaved", seed=301)
    first = wl.make_batch(cfg)
    second = wl.make_batch(dataclasses.replace(cfg, B=5, K=2))          # same seed: same id map
    v = tli.Verifier(cfg.V_t, cfg.V_d, first["id_map"])
    no_workspace = torch.empty(0, dtype=torch.uint8, device="cuda")     # data_ptr() == 0: nothing to lean on
    assert no_workspace.data_ptr() == 0
    for batch in (first, second):
        dev = to_device(batch)
        B, K = batch["draft_ids"].shape
        expect = _run(tli.tli_verify, v.ctx, dev, v.workspace(B, K, tli.TLI_BF16))
        got = _run(tli.tli_verify_static, v.ctx, dev, no_workspace)
        for k in ("accepted", "next_token", "row_status"):
            np.testing.assert_array_equal(got[k], expect[k], err_msg=k)
        for k in ("p_draft", "q_draft"):
            np.testing.assert_allclose(got[k], expect[k], rtol=0, atol=1e-5, err_msg=k)
        assert (got["accepted"] >= 0).all() and (got["next_token"] >= 0).all()
        rep = compare(batch, got)                    # and against the oracle, by the rule of the parity tests
        assert rep.ok(), str(rep)
    v.close()


def test_static_scratch_refuses_batches_beyond_its_size():
    cfg = wl.tiny_config(B=2, K=1, V_t=300000, V_d=1000, dtype=wl.F32, f_mapped=0.5, seed=302)
    batch = wl.make_batch(cfg)
    v = tli.Verifier(cfg.V_t, cfg.V_d, batch["id_map"])
    dev = to_device(batch)
    out = _outputs(2, 1)
    args = tli.make_args(dev["target_logits"], dev["drafter_logits"], dev["draft_ids"], dev["temperature"],
                         dev["uniforms"], out["accepted"], out["next_token"],
                         torch.empty(0, dtype=torch.uint8, device="cuda"))
    args.B = 20000                                  # that many sequences of this vocabulary need ~14 MiB of scratch
    assert tli.tli_workspace_bytes(v.ctx, 20000, 1, tli.TLI_F32) > tli.TLI_STATIC_SCRATCH_BYTES
    rc = tli.load().tli_verify_static(v.ctx, ctypes.byref(args), None)
    assert rc == tli.TLI_ERR_STATIC_SCRATCH
    assert b"TLI_STATIC_SCRATCH_BYTES" in tli.load().tli_status_string(rc)
    torch.cuda.synchronize()
    assert (out["accepted"].cpu() == -7).all()      # nothing was launched
    args.B = 2
    tli.tli_verify_static(v.ctx, args)              # the real batch fits
    torch.cuda.synchronize()
    assert (out["accepted"].cpu() >= 0).all()
    v.close()
