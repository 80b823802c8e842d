"""Comparison harness: the CUDA library against the fp64 oracle on the same stored inputs.

Rule (per sequence): results must be identical, except that a difference is
excused -- and counted -- when moving one uniform by less than 1e-6 explains it:

  (i)  the accept decision at position j may differ only if
       |u[b,j] - thr_oracle[b,j]| < 1e-6; the rest of the row is then compared
       with the oracle re-run with that decision forced;
  (ii) next_token may differ only if the GPU's token has positive weight in the
       oracle's distribution and v = u[b,K] lies within 1e-6 of the oracle's
       normalised CDF interval of that token.

Temperature-0 rows get no excuses.  p_draft / q_draft must agree within 1e-5.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np
import torch

import oracle
from paper_2502_05202_b200 import tli, workload as wl

TOL_U = 1e-6
TOL_P = 1e-5


def to_device(batch: Dict[str, np.ndarray], device="cuda") -> Dict[str, torch.Tensor]:
    """Copy one workload batch to the device; uint16 logits are reinterpreted as bfloat16."""
    out = {}
    for k in ("target_logits", "drafter_logits"):
        t = torch.from_numpy(batch[k])
        if t.dtype == torch.uint16:
            t = t.view(torch.bfloat16)
        out[k] = t.to(device)
    out["draft_ids"] = torch.from_numpy(batch["draft_ids"]).to(device)
    out["draft_lengths"] = (torch.from_numpy(np.asarray(batch["draft_lengths"], np.int32)).to(device)
                            if batch.get("draft_lengths") is not None else None)
    out["temperature"] = torch.from_numpy(batch["temperature"]).to(device)
    out["uniforms"] = torch.from_numpy(batch["uniforms"]).to(device)
    return out


def run_gpu(batch: Dict[str, np.ndarray], verifier: Optional[tli.Verifier] = None,
            dev: Optional[Dict[str, torch.Tensor]] = None, tiled: bool = False) -> Dict[str, np.ndarray]:
    """One tli_verify() call.  Without a verifier of the caller's a context is made for the call
    (`tiled`: the extra token by the tile kernels whatever the size) and the call is repeated on it:
    the second call must give the same results bit for bit."""
    if dev is None:
        dev = to_device(batch)

    def once(v):
        out = v.verify(dev["target_logits"], dev["drafter_logits"], dev["draft_ids"],
                       dev["temperature"], dev["uniforms"], draft_lengths=dev.get("draft_lengths"))
        torch.cuda.synchronize()
        return {k: x.cpu().numpy() for k, x in out.items()}

    if verifier is not None:
        return once(verifier)
    V_t = batch["target_logits"].shape[2]
    V_d = batch["drafter_logits"].shape[2]
    v = tli.Verifier(V_t, V_d, batch["id_map"], tiled=tiled)
    r = once(v)
    r2 = once(v)                                  # a second call on the same context: counters came back to zero
    v.close()
    for k in r:
        np.testing.assert_array_equal(r[k], r2[k], err_msg="repeat call differs (%s, tiled=%s)" % (k, tiled))
    return r


def run_oracle(batch: Dict[str, np.ndarray], threads: int = 8, **kw) -> Dict[str, np.ndarray]:
    return oracle.verify(batch["target_logits"], batch["drafter_logits"], batch["id_map"], batch["draft_ids"],
                         batch["temperature"], batch["uniforms"], threads=threads,
                         draft_lengths=batch.get("draft_lengths"), **kw)


@dataclass
class Report:
    rows: int = 0
    exact: int = 0
    excused_threshold: int = 0
    excused_sampler: int = 0
    failures: List[str] = field(default_factory=list)
    max_p_err: float = 0.0
    max_q_err: float = 0.0

    def ok(self) -> bool:
        return not self.failures

    def __str__(self) -> str:
        return ("rows=%d exact=%d excused_thr=%d excused_sampler=%d failures=%d max|dp|=%.2e max|dq|=%.2e%s" %
                (self.rows, self.exact, self.excused_threshold, self.excused_sampler, len(self.failures),
                 self.max_p_err, self.max_q_err, ("\n  " + "\n  ".join(self.failures[:10])) if self.failures else ""))


def _sub(batch, rows):
    rows = np.asarray(rows)
    return {"target_logits": batch["target_logits"][rows], "drafter_logits": batch["drafter_logits"][rows],
            "id_map": batch["id_map"], "draft_ids": batch["draft_ids"][rows],
            "temperature": batch["temperature"][rows], "uniforms": batch["uniforms"][rows],
            "draft_lengths": None if batch.get("draft_lengths") is None else np.asarray(batch["draft_lengths"])[rows]}


def compare(batch: Dict[str, np.ndarray], gpu: Dict[str, np.ndarray], orc: Optional[Dict[str, np.ndarray]] = None,
            threads: int = 8) -> Report:
    if orc is None:
        orc = run_oracle(batch, threads=threads)
    B, K = batch["draft_ids"].shape
    tau = batch["temperature"]
    u = batch["uniforms"].astype(np.float64)
    rep = Report(rows=B)

    # flags and diagnostics
    oflags = orc["flags"] & ~oracle.FLAG_SELFCHECK
    if (orc["flags"] & oracle.FLAG_SELFCHECK).any():
        rep.failures.append("oracle self-check flag set")
    bad = np.flatnonzero(oflags != gpu["row_status"])
    for b in bad[:5]:
        rep.failures.append("row %d: status gpu=%d oracle=%d" % (b, gpu["row_status"][b], oflags[b]))
    if "p_draft" in gpu:
        dp = np.abs(gpu["p_draft"].astype(np.float64) - orc["p_draft"])
        dq = np.abs(gpu["q_draft"].astype(np.float64) - orc["q_draft"])
        sampled = tau > 0
        if sampled.any():
            rep.max_p_err = float(dp[sampled].max())
            rep.max_q_err = float(dq[sampled].max())
        if rep.max_p_err > TOL_P or rep.max_q_err > TOL_P:
            rep.failures.append("draft probabilities differ: |dp|=%.3e |dq|=%.3e" % (rep.max_p_err, rep.max_q_err))

    n_g, n_o = gpu["accepted"].astype(np.int64), orc["accepted"].astype(np.int64)
    t_g, t_o = gpu["next_token"].astype(np.int64), orc["next_token"].astype(np.int64)
    same = (n_g == n_o) & (t_g == t_o)
    rep.exact = int(same.sum())
    todo = np.flatnonzero(~same)
    greedy_bad = [b for b in todo if tau[b] == 0]
    for b in greedy_bad[:5]:
        rep.failures.append("row %d (temperature 0): gpu (%d,%d) oracle (%d,%d)" % (b, n_g[b], t_g[b], n_o[b], t_o[b]))
    todo = np.array([b for b in todo if tau[b] != 0 and not (oflags[b] & (oracle.FLAG_NONFINITE | oracle.FLAG_BAD_TEMPERATURE))],
                    dtype=np.int64)
    if len(todo) == 0:
        return rep

    # (i) accept decisions: force the GPU's decisions where the oracle's threshold is within 1e-6 of u
    force = np.full((len(todo), K), -1, np.int8)
    thr = orc["thr"][todo].copy()
    n_cur = n_o[todo].copy()
    alive = np.ones(len(todo), bool)
    excused_thr = np.zeros(len(todo), bool)
    for _ in range(K + 1):
        diff = alive & (n_cur != n_g[todo])
        if not diff.any():
            break
        for i in np.flatnonzero(diff):
            b = todo[i]
            j = int(min(n_cur[i], n_g[b]))
            if abs(u[b, j] - thr[i, j]) < TOL_U:
                force[i, j] = 1 if n_g[b] > j else 0
                excused_thr[i] = True
            else:
                rep.failures.append("row %d: accepted gpu=%d oracle=%d, |u-thr|=%.3e at position %d" %
                                    (b, n_g[b], n_o[b], abs(u[b, j] - thr[i, j]), j))
                alive[i] = False
        idx = np.flatnonzero(diff & alive)
        if len(idx) == 0:
            break
        re = run_oracle(_sub(batch, todo[idx]), threads=threads, force_accept=force[idx])
        n_cur[idx] = re["accepted"]
        thr[idx] = re["thr"]
    # (ii) the sampled token, against the oracle run with the same accept decisions
    idx = np.flatnonzero(alive)
    if len(idx):
        re = run_oracle(_sub(batch, todo[idx]), threads=threads, force_accept=force[idx],
                        probe_token=t_g[todo[idx]].astype(np.int32))
        for k, i in enumerate(idx):
            b = todo[i]
            if re["accepted"][k] != n_g[b]:
                rep.failures.append("row %d: accepted gpu=%d oracle(forced)=%d" % (b, n_g[b], re["accepted"][k]))
                continue
            if re["next_token"][k] == t_g[b]:
                if excused_thr[i]:
                    rep.excused_threshold += 1
                continue
            v = u[b, K]
            if re["probe_w"][k] > 0 and re["probe_lo"][k] - TOL_U <= v <= re["probe_hi"][k] + TOL_U:
                rep.excused_sampler += 1
                if excused_thr[i]:
                    rep.excused_threshold += 1
            else:
                rep.failures.append("row %d: next_token gpu=%d oracle=%d, v=%.9f gpu-token interval [%.9f, %.9f] w=%.3e" %
                                    (b, t_g[b], re["next_token"][k], v, re["probe_lo"][k], re["probe_hi"][k], re["probe_w"][k]))
    return rep


def check(batch: Dict[str, np.ndarray], verifier: Optional[tli.Verifier] = None, threads: int = 8) -> Report:
    """The GPU against the oracle.  Without a verifier of the caller's both forms of the call are
    checked (extra token by size rule, and by the tile kernels); the report is the default form's."""
    if verifier is not None:
        rep = compare(batch, run_gpu(batch, verifier), threads=threads)
        assert rep.ok(), str(rep)
        return rep
    orc = run_oracle(batch, threads=threads)
    dev = to_device(batch)
    rep = compare(batch, run_gpu(batch, dev=dev), orc=orc, threads=threads)
    assert rep.ok(), str(rep)
    rep_tiled = compare(batch, run_gpu(batch, dev=dev, tiled=True), orc=orc, threads=threads)
    assert rep_tiled.ok(), "tile kernels: " + str(rep_tiled)
    return rep
