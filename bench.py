#!/usr/bin/env python
"""Benchmark of TLI verification (draft positions verified per second).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config cfg3] [--impl reference]

A step is one tli_verify() call on one synthetic batch: all kernels, all
sequences.  The headline workload is the largest of the five (cfg3: B=256, K=4,
V_t=256000, V_d=128256, fp32 logits, 1.8 GB per call, larger than L2).  With N>1
(under torchrun) the batch is split into contiguous blocks of sequences, one per
rank -- sequences are independent, there is no collective on the data path -- and
the value is the whole batch divided by the slowest rank's time (strong scaling).

Prints ONE JSON line.  `--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "draft positions verified/s"
UNIT = "positions/s"
L2_ROTATE_BYTES = 400 << 20          # distinct input bytes cycled through when one batch fits in L2
NOMINAL_HBM_GBS = 8000.0             # the nominal peak the target is worded against; fractions are given of both
KERNEL_SOURCE = os.path.join(ROOT, "paper_2502_05202_b200", "csrc", "tli.cu")
COUNTERS_FILE = os.path.join(ROOT, "profiles", "stats_kernel_counters.json")


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def algorithmic_bytes(cfg, batch) -> int:
    """All logits read once; temperature-0 sequences do not read drafter logits."""
    import numpy as np
    greedy = int((np.asarray(batch["temperature"]) == 0).sum())
    return cfg.elt * (cfg.B * (cfg.K + 1) * cfg.V_t + (cfg.B - greedy) * cfg.K * cfg.V_d)


class ClockSampler:
    """nvidia-smi clocks and throttle reasons of one GPU, sampled every 50 ms in the background."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ---------------------------------------------------------------------------
# CPU oracle legs
# ---------------------------------------------------------------------------

def time_oracle(batch, positions, min_seconds=10.0, max_reps=50):
    """The oracle as it stands, rows split over all host cores; returns (positions/s, cores, reps, seconds)."""
    import oracle
    cores = os.cpu_count() or 1
    oracle.build()
    run = lambda: oracle.verify(batch["target_logits"], batch["drafter_logits"], batch["id_map"], batch["draft_ids"],
                                batch["temperature"], batch["uniforms"], threads=cores)
    t0 = time.perf_counter()
    reps = 0
    while True:
        run()
        reps += 1
        dt = time.perf_counter() - t0
        if dt >= min_seconds or reps >= max_reps:
            break
    return positions * reps / dt, min(cores, len(batch["temperature"])), reps, dt


def time_oracle_single_thread(batch, K, rows=8, min_seconds=2.0, max_reps=20):
    """The oracle on one thread, on the first few sequences; returns (positions/s, sequences used)."""
    import oracle
    rows = min(rows, len(batch["temperature"]))
    sub = {k: (v if k == "id_map" else v[:rows]) for k, v in batch.items()
           if k in ("target_logits", "drafter_logits", "id_map", "draft_ids", "temperature", "uniforms")}
    run = lambda: oracle.verify(sub["target_logits"], sub["drafter_logits"], sub["id_map"], sub["draft_ids"],
                                sub["temperature"], sub["uniforms"], threads=1)
    t0 = time.perf_counter()
    reps = 0
    while True:
        run()
        reps += 1
        dt = time.perf_counter() - t0
        if dt >= min_seconds or reps >= max_reps:
            break
    return rows * K * reps / dt, rows


def reference_arm(args):
    """`--impl reference`: the CPU oracle on the same workload, rank 0 only."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from paper_2502_05202_b200 import workload as wl
    import oracle
    cfg = wl.config_by_name(args.config)
    cores = os.cpu_count() or 1
    rows = list(range(min(cfg.B, max(cores, 8) * 2)))          # bounded sample: a few rows per core
    batch = wl.make_batch(cfg, rows=rows)
    positions = len(rows) * cfg.K
    oracle.build()
    run = lambda: oracle.verify(batch["target_logits"], batch["drafter_logits"], batch["id_map"], batch["draft_ids"],
                                batch["temperature"], batch["uniforms"], threads=cores)
    for _ in range(args.warmup):
        run()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        run()
    dt = time.perf_counter() - t0
    value = positions * args.steps / dt
    used = min(cores, len(rows))
    sample = "first %d of %d sequences of %s per step (%d positions), all rows in fp64" % (len(rows), cfg.B, cfg.name, positions)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(cfg, None),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": used, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def source_digest():
    import hashlib
    with open(KERNEL_SOURCE, "rb") as f:
        return hashlib.sha256(f.read()).hexdigest()


def stats_kernel_counters(cfg):
    """ncu counters of one tli_stats_kernel launch on this workload, from the summary kept beside the
    other profiles: {"dram_bytes": read + write, "warp_instructions": ...} scaled to the batch by the
    sequences it holds (traffic and instruction count grow in proportion to B).  None when there is no
    capture of this workload, or when the kernel source has changed since the capture was taken."""
    try:
        with open(COUNTERS_FILE) as f:
            data = json.load(f)
    except (OSError, ValueError):
        return None
    if data.get("source_sha256") != source_digest():
        return None
    c = data.get("workloads", {}).get(cfg.name)
    if not c or cfg.B % c["B"]:
        return None
    k = cfg.B // c["B"]
    return {"dram_bytes": (c["dram_bytes_read"] + c["dram_bytes_write"]) * k,
            "warp_instructions": c["warp_instructions"] * k}


def workload_config(cfg, l2_note):
    c = {"workload": cfg.name, "B": cfg.B, "K": cfg.K, "V_t": cfg.V_t, "V_d": cfg.V_d,
         "logits": "f32" if cfg.elt == 4 else "bf16", "mapped_fraction": cfg.f_mapped,
         "positions_per_step": cfg.positions, "logit_bytes_per_step": cfg.logit_bytes}
    if l2_note:
        c["l2"] = l2_note
    return c


# ---------------------------------------------------------------------------
# GPU arm
# ---------------------------------------------------------------------------

class GpuCase:
    """One workload resident on the device: enough copies of the inputs to defeat L2, outputs, scratch."""

    def __init__(self, cfg, device, torch, tli, wl, want_host=False, rows=None, batch=None):
        self.cfg, self.torch, self.tli = cfg, torch, tli
        if batch is not None:                        # host arrays of a case that exists already
            self.batch = batch
        elif rows is not None:                       # a block of the batch's sequences (one rank of several)
            import dataclasses
            self.batch = wl.make_batch(cfg, rows=list(rows))
            cfg = self.cfg = dataclasses.replace(cfg, B=len(rows))
        else:
            self.batch = wl.make_batch(cfg)
        self.bytes = algorithmic_bytes(cfg, self.batch)
        l2 = torch.cuda.get_device_properties(device).L2_cache_size
        self.copies = 1 if cfg.logit_bytes > 2 * l2 else max(2, -(-L2_ROTATE_BYTES // cfg.logit_bytes))
        self.l2_note = ("inputs larger than L2 (%d MB per step vs %d MB)" % (cfg.logit_bytes >> 20, l2 >> 20)
                        if self.copies == 1 else
                        "%d distinct input copies rotated (%d MB in all vs %d MB L2)" %
                        (self.copies, (self.copies * cfg.logit_bytes) >> 20, l2 >> 20))
        b = self.batch
        zt = torch.from_numpy(b["target_logits"])
        zd = torch.from_numpy(b["drafter_logits"])
        if zt.dtype == torch.uint16:
            zt, zd = zt.view(torch.bfloat16), zd.view(torch.bfloat16)
        self.host = None
        if want_host:
            self.host = {"zt": zt.pin_memory(), "zd": zd.pin_memory(),
                         "draft": torch.from_numpy(b["draft_ids"]).pin_memory(),
                         "tau": torch.from_numpy(b["temperature"]).pin_memory(),
                         "u": torch.from_numpy(b["uniforms"]).pin_memory(),
                         "out": torch.empty(2, cfg.B, dtype=torch.int32).pin_memory()}
        self.zt = [zt.to(device)]
        self.zd = [zd.to(device)]
        for _ in range(self.copies - 1):
            self.zt.append(self.zt[0].clone())
            self.zd.append(self.zd[0].clone())
        self.draft = torch.from_numpy(b["draft_ids"]).to(device)
        self.tau = torch.from_numpy(b["temperature"]).to(device)
        self.u = torch.from_numpy(b["uniforms"]).to(device)
        self.out = torch.empty(2, cfg.B, dtype=torch.int32, device=device)      # accepted, next_token
        self.status = torch.empty(cfg.B, dtype=torch.int32, device=device)
        self.ver = tli.Verifier(cfg.V_t, cfg.V_d, b["id_map"], device=device.index)
        self.dt = tli.TLI_F32 if cfg.elt == 4 else tli.TLI_BF16
        self.plan = tli.tli_verify_plan(self.ver.ctx, cfg.B, cfg.K, self.dt)
        self.ws = self.ver.workspace(cfg.B, cfg.K, self.dt)
        self.args = [tli.make_args(self.zt[i], self.zd[i], self.draft, self.tau, self.u, self.out[0], self.out[1],
                                   self.ws, self.status) for i in range(self.copies)]
        self.stream = torch.cuda.current_stream().cuda_stream
        self.calls = 0
        self.host_args = None
        if want_host:
            dt = tli.TLI_F32 if cfg.elt == 4 else tli.TLI_BF16
            self.host_buf = torch.empty(tli.tli_verify_host_buffer_bytes(self.ver.ctx, cfg.B, cfg.K, dt),
                                        dtype=torch.uint8, device=device)
            h = self.host
            self.host_args = tli.make_host_args(h["zt"], h["zd"], h["draft"], h["tau"], h["u"],
                                                h["out"][0], h["out"][1], self.host_buf)

    def step(self):
        self.tli.tli_verify(self.ver.ctx, self.args[self.calls % self.copies], self.stream)
        self.calls += 1

    def probe(self):
        """The launches of one call with kernels that do nothing."""
        self.tli.tli_launch_probe(self.ver.ctx, self.cfg.B, self.cfg.K, self.dt, self.stream)

    def touched_bytes(self):
        """Bytes a call reads in all: every logit once, plus the second pass over target row n of every
        sampled sequence and, where a draft was rejected, over drafter row n."""
        import numpy as np
        acc = self.out[0].cpu().numpy()
        tau = np.asarray(self.batch["temperature"])
        sampled = tau > 0
        extra = int(sampled.sum()) * self.cfg.V_t + int((sampled & (acc < self.cfg.K)).sum()) * self.cfg.V_d
        return self.bytes + self.cfg.elt * extra

    def sustained(self, seconds, sampler_index):
        """Back-to-back calls for `seconds`: ms per call under a sustained load, with the SM clock seen."""
        torch = self.torch
        for _ in range(3):
            self.step()
        torch.cuda.synchronize()
        probe_ms = timed(torch, None, 50, self.step, 1) / 50
        calls = max(50, int(seconds / (probe_ms * 1e-3)))
        sampler = ClockSampler(sampler_index)
        sampler.start()
        ms = timed(torch, None, calls, self.step, 1) / calls
        clocks = sampler.stop()
        mhz = clocks.get("sm_mhz")
        return {"seconds": ms * calls * 1e-3, "calls": calls, "ms_per_call": ms, "sm_mhz_median": mhz,
                "ms_times_mhz": (ms * mhz) if mhz else None, "reasons": clocks.get("reasons"),
                "path_frac_of_peak": None}

    def step_e2e(self):
        """tli_verify_host(): pinned host buffers in, host results out -- H2D of every input, the kernels,
        D2H of (accepted, next_token), all inside the one C call."""
        self.tli.tli_verify_host(self.ver.ctx, self.host_args, self.stream)

    def make_graph(self):
        """One CUDA graph holding a tli_verify() call on every input copy; returns (graph, calls in it)."""
        torch = self.torch
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            h = torch.cuda.current_stream().cuda_stream
            for i in range(self.copies):
                self.tli.tli_verify(self.ver.ctx, self.args[i], h)
        torch.cuda.current_stream().wait_stream(side)
        return g, self.copies

    def per_call_ms(self, calls):
        """Events around single calls: (median, min) ms."""
        torch = self.torch
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(calls)]
        for a, b in ev:
            a.record()
            self.step()
            b.record()
        torch.cuda.synchronize()
        t = [a.elapsed_time(b) for a, b in ev]
        return statistics.median(t), min(t)

    def draft_timing(self, steps):
        """tli_draft_sample() on this workload's drafter logits, all K rows per sequence: ms per call."""
        torch, tli, cfg = self.torch, self.tli, self.cfg
        ids = torch.empty(cfg.B, cfg.K, dtype=torch.int32, device=self.zd[0].device)
        need = tli.tli_draft_workspace_bytes(self.ver.ctx, cfg.B, cfg.K, tli.TLI_F32 if cfg.elt == 4 else tli.TLI_BF16)
        ws = torch.empty(need, dtype=torch.uint8, device=self.zd[0].device)
        u = self.u[:, :cfg.K].contiguous()
        args = [tli.make_draft_args(z, self.tau, u, ids, ws) for z in self.zd]
        n = [0]

        def step():
            tli.tli_draft_sample(self.ver.ctx, args[n[0] % len(args)], self.stream)
            n[0] += 1
        for _ in range(3 + len(args)):
            step()
        ms = timed(torch, None, steps, step, 1) / steps
        assert int((ids < 0).sum()) == 0, "a draft id could not be drawn on benchmark inputs"
        greedy = int((self.tau == 0).sum())
        nbytes = cfg.elt * cfg.B * cfg.K * cfg.V_d
        return {"ms_per_call": ms, "rows_per_s": cfg.B * cfg.K / (ms * 1e-3), "gbs": nbytes / (ms * 1e-3) / 1e9,
                "rows_per_call": cfg.B * cfg.K, "bytes_per_call": nbytes, "greedy_sequences": greedy}

    def slem_timing(self, steps):
        """tli_slem_verify() on this workload's target logits (candidates: the drafts carried to target ids)."""
        import numpy as np
        torch, tli, cfg = self.torch, self.tli, self.cfg
        dev = self.zt[0].device
        cand = torch.from_numpy(self.batch["id_map"][self.batch["draft_ids"]].astype(np.int32)).to(dev)
        acc = torch.empty(cfg.B, dtype=torch.int32, device=dev)
        nxt = torch.empty(cfg.B, dtype=torch.int32, device=dev)
        st = torch.empty(cfg.B, dtype=torch.int32, device=dev)
        need = tli.tli_slem_workspace_bytes(self.ver.ctx, cfg.B, cfg.K, tli.TLI_F32 if cfg.elt == 4 else tli.TLI_BF16)
        ws = torch.empty(need, dtype=torch.uint8, device=dev)
        args = [tli.make_slem_args(z, cand, self.tau, self.u, acc, nxt, ws, row_status=st) for z in self.zt]
        n = [0]

        def step():
            tli.tli_slem_verify(self.ver.ctx, args[n[0] % len(args)], self.stream)
            n[0] += 1
        for _ in range(3 + len(args)):
            step()
        ms = timed(torch, None, steps, step, 1) / steps
        assert int(st.abs().sum()) == 0, "row_status not clean on benchmark inputs"
        nbytes = cfg.elt * cfg.B * (cfg.K + 1) * cfg.V_t
        return {"ms_per_call": ms, "positions_per_s": cfg.B * cfg.K / (ms * 1e-3), "gbs": nbytes / (ms * 1e-3) / 1e9,
                "rows_per_call": cfg.B * (cfg.K + 1), "bytes_per_call": nbytes,
                "mean_accepted": float(acc.float().mean().item())}

    def rates_timing(self, steps):
        """tli_acceptance_rates() on this workload (K positions per sequence): ms per call."""
        torch, tli, cfg = self.torch, self.tli, self.cfg
        dev = self.zt[0].device
        dt = tli.TLI_F32 if cfg.elt == 4 else tli.TLI_BF16
        need = tli.tli_rates_workspace_bytes(self.ver.ctx, cfg.B, cfg.K, dt)
        if need == 0:
            return None
        outs = [torch.empty(cfg.B, cfg.K, dtype=torch.float32, device=dev) for _ in range(3)]
        st = torch.empty(cfg.B, cfg.K, dtype=torch.int32, device=dev)
        ws = torch.empty(need, dtype=torch.uint8, device=dev)
        args = [tli.make_rates_args(zt, zd, self.tau, *outs, ws, st) for zt, zd in zip(self.zt, self.zd)]
        n = [0]

        def step():
            tli.tli_acceptance_rates(self.ver.ctx, args[n[0] % len(args)], self.stream)
            n[0] += 1
        for _ in range(3 + len(args)):
            step()
        ms = timed(torch, None, steps, step, 1) / steps
        assert int(st.abs().sum()) == 0, "position_status not clean on benchmark inputs"
        greedy = int((self.tau == 0).sum())
        # target rows once, drafter rows twice (statistics, then the pair pass); the gathers are not counted
        nbytes = cfg.elt * cfg.B * cfg.K * (cfg.V_t + 2 * cfg.V_d)
        return {"ms_per_call": ms, "positions_per_s": cfg.B * cfg.K / (ms * 1e-3), "gbs": nbytes / (ms * 1e-3) / 1e9,
                "bytes_per_call": nbytes, "greedy_sequences": greedy,
                "mean_alpha_tli": float(outs[2].mean().item()), "mean_alpha_union": float(outs[1].mean().item()),
                "mean_mass": float(outs[0].mean().item())}

    def e2e_bytes(self):
        h = self.host
        h2d = sum(h[k].numel() * h[k].element_size() for k in ("zt", "zd", "draft", "tau", "u"))
        return h2d, h["out"].numel() * h["out"].element_size()

    def profile(self, steps):
        """Average ms of the three kernels: statistics, decision, sampling."""
        acc = [0.0, 0.0, 0.0]
        for _ in range(steps):
            ms = self.tli.tli_verify_profile(self.ver.ctx, self.args[self.calls % self.copies], self.stream)
            self.calls += 1
            for i in range(3):
                acc[i] += ms[i]
        return tuple(x / steps for x in acc)

    def check(self):
        st = self.status.cpu()
        assert int(st.abs().sum()) == 0, "row_status not clean on benchmark inputs"

    def close(self):
        self.ver.close()


def timed(torch, dist, steps, fn, world):
    """K steps between two events, barrier + synchronize on both sides, max over ranks; returns ms in all."""
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    if world > 1:
        t = torch.tensor([ms], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    return ms


def independent_streams(case, device, torch, tli, wl, nstreams, steps):
    """Per-call time when `nstreams` independent batches of this workload (own context, inputs, outputs and
    scratch each) are verified in turn on as many CUDA streams: the dependent tail of one call then runs
    under the streaming of the next.  What a server with several batches in flight sees; the figures of a
    single stream of calls stay the headline."""
    cases = [case] + [GpuCase(case.cfg, device, torch, tli, wl, batch=case.batch) for _ in range(nstreams - 1)]
    streams = [torch.cuda.Stream() for _ in range(nstreams)]
    saved = case.stream
    for c, st in zip(cases, streams):
        c.stream = st.cuda_stream

    def run(n):
        for i in range(n):
            cases[i % nstreams].step()
    run(4 * nstreams)
    torch.cuda.synchronize()
    n = max(steps, 4 * case.copies) // nstreams * nstreams
    best = float("inf")
    for _ in range(3):
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for st in streams:
            st.wait_event(e0)
        run(n)
        for st in streams:
            torch.cuda.current_stream().wait_stream(st)
        e1.record()
        torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1) / n)
    for c in cases:
        c.check()
    for c in cases[1:]:
        c.close()
    case.stream = saved
    return best


def call_timings(case, torch, steps):
    """Per-call figures beside the K-step loop: events around single calls, and a CUDA-graph replay."""
    med, mn = case.per_call_ms(min(max(steps, 20), 200))
    g, n = case.make_graph()
    reps = max(3, -(-steps // n))
    for _ in range(2):
        g.replay()
    ms = timed(torch, None, reps, g.replay, 1) / (reps * n)
    del g
    return {"ms_call_median": med, "ms_call_min": mn, "ms_call_graph_replay": ms}


def gpu_arm(args):
    import torch
    from paper_2502_05202_b200 import tli, workload as wl
    tli.load()                                   # fails loudly when the CUDA library is missing
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        if world == 1 and args.gpus > 1:
            raise SystemExit("--gpus %d needs torchrun with that many ranks" % args.gpus)
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    peak, peak_kind = load_peaks()
    cfg = wl.config_by_name(args.config)
    if args.batch:
        import dataclasses
        cfg = dataclasses.replace(cfg, B=args.batch)
    if args.kernels_only:
        args.no_per_config = True
    rows = None
    if world > 1:
        from paper_2502_05202_b200 import shard
        b0, b1 = shard.row_block(cfg.B, rank, world)            # this rank's sequences; nothing is exchanged
        rows = range(b0, b1)
    case = GpuCase(cfg, device, torch, tli, wl, want_host=not args.kernels_only, rows=rows)
    sms = torch.cuda.get_device_properties(device).multi_processor_count

    def describe(c, ms_step, with_extras):
        """Figures of one workload from a device-timed loop of `ms_step` per call."""
        gbs = c.bytes / (ms_step * 1e-3) / 1e9
        c.profile(3)
        ms_stats, ms_decide, ms_sample = c.profile(min(max(args.steps, 20), 50))
        counters = stats_kernel_counters(c.cfg)
        stats_gbs = c.bytes / (ms_stats * 1e-3) / 1e9
        d = {"workload": c.cfg.name, "ms_per_step": ms_step, "value": c.cfg.positions / (ms_step * 1e-3),
             "path_gbs": gbs, "path_frac_of_peak": gbs / peak, "path_frac_of_nominal": gbs / NOMINAL_HBM_GBS,
             "roofline_ms_at_peak": c.bytes / (peak * 1e9) * 1e3,
             "call_traffic_ratio": c.touched_bytes() / c.bytes,
             "plan": c.plan, "launches_per_call": c.plan["launches"],
             "ms_stats_kernel": ms_stats, "ms_decide_kernel": ms_decide, "ms_sample_kernel": ms_sample,
             "roofline": {"kernel": "tli_stats_kernel", "bound": "hbm", "achieved": stats_gbs, "peak": peak,
                          "peak_kind": peak_kind, "unit": "GB/s", "frac": stats_gbs / peak,
                          "frac_of_nominal": stats_gbs / NOMINAL_HBM_GBS,
                          "traffic": counters["dram_bytes"] if counters else None,
                          "algorithmic_bytes": c.bytes, "path_frac": gbs / peak,
                          "note": ("frac above 1: the peak is a copy's read+write rate, a read-only stream can exceed it"
                                   if stats_gbs > peak else None)},
             "l2": c.l2_note}
        if with_extras:
            d.update(call_timings(c, torch, args.steps))
            # the floor of a call: its launches with kernels that do nothing
            for _ in range(5):
                c.probe()
            n = max(args.steps, 100)
            d["launch_floor_ms"] = timed(torch, None, n, c.probe, 1) / n
            sus = c.sustained(args.sustain_seconds, local)
            sus["path_frac_of_peak"] = c.bytes / (sus["ms_per_call"] * 1e-3) / 1e9 / peak
            d["sustained"] = sus
            if counters and sus.get("sm_mhz_median"):
                # every issue slot of the GPU busy with this kernel's instructions: its floor whatever memory does
                d["roofline"]["issue_floor_ms"] = counters["warp_instructions"] / (4 * sms * sus["sm_mhz_median"] * 1e6) * 1e3
            # the other form of the sampling pass
            tli.tli_set_tiled(c.ver.ctx, True)
            for _ in range(3 + c.copies):
                c.step()
            n = max(args.steps, 2 * c.copies)
            d["ms_per_step_tile_kernels"] = timed(torch, None, n, c.step, 1) / n
            tli.tli_set_tiled(c.ver.ctx, False)
            d["independent_streams"] = {}
            for ns in (2, 3):
                m = independent_streams(c, device, torch, tli, wl, ns, max(args.steps, 100))
                d["independent_streams"][str(ns)] = {"ms_per_call": m, "path_frac_of_peak": c.bytes / (m * 1e-3) / 1e9 / peak}
            d["draft_sample"] = c.draft_timing(max(args.steps, 20))
            d["slem_verify"] = c.slem_timing(max(args.steps, 20))
            d["acceptance_rates"] = c.rates_timing(max(args.steps, 20))
        return d

    for _ in range(max(args.warmup, 3)):
        case.step()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ms = timed(torch, dist, args.steps, case.step, world)
    clocks = sampler.stop() if rank == 0 else None
    ms_step = ms / args.steps
    head = describe(case, ms_step, with_extras=(world == 1 and not args.kernels_only))
    case.check()
    # end to end: host buffers in, host results out
    e2e_steps = max(3, min(args.steps, 10))
    if args.kernels_only:
        ms_e2e, h2d, d2h = float("nan"), 0, 0
    else:
        for _ in range(2):
            case.step_e2e()
        ms_e2e = timed(torch, dist, e2e_steps, case.step_e2e, world)
        h2d, d2h = case.e2e_bytes()
    total_bytes = case.bytes
    if world > 1:
        t = torch.tensor([h2d, d2h, total_bytes], dtype=torch.int64, device="cuda")
        dist.all_reduce(t)
        h2d, d2h, total_bytes = int(t[0]), int(t[1]), int(t[2])

    value = cfg.positions / (ms_step * 1e-3)             # the whole batch, all ranks, over the slowest rank's time
    path_gbs = total_bytes / (ms_step * 1e-3) / 1e9
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "strong" if world > 1 else "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": dict(workload_config(cfg, case.l2_note),
                       parallelism=("sequences split into %d contiguous blocks, one per GPU, no collective" % world)
                       if world > 1 else "one GPU"),
        "clocks": clocks,
        "e2e": {"value": cfg.positions / (ms_e2e / e2e_steps * 1e-3), "unit": UNIT,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e / e2e_steps},
        "gpu_launches": case.plan["launches"] * args.steps,
        "path_gbs": path_gbs,
        "path_frac_of_peak": path_gbs / (peak * world),
        "path_frac_of_nominal": path_gbs / (NOMINAL_HBM_GBS * world),
        "roofline": head["roofline"],
    }
    if "ms_call_median" in head:
        out["per_call"] = {k: head[k] for k in ("ms_call_median", "ms_call_min", "ms_call_graph_replay")}
    for k in ("draft_sample", "slem_verify", "acceptance_rates", "sustained", "launch_floor_ms"):
        out[k] = head.get(k)
    headline_batch = case.batch
    case.close()
    del case
    torch.cuda.empty_cache()

    if rank == 0 and world == 1 and not args.no_per_config:
        per = []
        for c in wl.CONFIGS:
            if c.name == cfg.name:
                per.append(head)
                continue
            k = GpuCase(c, device, torch, tli, wl)
            for _ in range(max(args.warmup, 3) + k.copies):
                k.step()
            steps = max(args.steps, 2 * k.copies)
            m = timed(torch, None, steps, k.step, 1) / steps
            per.append(describe(k, m, with_extras=True))
            k.check()
            k.close()
            del k
            torch.cuda.empty_cache()
        out["per_config"] = per

    if rank == 0 and world == 1 and not args.kernels_only:
        v, cores, reps, secs = time_oracle(headline_batch, cfg.positions, min_seconds=args.cpu_seconds)
        v1, rows1 = time_oracle_single_thread(headline_batch, cfg.K)
        out["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                               "sample": "all %d sequences of %s, %d repetitions in %.1f s" % (cfg.B, cfg.name, reps, secs),
                               "single_thread_value": v1,
                               "single_thread_sample": "first %d sequences of %s on one thread" % (rows1, cfg.name)}
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default="cfg3")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-per-config", action="store_true", help="skip the four other workloads")
    ap.add_argument("--cpu-seconds", type=float, default=10.0, help="CPU time given to the oracle baseline leg")
    ap.add_argument("--sustain-seconds", type=float, default=2.0,
                    help="length of the sustained leg per workload (back-to-back calls, clocks sampled)")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's B (profiling on a smaller case)")
    ap.add_argument("--kernels-only", action="store_true",
                    help="only the device-timed loop: no per-config, end-to-end or CPU legs (for profiler runs)")
    args = ap.parse_args()
    if args.impl == "reference":
        reference_arm(args)
    else:
        gpu_arm(args)


if __name__ == "__main__":
    main()
