"""Seeded synthetic inputs for TLI verification.

This module only *draws inputs*: logits, the drafter->target id map, draft
ids, temperatures and uniforms.  It holds none of the verification arithmetic
(no softmax, no acceptance test, no residual, no CDF) and is the one module
that both the CUDA path's callers and the CPU oracle's callers may share.

Shapes follow the vocabulary sizes the paper tabulates (32 000 ... 256 000) and
the overlap ratios it reports (0.12 - 0.85 of the target vocabulary); the
datasets and model weights behind those tables are not used, every value here
is drawn from a counter-based generator (Philox) keyed by
``(seed, tensor tag, sequence index)`` so that any sequence can be rebuilt in
isolation.

Recipe per sequence ``b`` (all noise iid):

* target logits ``zt[b, j, t] = 3 N(0,1) - zipf_s * ln(rank(t))`` for the
  K+1 target rows, ``rank`` a fixed random permutation of the target ids;
* id map: ``round(f * V_d)`` drafter ids chosen without replacement, each sent
  to a distinct random target id, all others ``-1``;
* drafter logits ``zd[b, j, x] = zt[b, j, map[x]] + sigma N(0,1)`` on mapped
  ids and ``N(-2, 1)`` elsewhere;
* logits are stored as float32 or as bfloat16 (round to nearest even) and all
  consumers read the stored bits;
* draft ids are drawn from the drafter distribution restricted to the mapped
  ids at the sequence's temperature -- done with the Gumbel-max trick
  (arg-max of ``zd / tau + Gumbel noise``) so that no softmax is evaluated
  here; temperature-0 sequences take the arg-max of the mapped drafter
  logits;  ``draft_mode="raw"`` draws over *all* drafter ids instead, which
  produces some drafts outside the intersection;
* uniforms are ``k * 2**-24`` with ``k`` uniform in ``[0, 2**24)``.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence

import numpy as np

F32 = 0
BF16 = 1

_TAG_RANK = 1
_TAG_MAP = 2
_TAG_TARGET = 3
_TAG_DRAFTER = 4
_TAG_DRAFT = 5
_TAG_UNIFORM = 6
_TAG_TEMPERATURE = 7


@dataclass(frozen=True)
class Config:
    """One synthetic workload."""

    name: str
    B: int
    K: int
    V_t: int
    V_d: int
    dtype: int                      # F32 or BF16
    f_mapped: float                 # share of drafter ids inside the intersection
    zipf_s: float = 1.1             # slope of the log-rank bias
    sigma_d: float = 1.0            # drafter noise on mapped ids
    temperatures: Sequence[float] = (1.0,)   # choices for the per-row draw
    greedy_rows: str = "none"       # "none" | "first_half" | "interleaved"
    seed: int = 1000

    @property
    def positions(self) -> int:
        return self.B * self.K

    @property
    def elt(self) -> int:
        return 4 if self.dtype == F32 else 2

    @property
    def logit_bytes(self) -> int:
        """Bytes of all logits, each read once."""
        return self.elt * self.B * ((self.K + 1) * self.V_t + self.K * self.V_d)


CONFIGS: List[Config] = [
    Config("cfg0", B=1, K=5, V_t=32000, V_d=32768, dtype=F32, f_mapped=0.70,
           zipf_s=1.1, sigma_d=1.0, temperatures=(1.0,), seed=1000),
    Config("cfg1", B=8, K=5, V_t=128256, V_d=49152, dtype=BF16, f_mapped=0.40,
           zipf_s=1.1, sigma_d=1.5, temperatures=(0.7,), seed=1001),
    Config("cfg2", B=64, K=8, V_t=152064, V_d=32000, dtype=BF16, f_mapped=0.85,
           zipf_s=1.1, sigma_d=0.8, temperatures=(0.5, 0.8, 1.0), seed=1002),
    Config("cfg3", B=256, K=4, V_t=256000, V_d=128256, dtype=F32, f_mapped=0.55,
           zipf_s=1.2, sigma_d=1.0, temperatures=(1.0,), seed=1003),
    Config("cfg4", B=32, K=16, V_t=128256, V_d=50257, dtype=BF16, f_mapped=0.30,
           zipf_s=1.1, sigma_d=2.0, temperatures=(0.9,), greedy_rows="first_half",
           seed=1004),
]


def config_by_name(name: str) -> Config:
    for c in CONFIGS:
        if c.name == name:
            return c
    raise KeyError(name)


# --------------------------------------------------------------------------
# storage formats
# --------------------------------------------------------------------------

def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round to nearest even."""
    bits = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = bits + np.uint32(0x7FFF) + ((bits >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns (uint16) -> float32, exact."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def store(x: np.ndarray, dtype: int) -> np.ndarray:
    """Round float32 values to the storage format; returns float32 (F32) or uint16 bits (BF16)."""
    if dtype == F32:
        return np.ascontiguousarray(x, dtype=np.float32)
    return f32_to_bf16_bits(x)


def stored_to_f32(x: np.ndarray, dtype: int) -> np.ndarray:
    return x if dtype == F32 else bf16_bits_to_f32(x)


# --------------------------------------------------------------------------
# generators
# --------------------------------------------------------------------------

def _rng(seed: int, tag: int, index: int = 0) -> np.random.Generator:
    key = np.array([np.uint64(seed), (np.uint64(tag) << np.uint64(40)) | np.uint64(index)], dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def make_rank_bias(cfg: Config) -> np.ndarray:
    """``-zipf_s * ln(rank(t))`` with ``rank`` a seeded permutation of 1..V_t (float32 [V_t])."""
    rank = _rng(cfg.seed, _TAG_RANK).permutation(cfg.V_t).astype(np.float64) + 1.0
    return (-cfg.zipf_s * np.log(rank)).astype(np.float32)


def make_id_map(cfg: Config) -> np.ndarray:
    """int32 [V_d]: drafter id -> target id, -1 outside the intersection; injective on mapped ids."""
    rng = _rng(cfg.seed, _TAG_MAP)
    n = int(round(cfg.f_mapped * cfg.V_d))
    n = min(n, cfg.V_t, cfg.V_d)
    id_map = np.full(cfg.V_d, -1, dtype=np.int32)
    if n > 0:
        xs = rng.permutation(cfg.V_d)[:n]
        ts = rng.permutation(cfg.V_t)[:n]
        id_map[xs] = ts.astype(np.int32)
    return id_map


def make_temperatures(cfg: Config) -> np.ndarray:
    rng = _rng(cfg.seed, _TAG_TEMPERATURE)
    choices = np.asarray(cfg.temperatures, dtype=np.float32)
    tau = choices[rng.integers(0, len(choices), size=cfg.B)]
    if cfg.greedy_rows == "first_half":
        tau[: cfg.B // 2] = 0.0
    elif cfg.greedy_rows == "interleaved":
        tau[0::2] = 0.0
    elif cfg.greedy_rows != "none":
        raise ValueError(cfg.greedy_rows)
    return tau.astype(np.float32)


def _make_row(cfg: Config, b: int, bias: np.ndarray, id_map: np.ndarray, tau: float,
              draft_mode: str):
    K, V_t, V_d = cfg.K, cfg.V_t, cfg.V_d
    zt = _rng(cfg.seed, _TAG_TARGET, b).standard_normal((K + 1, V_t), dtype=np.float32)
    zt *= np.float32(3.0)
    zt += bias[None, :]
    noise = _rng(cfg.seed, _TAG_DRAFTER, b).standard_normal((K, V_d), dtype=np.float32)
    mapped = id_map >= 0
    src = np.where(mapped, id_map, 0)
    zd = np.where(mapped[None, :],
                  zt[:K][:, src] + np.float32(cfg.sigma_d) * noise,
                  noise - np.float32(2.0)).astype(np.float32)
    zt_s = store(zt, cfg.dtype)
    zd_s = store(zd, cfg.dtype)

    # draft ids from the stored drafter logits
    zd_r = stored_to_f32(zd_s, cfg.dtype).astype(np.float64)
    rng_d = _rng(cfg.seed, _TAG_DRAFT, b)
    allowed = mapped if (draft_mode == "intersection" and mapped.any()) else np.ones(V_d, dtype=bool)
    if tau > 0.0:
        g = -np.log(-np.log(rng_d.random((K, V_d))))
        score = zd_r / float(tau) + g
    else:
        score = zd_r
    score = np.where(allowed[None, :], score, -np.inf)
    draft = np.argmax(score, axis=1).astype(np.int32)

    k24 = _rng(cfg.seed, _TAG_UNIFORM, b).integers(0, 1 << 24, size=K + 1)
    u = (k24.astype(np.float64) * 2.0 ** -24).astype(np.float32)
    return zt_s, zd_s, draft, u


def make_batch(cfg: Config, rows: Optional[Sequence[int]] = None, draft_mode: str = "intersection",
               threads: int = 8) -> Dict[str, np.ndarray]:
    """Build the inputs of one verification call.

    ``rows`` selects which sequences to build (default: all ``cfg.B``); row
    ``b`` is bit-identical however it is selected.  Returned arrays:
    ``target_logits [R,K+1,V_t]``, ``drafter_logits [R,K,V_d]`` (float32, or
    uint16 bfloat16 bit patterns), ``id_map int32 [V_d]``, ``draft_ids int32
    [R,K]``, ``temperature float32 [R]``, ``uniforms float32 [R,K+1]``.
    """
    if draft_mode not in ("intersection", "raw"):
        raise ValueError(draft_mode)
    rows = list(range(cfg.B)) if rows is None else list(rows)
    bias = make_rank_bias(cfg)
    id_map = make_id_map(cfg)
    tau_all = make_temperatures(cfg)
    store_dt = np.float32 if cfg.dtype == F32 else np.uint16
    R = len(rows)
    zt = np.empty((R, cfg.K + 1, cfg.V_t), dtype=store_dt)
    zd = np.empty((R, cfg.K, cfg.V_d), dtype=store_dt)
    draft = np.empty((R, cfg.K), dtype=np.int32)
    u = np.empty((R, cfg.K + 1), dtype=np.float32)

    def work(i: int) -> None:
        b = rows[i]
        zt[i], zd[i], draft[i], u[i] = _make_row(cfg, b, bias, id_map, float(tau_all[b]), draft_mode)

    if threads > 1 and R > 1:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(work, range(R)))
    else:
        for i in range(R):
            work(i)
    return {
        "target_logits": zt,
        "drafter_logits": zd,
        "id_map": id_map,
        "draft_ids": draft,
        "temperature": tau_all[rows].copy(),
        "uniforms": u,
    }


def tiny_config(name: str = "tiny", B: int = 4, K: int = 3, V_t: int = 11, V_d: int = 13,
                dtype: int = F32, f_mapped: float = 0.6, seed: int = 7, **kw) -> Config:
    """Small-vocabulary workloads for tests."""
    return Config(name, B=B, K=K, V_t=V_t, V_d=V_d, dtype=dtype, f_mapped=f_mapped, seed=seed, **kw)
