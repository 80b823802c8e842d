"""TEST INFRASTRUCTURE -- not part of the product path.

ctypes front end of the fp64 CPU oracle in ``tli_oracle.c`` (Algorithms 4 and 5
of the paper: ``verify`` for the verification half, ``draft`` for drawing the
draft ids from q'), of Algorithm 2's exact-match verification (``slem``) and of
the paper's expected acceptance rates (``rates``).  Only tests, the smoke check and the benchmark's CPU-baseline
legs may import this package; the CUDA library never does, and this package
imports nothing from it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor
from typing import Dict, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tli_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

F32 = 0
BF16 = 1

FLAG_DRAFT_RANGE = 1
FLAG_DRAFT_UNMAPPED = 2
FLAG_NONFINITE = 4
FLAG_FALLBACK = 8
FLAG_BAD_TEMPERATURE = 32
FLAG_SELFCHECK = 64


class _Args(ctypes.Structure):
    _fields_ = [
        ("B", ctypes.c_int32), ("K", ctypes.c_int32), ("V_t", ctypes.c_int32), ("V_d", ctypes.c_int32),
        ("dtype", ctypes.c_int32),
        ("target_logits", ctypes.c_void_p), ("t_stride_b", ctypes.c_int64), ("t_stride_k", ctypes.c_int64),
        ("drafter_logits", ctypes.c_void_p), ("d_stride_b", ctypes.c_int64), ("d_stride_k", ctypes.c_int64),
        ("id_map", ctypes.c_void_p), ("draft_ids", ctypes.c_void_p),
        ("temperature", ctypes.c_void_p), ("uniforms", ctypes.c_void_p),
        ("force_accept", ctypes.c_void_p), ("probe_token", ctypes.c_void_p),
        ("accepted", ctypes.c_void_p), ("next_token", ctypes.c_void_p), ("flags", ctypes.c_void_p),
        ("thr", ctypes.c_void_p), ("p_draft", ctypes.c_void_p), ("q_draft", ctypes.c_void_p),
        ("cdf_lo", ctypes.c_void_p), ("cdf_hi", ctypes.c_void_p), ("total", ctypes.c_void_p),
        ("probe_lo", ctypes.c_void_p), ("probe_hi", ctypes.c_void_p), ("probe_w", ctypes.c_void_p),
        ("draft_lengths", ctypes.c_void_p),
    ]


class _DraftArgs(ctypes.Structure):
    _fields_ = [
        ("B", ctypes.c_int32), ("R", ctypes.c_int32), ("V_d", ctypes.c_int32), ("dtype", ctypes.c_int32),
        ("drafter_logits", ctypes.c_void_p), ("d_stride_b", ctypes.c_int64), ("d_stride_r", ctypes.c_int64),
        ("id_map", ctypes.c_void_p), ("temperature", ctypes.c_void_p), ("uniforms", ctypes.c_void_p),
        ("probe_id", ctypes.c_void_p),
        ("draft_ids", ctypes.c_void_p), ("flags", ctypes.c_void_p), ("q_draft", ctypes.c_void_p),
        ("cdf_lo", ctypes.c_void_p), ("cdf_hi", ctypes.c_void_p),
        ("probe_lo", ctypes.c_void_p), ("probe_hi", ctypes.c_void_p), ("probe_w", ctypes.c_void_p),
    ]


class _SlemArgs(ctypes.Structure):
    _fields_ = [
        ("B", ctypes.c_int32), ("M", ctypes.c_int32), ("V_t", ctypes.c_int32), ("dtype", ctypes.c_int32),
        ("target_logits", ctypes.c_void_p), ("t_stride_b", ctypes.c_int64), ("t_stride_k", ctypes.c_int64),
        ("candidates", ctypes.c_void_p), ("lengths", ctypes.c_void_p),
        ("temperature", ctypes.c_void_p), ("uniforms", ctypes.c_void_p), ("probe_token", ctypes.c_void_p),
        ("sampled", ctypes.c_void_p), ("accepted", ctypes.c_void_p), ("next_token", ctypes.c_void_p),
        ("flags", ctypes.c_void_p), ("cdf_lo", ctypes.c_void_p), ("cdf_hi", ctypes.c_void_p),
        ("probe_lo", ctypes.c_void_p), ("probe_hi", ctypes.c_void_p), ("probe_w", ctypes.c_void_p),
    ]


class _RatesArgs(ctypes.Structure):
    _fields_ = [
        ("B", ctypes.c_int32), ("K", ctypes.c_int32), ("V_t", ctypes.c_int32), ("V_d", ctypes.c_int32),
        ("dtype", ctypes.c_int32),
        ("target_logits", ctypes.c_void_p), ("t_stride_b", ctypes.c_int64), ("t_stride_k", ctypes.c_int64),
        ("drafter_logits", ctypes.c_void_p), ("d_stride_b", ctypes.c_int64), ("d_stride_k", ctypes.c_int64),
        ("id_map", ctypes.c_void_p), ("temperature", ctypes.c_void_p),
        ("mass", ctypes.c_void_p), ("alpha_union", ctypes.c_void_p), ("alpha_tli", ctypes.c_void_p),
        ("flags", ctypes.c_void_p),
    ]


def build(force: bool = False) -> str:
    """Compile ``tli_oracle.c`` with gcc -O2 into ``liboracle.so`` beside it."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.oracle_tli_verify.argtypes = [ctypes.POINTER(_Args), ctypes.c_int32, ctypes.c_int32]
        lib.oracle_tli_verify.restype = ctypes.c_int
        lib.oracle_tli_distributions.argtypes = [ctypes.POINTER(_Args), ctypes.c_int32, ctypes.c_int32,
                                                 ctypes.c_void_p, ctypes.c_void_p]
        lib.oracle_tli_distributions.restype = ctypes.c_int
        lib.oracle_tli_draft.argtypes = [ctypes.POINTER(_DraftArgs), ctypes.c_int32, ctypes.c_int32]
        lib.oracle_tli_draft.restype = ctypes.c_int
        lib.oracle_slem_verify.argtypes = [ctypes.POINTER(_SlemArgs), ctypes.c_int32, ctypes.c_int32]
        lib.oracle_slem_verify.restype = ctypes.c_int
        lib.oracle_tli_rates.argtypes = [ctypes.POINTER(_RatesArgs), ctypes.c_int32, ctypes.c_int32]
        lib.oracle_tli_rates.restype = ctypes.c_int
        _lib = lib
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data


class _Call:
    """Keeps the numpy arrays of one call alive next to the C struct."""

    def __init__(self, target_logits, drafter_logits, id_map, draft_ids, temperature, uniforms,
                 force_accept=None, probe_token=None, draft_lengths=None):
        zt = np.asarray(target_logits)
        zd = np.asarray(drafter_logits)
        if zt.dtype == np.float32 and zd.dtype == np.float32:
            dtype = F32
        elif zt.dtype == np.uint16 and zd.dtype == np.uint16:
            dtype = BF16
        else:
            raise TypeError("logits must both be float32 or both be uint16 bfloat16 bit patterns")
        if zt.ndim != 3 or zd.ndim != 3:
            raise ValueError("logits must be [B,K+1,V_t] and [B,K,V_d]")
        B, K1, V_t = zt.shape
        K = K1 - 1
        if zd.shape[0] != B or zd.shape[1] != K:
            raise ValueError("drafter logits must be [B,K,V_d]")
        V_d = zd.shape[2]
        if zt.strides[2] != zt.itemsize or zd.strides[2] != zd.itemsize:
            raise ValueError("vocabulary axis must be contiguous")
        self.zt, self.zd = zt, zd
        self.id_map = np.ascontiguousarray(id_map, dtype=np.int32)
        self.draft = np.ascontiguousarray(draft_ids, dtype=np.int32).reshape(B, K)
        self.tau = np.ascontiguousarray(temperature, dtype=np.float32).reshape(B)
        self.u = np.ascontiguousarray(uniforms, dtype=np.float32).reshape(B, K + 1)
        if self.id_map.shape != (V_d,):
            raise ValueError("id_map must be [V_d]")
        self.force = None if force_accept is None else np.ascontiguousarray(force_accept, dtype=np.int8).reshape(B, K)
        self.probe = None if probe_token is None else np.ascontiguousarray(probe_token, dtype=np.int32).reshape(B)
        self.lengths = None if draft_lengths is None else np.ascontiguousarray(draft_lengths, dtype=np.int32).reshape(B)
        self.out: Dict[str, np.ndarray] = {
            "accepted": np.zeros(B, np.int32), "next_token": np.zeros(B, np.int32),
            "flags": np.zeros(B, np.int32),
            "thr": np.zeros((B, K), np.float64), "p_draft": np.zeros((B, K), np.float64),
            "q_draft": np.zeros((B, K), np.float64),
            "cdf_lo": np.zeros(B, np.float64), "cdf_hi": np.zeros(B, np.float64),
            "total": np.zeros(B, np.float64),
        }
        if self.probe is not None:
            self.out.update(probe_lo=np.zeros(B, np.float64), probe_hi=np.zeros(B, np.float64),
                            probe_w=np.zeros(B, np.float64))
        o = self.out
        self.B, self.K = B, K
        self.args = _Args(
            B, K, V_t, V_d, dtype,
            zt.ctypes.data, zt.strides[0] // zt.itemsize, zt.strides[1] // zt.itemsize,
            zd.ctypes.data, zd.strides[0] // zd.itemsize, zd.strides[1] // zd.itemsize,
            _ptr(self.id_map), _ptr(self.draft), _ptr(self.tau), _ptr(self.u),
            _ptr(self.force), _ptr(self.probe),
            _ptr(o["accepted"]), _ptr(o["next_token"]), _ptr(o["flags"]),
            _ptr(o["thr"]), _ptr(o["p_draft"]), _ptr(o["q_draft"]),
            _ptr(o["cdf_lo"]), _ptr(o["cdf_hi"]), _ptr(o["total"]),
            _ptr(o.get("probe_lo")), _ptr(o.get("probe_hi")), _ptr(o.get("probe_w")),
            _ptr(self.lengths),
        )


def verify(target_logits, drafter_logits, id_map, draft_ids, temperature, uniforms,
           force_accept=None, probe_token=None, threads: int = 1, draft_lengths=None) -> Dict[str, np.ndarray]:
    """Run the oracle on a whole batch.

    Logits are float32 arrays or uint16 arrays holding bfloat16 bit patterns;
    the batch axes may be strided (a zero batch stride broadcasts one set of
    logits to every row).  ``threads`` > 1 splits the rows over that many host
    threads; the arithmetic per row is unchanged.  Returns a dict with
    ``accepted``, ``next_token``, ``flags`` (int32 [B]), ``thr``, ``p_draft``,
    ``q_draft`` (float64 [B,K]), ``cdf_lo``, ``cdf_hi``, ``total`` (float64
    [B]) and, when ``probe_token`` is given, ``probe_lo/hi/w``.  With
    ``draft_lengths`` (int32 [B], 0..K) only that many drafts of a sequence
    count and its extra token comes from target row ``draft_lengths[b]`` when
    all of them are accepted.
    """
    lib = _load()
    call = _Call(target_logits, drafter_logits, id_map, draft_ids, temperature, uniforms,
                 force_accept, probe_token, draft_lengths)
    B = call.B
    threads = max(1, min(int(threads), B))

    def run(lo_hi):
        rc = lib.oracle_tli_verify(ctypes.byref(call.args), lo_hi[0], lo_hi[1])
        if rc != 0:
            raise RuntimeError("oracle_tli_verify failed with code %d" % rc)

    if threads == 1:
        run((0, B))
    else:
        cuts = [(B * i) // threads for i in range(threads + 1)]
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(run, [(cuts[i], cuts[i + 1]) for i in range(threads)]))
    return call.out


def distributions(target_logits, drafter_logits, id_map, temperature, b: int, j: int):
    """(p, q'_T) of row ``b`` position ``j`` as float64 [V_t] arrays, q' carried to target ids."""
    lib = _load()
    zt = np.asarray(target_logits)
    B, K1, V_t = zt.shape
    K = K1 - 1
    call = _Call(target_logits, drafter_logits, id_map, np.zeros((B, K), np.int32), temperature,
                 np.zeros((B, K + 1), np.float32))
    p = np.zeros(V_t, np.float64)
    qT = np.zeros(V_t, np.float64)
    rc = lib.oracle_tli_distributions(ctypes.byref(call.args), b, j, p.ctypes.data, qT.ctypes.data)
    if rc != 0:
        raise RuntimeError("oracle_tli_distributions failed with code %d" % rc)
    return p, qT


def draft(drafter_logits, id_map, temperature, uniforms, probe_id=None, threads: int = 1) -> Dict[str, np.ndarray]:
    """Draw one drafter id per row of ``drafter_logits`` [B,R,V_d] from Algorithm 4's q'.

    ``uniforms`` is [B,R].  Returns ``draft_ids`` (int32 [B,R], -1 where none can be drawn),
    ``flags`` (int32 [B]), ``q_draft``, ``cdf_lo``, ``cdf_hi`` (float64 [B,R]) and, with
    ``probe_id`` (int32 [B,R]), ``probe_lo/hi/w``: the normalised CDF interval and weight of that id.
    """
    lib = _load()
    zd = np.asarray(drafter_logits)
    if zd.dtype == np.float32:
        dtype = F32
    elif zd.dtype == np.uint16:
        dtype = BF16
    else:
        raise TypeError("logits must be float32 or uint16 bfloat16 bit patterns")
    if zd.ndim != 3 or zd.strides[2] != zd.itemsize:
        raise ValueError("drafter logits must be [B,R,V_d] with a contiguous vocabulary axis")
    B, R, V_d = zd.shape
    idm = np.ascontiguousarray(id_map, dtype=np.int32)
    if idm.shape != (V_d,):
        raise ValueError("id_map must be [V_d]")
    tau = np.ascontiguousarray(temperature, dtype=np.float32).reshape(B)
    u = np.ascontiguousarray(uniforms, dtype=np.float32).reshape(B, R)
    probe = None if probe_id is None else np.ascontiguousarray(probe_id, dtype=np.int32).reshape(B, R)
    out: Dict[str, np.ndarray] = {
        "draft_ids": np.zeros((B, R), np.int32), "flags": np.zeros(B, np.int32),
        "q_draft": np.zeros((B, R), np.float64), "cdf_lo": np.zeros((B, R), np.float64),
        "cdf_hi": np.zeros((B, R), np.float64),
    }
    if probe is not None:
        out.update(probe_lo=np.zeros((B, R), np.float64), probe_hi=np.zeros((B, R), np.float64),
                   probe_w=np.zeros((B, R), np.float64))
    args = _DraftArgs(B, R, V_d, dtype, zd.ctypes.data, zd.strides[0] // zd.itemsize, zd.strides[1] // zd.itemsize,
                      _ptr(idm), _ptr(tau), _ptr(u), _ptr(probe),
                      _ptr(out["draft_ids"]), _ptr(out["flags"]), _ptr(out["q_draft"]),
                      _ptr(out["cdf_lo"]), _ptr(out["cdf_hi"]),
                      _ptr(out.get("probe_lo")), _ptr(out.get("probe_hi")), _ptr(out.get("probe_w")))
    threads = max(1, min(int(threads), B))

    def run(lo_hi):
        rc = lib.oracle_tli_draft(ctypes.byref(args), lo_hi[0], lo_hi[1])
        if rc != 0:
            raise RuntimeError("oracle_tli_draft failed with code %d" % rc)

    if threads == 1:
        run((0, B))
    else:
        cuts = [(B * i) // threads for i in range(threads + 1)]
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(run, [(cuts[i], cuts[i + 1]) for i in range(threads)]))
    return out


def slem(target_logits, candidates, temperature, uniforms, lengths=None, probe_token=None,
         threads: int = 1) -> Dict[str, np.ndarray]:
    """Algorithm 2's verification: sample t'_j from each of the M+1 target rows, first mismatch with
    ``candidates`` (int32 [B,M], the re-tokenised drafts).  Returns ``sampled`` (int32 [B,M+1]),
    ``accepted``, ``next_token``, ``flags`` (int32 [B]), ``cdf_lo``, ``cdf_hi`` (float64 [B,M+1]) and,
    with ``probe_token`` (int32 [B,M+1]), ``probe_lo/hi/w``."""
    lib = _load()
    zt = np.asarray(target_logits)
    if zt.dtype == np.float32:
        dtype = F32
    elif zt.dtype == np.uint16:
        dtype = BF16
    else:
        raise TypeError("logits must be float32 or uint16 bfloat16 bit patterns")
    if zt.ndim != 3 or zt.strides[2] != zt.itemsize:
        raise ValueError("target logits must be [B,M+1,V_t] with a contiguous vocabulary axis")
    B, M1, V_t = zt.shape
    M = M1 - 1
    cand = np.ascontiguousarray(candidates, dtype=np.int32).reshape(B, M)
    tau = np.ascontiguousarray(temperature, dtype=np.float32).reshape(B)
    u = np.ascontiguousarray(uniforms, dtype=np.float32).reshape(B, M + 1)
    ln = None if lengths is None else np.ascontiguousarray(lengths, dtype=np.int32).reshape(B)
    probe = None if probe_token is None else np.ascontiguousarray(probe_token, dtype=np.int32).reshape(B, M + 1)
    out: Dict[str, np.ndarray] = {
        "sampled": np.zeros((B, M + 1), np.int32), "accepted": np.zeros(B, np.int32),
        "next_token": np.zeros(B, np.int32), "flags": np.zeros(B, np.int32),
        "cdf_lo": np.zeros((B, M + 1), np.float64), "cdf_hi": np.zeros((B, M + 1), np.float64),
    }
    if probe is not None:
        out.update(probe_lo=np.zeros((B, M + 1), np.float64), probe_hi=np.zeros((B, M + 1), np.float64),
                   probe_w=np.zeros((B, M + 1), np.float64))
    args = _SlemArgs(B, M, V_t, dtype, zt.ctypes.data, zt.strides[0] // zt.itemsize, zt.strides[1] // zt.itemsize,
                     _ptr(cand), _ptr(ln), _ptr(tau), _ptr(u), _ptr(probe),
                     _ptr(out["sampled"]), _ptr(out["accepted"]), _ptr(out["next_token"]), _ptr(out["flags"]),
                     _ptr(out["cdf_lo"]), _ptr(out["cdf_hi"]),
                     _ptr(out.get("probe_lo")), _ptr(out.get("probe_hi")), _ptr(out.get("probe_w")))
    threads = max(1, min(int(threads), B))

    def run(lo_hi):
        rc = lib.oracle_slem_verify(ctypes.byref(args), lo_hi[0], lo_hi[1])
        if rc != 0:
            raise RuntimeError("oracle_slem_verify failed with code %d" % rc)

    if threads == 1:
        run((0, B))
    else:
        cuts = [(B * i) // threads for i in range(threads + 1)]
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(run, [(cuts[i], cuts[i + 1]) for i in range(threads)]))
    return out


def rates(target_logits, drafter_logits, id_map, temperature, threads: int = 1) -> Dict[str, np.ndarray]:
    """Expected acceptance rates per draft position: ``mass`` (drafter mass on the intersection),
    ``alpha_union`` (drafting from q) and ``alpha_tli`` (drafting from q'), float64 [B,K]; ``flags`` int32 [B].
    ``target_logits`` is [B,>=K,V_t] (rows 0..K-1 are read), ``drafter_logits`` [B,K,V_d]."""
    lib = _load()
    zt, zd = np.asarray(target_logits), np.asarray(drafter_logits)
    if zt.dtype == np.float32 and zd.dtype == np.float32:
        dtype = F32
    elif zt.dtype == np.uint16 and zd.dtype == np.uint16:
        dtype = BF16
    else:
        raise TypeError("logits must both be float32 or both be uint16 bfloat16 bit patterns")
    if zt.ndim != 3 or zd.ndim != 3 or zt.strides[2] != zt.itemsize or zd.strides[2] != zd.itemsize:
        raise ValueError("logits must be 3-d with a contiguous vocabulary axis")
    B, K, V_d = zd.shape
    if zt.shape[0] != B or zt.shape[1] < K:
        raise ValueError("target logits must be [B,>=K,V_t]")
    V_t = zt.shape[2]
    idm = np.ascontiguousarray(id_map, dtype=np.int32)
    tau = np.ascontiguousarray(temperature, dtype=np.float32).reshape(B)
    out = {"mass": np.zeros((B, K)), "alpha_union": np.zeros((B, K)), "alpha_tli": np.zeros((B, K)),
           "flags": np.zeros(B, np.int32)}
    args = _RatesArgs(B, K, V_t, V_d, dtype, zt.ctypes.data, zt.strides[0] // zt.itemsize, zt.strides[1] // zt.itemsize,
                      zd.ctypes.data, zd.strides[0] // zd.itemsize, zd.strides[1] // zd.itemsize,
                      _ptr(idm), _ptr(tau), _ptr(out["mass"]), _ptr(out["alpha_union"]), _ptr(out["alpha_tli"]),
                      _ptr(out["flags"]))
    threads = max(1, min(int(threads), B))

    def run(lo_hi):
        rc = lib.oracle_tli_rates(ctypes.byref(args), lo_hi[0], lo_hi[1])
        if rc != 0:
            raise RuntimeError("oracle_tli_rates failed with code %d" % rc)

    if threads == 1:
        run((0, B))
    else:
        cuts = [(B * i) // threads for i in range(threads + 1)]
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(run, [(cuts[i], cuts[i + 1]) for i in range(threads)]))
    return out
