"""Thin ctypes binding of the C ABI in include/tli.h.

Argument marshalling only: every step of the verification runs in the CUDA
library.  torch is used for device memory and streams.  There is no CPU
fallback: if ``libtli.so`` is missing or cannot be loaded, importing a function
from here raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtli.so")

TLI_F32 = 0
TLI_BF16 = 1
TLI_OK = 0
TLI_ERR_ARG = -1
TLI_ERR_BAD_MAP = -2
TLI_ERR_CUDA = -3
TLI_ERR_WORKSPACE = -4
TLI_ERR_UNSUPPORTED = -5
TLI_ERR_STATIC_SCRATCH = -6
TLI_ROW_DRAFT_RANGE = 1
TLI_ROW_DRAFT_UNMAPPED = 2
TLI_ROW_NONFINITE = 4
TLI_ROW_FALLBACK = 8
TLI_ROW_TIMEOUT = 16
TLI_ROW_BAD_TEMPERATURE = 32
TLI_MAX_B = 65535
TLI_MAX_K = 64
TLI_MAX_V = 1048576
TLI_MAX_SHARDS = 64
TLI_STATIC_SCRATCH_BYTES = 4194304

EXPORTS = ("tli_create", "tli_destroy", "tli_workspace_bytes", "tli_verify", "tli_verify_static", "tli_verify_profile", "tli_set_tiled", "tli_set_max_cluster", "tli_reset", "tli_selftest_bounded_wait",
           "tli_draft_workspace_bytes", "tli_draft_sample", "tli_slem_workspace_bytes", "tli_slem_verify",
           "tli_verify_host_buffer_bytes", "tli_verify_host", "tli_rates_workspace_bytes", "tli_acceptance_rates",
           "tli_ctx_info",
           "tli_shard_create", "tli_shard_info", "tli_shard_workspace_bytes", "tli_shard_record_bytes", "tli_shard_rows_bytes",
           "tli_shard_stats", "tli_shard_decide", "tli_shard_weights", "tli_shard_select",
           "tli_verify_plan", "tli_launch_probe",
           "tli_status_string", "tli_last_cuda_error")


class tli_verify_args(ctypes.Structure):
    _fields_ = [
        ("B", ctypes.c_int32), ("K", ctypes.c_int32), ("dtype", ctypes.c_int32),
        ("target_logits", ctypes.c_void_p), ("t_stride_b", ctypes.c_int64), ("t_stride_k", ctypes.c_int64),
        ("drafter_logits", ctypes.c_void_p), ("d_stride_b", ctypes.c_int64), ("d_stride_k", ctypes.c_int64),
        ("draft_ids", ctypes.c_void_p), ("temperature", ctypes.c_void_p), ("uniforms", ctypes.c_void_p),
        ("accepted", ctypes.c_void_p), ("next_token", ctypes.c_void_p), ("row_status", ctypes.c_void_p),
        ("p_draft", ctypes.c_void_p), ("q_draft", ctypes.c_void_p),
        ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
        ("draft_lengths", ctypes.c_void_p),
    ]


class tli_verify_host_args(ctypes.Structure):
    _fields_ = [
        ("B", ctypes.c_int32), ("K", ctypes.c_int32), ("dtype", ctypes.c_int32),
        ("target_logits", ctypes.c_void_p), ("drafter_logits", ctypes.c_void_p), ("draft_ids", ctypes.c_void_p),
        ("temperature", ctypes.c_void_p), ("uniforms", ctypes.c_void_p),
        ("accepted", ctypes.c_void_p), ("next_token", ctypes.c_void_p), ("row_status", ctypes.c_void_p),
        ("device_buffer", ctypes.c_void_p), ("device_buffer_bytes", ctypes.c_size_t),
    ]


class tli_rates_args(ctypes.Structure):
    _fields_ = [
        ("B", ctypes.c_int32), ("K", ctypes.c_int32), ("dtype", ctypes.c_int32),
        ("target_logits", ctypes.c_void_p), ("t_stride_b", ctypes.c_int64), ("t_stride_k", ctypes.c_int64),
        ("drafter_logits", ctypes.c_void_p), ("d_stride_b", ctypes.c_int64), ("d_stride_k", ctypes.c_int64),
        ("temperature", ctypes.c_void_p),
        ("mass", ctypes.c_void_p), ("alpha_union", ctypes.c_void_p), ("alpha_tli", ctypes.c_void_p),
        ("position_status", ctypes.c_void_p),
        ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
    ]


class tli_draft_args(ctypes.Structure):
    _fields_ = [
        ("B", ctypes.c_int32), ("R", ctypes.c_int32), ("dtype", ctypes.c_int32),
        ("drafter_logits", ctypes.c_void_p), ("d_stride_b", ctypes.c_int64), ("d_stride_r", ctypes.c_int64),
        ("temperature", ctypes.c_void_p), ("uniforms", ctypes.c_void_p),
        ("draft_ids", ctypes.c_void_p), ("q_draft", ctypes.c_void_p), ("draft_status", ctypes.c_void_p),
        ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
    ]


class tli_slem_args(ctypes.Structure):
    _fields_ = [
        ("B", ctypes.c_int32), ("M", ctypes.c_int32), ("dtype", ctypes.c_int32),
        ("target_logits", ctypes.c_void_p), ("t_stride_b", ctypes.c_int64), ("t_stride_k", ctypes.c_int64),
        ("candidates", ctypes.c_void_p), ("lengths", ctypes.c_void_p),
        ("temperature", ctypes.c_void_p), ("uniforms", ctypes.c_void_p),
        ("accepted", ctypes.c_void_p), ("next_token", ctypes.c_void_p), ("sampled", ctypes.c_void_p),
        ("row_status", ctypes.c_void_p),
        ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
    ]


class TLIError(RuntimeError):
    def __init__(self, code: int, where: str):
        lib = load()
        msg = lib.tli_status_string(code).decode()
        detail = lib.tli_last_cuda_error().decode() if code == TLI_ERR_CUDA else ""
        super().__init__("%s failed: %s (%d)%s" % (where, msg, code, (": " + detail) if detail else ""))
        self.code = code


_lib = None


def load() -> ctypes.CDLL:
    """Load libtli.so (built by ``python -m paper_2502_05202_b200.build``); raises if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError("CUDA library %s is missing; run `python -m paper_2502_05202_b200.build`" % LIB_PATH)
        lib = ctypes.CDLL(LIB_PATH)
        lib.tli_create.argtypes = [ctypes.POINTER(ctypes.c_void_p), ctypes.c_int, ctypes.c_int32, ctypes.c_int32,
                                   ctypes.c_void_p]
        lib.tli_create.restype = ctypes.c_int
        lib.tli_destroy.argtypes = [ctypes.c_void_p]
        lib.tli_destroy.restype = ctypes.c_int
        lib.tli_workspace_bytes.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32]
        lib.tli_workspace_bytes.restype = ctypes.c_size_t
        lib.tli_verify.argtypes = [ctypes.c_void_p, ctypes.POINTER(tli_verify_args), ctypes.c_void_p]
        lib.tli_verify.restype = ctypes.c_int
        lib.tli_verify_static.argtypes = [ctypes.c_void_p, ctypes.POINTER(tli_verify_args), ctypes.c_void_p]
        lib.tli_verify_static.restype = ctypes.c_int
        lib.tli_verify_profile.argtypes = [ctypes.c_void_p, ctypes.POINTER(tli_verify_args), ctypes.c_void_p,
                                           ctypes.POINTER(ctypes.c_float)]
        lib.tli_verify_profile.restype = ctypes.c_int
        lib.tli_draft_workspace_bytes.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32]
        lib.tli_draft_workspace_bytes.restype = ctypes.c_size_t
        lib.tli_draft_sample.argtypes = [ctypes.c_void_p, ctypes.POINTER(tli_draft_args), ctypes.c_void_p]
        lib.tli_draft_sample.restype = ctypes.c_int
        lib.tli_slem_workspace_bytes.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32]
        lib.tli_slem_workspace_bytes.restype = ctypes.c_size_t
        lib.tli_slem_verify.argtypes = [ctypes.c_void_p, ctypes.POINTER(tli_slem_args), ctypes.c_void_p]
        lib.tli_slem_verify.restype = ctypes.c_int
        lib.tli_verify_host_buffer_bytes.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32]
        lib.tli_verify_host_buffer_bytes.restype = ctypes.c_size_t
        lib.tli_verify_host.argtypes = [ctypes.c_void_p, ctypes.POINTER(tli_verify_host_args), ctypes.c_void_p]
        lib.tli_verify_host.restype = ctypes.c_int
        lib.tli_rates_workspace_bytes.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32]
        lib.tli_rates_workspace_bytes.restype = ctypes.c_size_t
        lib.tli_acceptance_rates.argtypes = [ctypes.c_void_p, ctypes.POINTER(tli_rates_args), ctypes.c_void_p]
        lib.tli_acceptance_rates.restype = ctypes.c_int
        lib.tli_shard_create.argtypes = [ctypes.POINTER(ctypes.c_void_p), ctypes.c_int, ctypes.c_int32, ctypes.c_int32,
                                         ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32]
        lib.tli_shard_create.restype = ctypes.c_int
        lib.tli_shard_info.argtypes = [ctypes.c_void_p] + [ctypes.POINTER(ctypes.c_int32)] * 6
        lib.tli_shard_info.restype = ctypes.c_int
        lib.tli_shard_workspace_bytes.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32]
        lib.tli_shard_workspace_bytes.restype = ctypes.c_size_t
        lib.tli_shard_record_bytes.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32]
        lib.tli_shard_record_bytes.restype = ctypes.c_size_t
        lib.tli_shard_rows_bytes.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32]
        lib.tli_shard_rows_bytes.restype = ctypes.c_size_t
        lib.tli_shard_stats.argtypes = [ctypes.c_void_p, ctypes.POINTER(tli_verify_args), ctypes.c_void_p, ctypes.c_void_p]
        lib.tli_shard_stats.restype = ctypes.c_int
        lib.tli_shard_decide.argtypes = [ctypes.c_void_p, ctypes.POINTER(tli_verify_args), ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        lib.tli_shard_decide.restype = ctypes.c_int
        lib.tli_shard_weights.argtypes = [ctypes.c_void_p, ctypes.POINTER(tli_verify_args), ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        lib.tli_shard_weights.restype = ctypes.c_int
        lib.tli_shard_select.argtypes = [ctypes.c_void_p, ctypes.POINTER(tli_verify_args), ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        lib.tli_shard_select.restype = ctypes.c_int
        lib.tli_verify_plan.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.POINTER(ctypes.c_int32)]
        lib.tli_verify_plan.restype = ctypes.c_int
        lib.tli_launch_probe.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p]
        lib.tli_launch_probe.restype = ctypes.c_int
        lib.tli_reset.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
        lib.tli_reset.restype = ctypes.c_int
        lib.tli_set_tiled.argtypes = [ctypes.c_void_p, ctypes.c_int]
        lib.tli_set_tiled.restype = ctypes.c_int
        lib.tli_set_max_cluster.argtypes = [ctypes.c_void_p, ctypes.c_int]
        lib.tli_set_max_cluster.restype = ctypes.c_int
        lib.tli_selftest_bounded_wait.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_uint, ctypes.POINTER(ctypes.c_int)]
        lib.tli_selftest_bounded_wait.restype = ctypes.c_int
        lib.tli_ctx_info.argtypes = [ctypes.c_void_p] + [ctypes.POINTER(ctypes.c_int32)] * 3
        lib.tli_ctx_info.restype = ctypes.c_int
        lib.tli_status_string.argtypes = [ctypes.c_int]
        lib.tli_status_string.restype = ctypes.c_char_p
        lib.tli_last_cuda_error.argtypes = []
        lib.tli_last_cuda_error.restype = ctypes.c_char_p
        _lib = lib
    return _lib


def tli_create(device: int, V_t: int, V_d: int, id_map) -> int:
    """tli_create(): returns the context handle; ``id_map`` is a host int32 array [V_d]."""
    m = np.ascontiguousarray(id_map, dtype=np.int32)
    if m.shape != (V_d,):
        raise ValueError("id_map must have V_d entries")
    h = ctypes.c_void_p()
    rc = load().tli_create(ctypes.byref(h), int(device), int(V_t), int(V_d), m.ctypes.data)
    if rc != TLI_OK:
        raise TLIError(rc, "tli_create")
    return h.value


def tli_destroy(ctx: int) -> None:
    rc = load().tli_destroy(ctx)
    if rc != TLI_OK:
        raise TLIError(rc, "tli_destroy")


def tli_workspace_bytes(ctx: int, B: int, K: int, dtype: int) -> int:
    return int(load().tli_workspace_bytes(ctx, B, K, dtype))


def _logit_dtype(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return TLI_F32
    if t.dtype == torch.bfloat16:
        return TLI_BF16
    raise TypeError("logits must be float32 or bfloat16")


def make_args(target_logits: torch.Tensor, drafter_logits: torch.Tensor, draft_ids: torch.Tensor,
              temperature: torch.Tensor, uniforms: torch.Tensor, accepted: torch.Tensor,
              next_token: torch.Tensor, workspace: torch.Tensor, row_status: Optional[torch.Tensor] = None,
              p_draft: Optional[torch.Tensor] = None, q_draft: Optional[torch.Tensor] = None,
              draft_lengths: Optional[torch.Tensor] = None) -> tli_verify_args:
    """Fill a tli_verify_args from device tensors (no copies; the tensors must outlive the call)."""
    B, K1, _ = target_logits.shape
    K = K1 - 1
    dt = _logit_dtype(target_logits)
    if _logit_dtype(drafter_logits) != dt:
        raise TypeError("both logit tensors must have the same dtype")
    if target_logits.stride(2) != 1 or drafter_logits.stride(2) != 1:
        raise ValueError("the vocabulary axis must be contiguous")
    if drafter_logits.shape[0] != B or drafter_logits.shape[1] != K:
        raise ValueError("drafter logits must be [B, K, V_d]")
    for name, t, dtype, shape in (("draft_ids", draft_ids, torch.int32, (B, K)),
                                  ("temperature", temperature, torch.float32, (B,)),
                                  ("uniforms", uniforms, torch.float32, (B, K + 1)),
                                  ("accepted", accepted, torch.int32, (B,)),
                                  ("next_token", next_token, torch.int32, (B,))):
        if t.dtype != dtype or tuple(t.shape) != shape or not t.is_contiguous():
            raise ValueError("%s must be a contiguous %s tensor of shape %s" % (name, dtype, shape))
    opt = lambda t: None if t is None else t.data_ptr()
    return tli_verify_args(
        B, K, dt,
        target_logits.data_ptr(), target_logits.stride(0), target_logits.stride(1),
        drafter_logits.data_ptr(), drafter_logits.stride(0), drafter_logits.stride(1),
        draft_ids.data_ptr(), temperature.data_ptr(), uniforms.data_ptr(),
        accepted.data_ptr(), next_token.data_ptr(), opt(row_status), opt(p_draft), opt(q_draft),
        workspace.data_ptr(), workspace.numel() * workspace.element_size(), opt(draft_lengths))


def tli_verify(ctx: int, args: tli_verify_args, stream: Optional[int] = None) -> None:
    """tli_verify() on ``stream`` (a cudaStream_t as int; default: torch's current stream)."""
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    rc = load().tli_verify(ctx, ctypes.byref(args), ctypes.c_void_p(stream))
    if rc != TLI_OK:
        raise TLIError(rc, "tli_verify")


def tli_verify_static(ctx: int, args: tli_verify_args, stream: Optional[int] = None) -> None:
    """tli_verify_static(): like tli_verify() but on the library's built-in 4 MiB scratch.

    For callers that cannot allocate device memory when they need to verify (all HBM already
    committed, or an allocation would stall the device).  ``args.workspace`` is ignored.  Calls
    that overlap on the GPU share the scratch and must be ordered by the caller."""
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    rc = load().tli_verify_static(ctx, ctypes.byref(args), ctypes.c_void_p(stream))
    if rc != TLI_OK:
        raise TLIError(rc, "tli_verify_static")


def tli_verify_host_buffer_bytes(ctx: int, B: int, K: int, dtype: int) -> int:
    return int(load().tli_verify_host_buffer_bytes(ctx, B, K, dtype))


def make_host_args(target_logits: torch.Tensor, drafter_logits: torch.Tensor, draft_ids: torch.Tensor,
                   temperature: torch.Tensor, uniforms: torch.Tensor, accepted: torch.Tensor, next_token: torch.Tensor,
                   device_buffer: torch.Tensor, row_status: Optional[torch.Tensor] = None) -> tli_verify_host_args:
    """Fill a tli_verify_host_args: contiguous CPU tensors (pinned for an asynchronous call) and a device buffer."""
    B, K1, _ = target_logits.shape
    for t in (target_logits, drafter_logits, draft_ids, temperature, uniforms, accepted, next_token):
        if t.is_cuda or not t.is_contiguous():
            raise ValueError("host tensors must be contiguous CPU tensors")
    return tli_verify_host_args(B, K1 - 1, _logit_dtype(target_logits), target_logits.data_ptr(), drafter_logits.data_ptr(),
                                draft_ids.data_ptr(), temperature.data_ptr(), uniforms.data_ptr(),
                                accepted.data_ptr(), next_token.data_ptr(),
                                None if row_status is None else row_status.data_ptr(),
                                device_buffer.data_ptr(), device_buffer.numel() * device_buffer.element_size())


def tli_verify_host(ctx: int, args: tli_verify_host_args, stream: Optional[int] = None) -> None:
    """tli_verify_host() on ``stream``; the outputs are valid after the stream has been synchronised."""
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    rc = load().tli_verify_host(ctx, ctypes.byref(args), ctypes.c_void_p(stream))
    if rc != TLI_OK:
        raise TLIError(rc, "tli_verify_host")


def tli_rates_workspace_bytes(ctx: int, B: int, K: int, dtype: int) -> int:
    return int(load().tli_rates_workspace_bytes(ctx, B, K, dtype))


def make_rates_args(target_logits: torch.Tensor, drafter_logits: torch.Tensor, temperature: torch.Tensor,
                    mass: torch.Tensor, alpha_union: torch.Tensor, alpha_tli: torch.Tensor, workspace: torch.Tensor,
                    position_status: Optional[torch.Tensor] = None) -> tli_rates_args:
    """Fill a tli_rates_args from device tensors (no copies; the tensors must outlive the call)."""
    B, K, _ = drafter_logits.shape
    dt = _logit_dtype(target_logits)
    if _logit_dtype(drafter_logits) != dt:
        raise TypeError("both logit tensors must have the same dtype")
    if target_logits.stride(2) != 1 or drafter_logits.stride(2) != 1:
        raise ValueError("the vocabulary axis must be contiguous")
    if target_logits.shape[0] != B or target_logits.shape[1] < K:
        raise ValueError("target logits must be [B, >=K, V_t]")
    for name, t in (("mass", mass), ("alpha_union", alpha_union), ("alpha_tli", alpha_tli)):
        if t.dtype != torch.float32 or tuple(t.shape) != (B, K) or not t.is_contiguous():
            raise ValueError("%s must be a contiguous float32 tensor of shape %s" % (name, (B, K)))
    return tli_rates_args(B, K, dt, target_logits.data_ptr(), target_logits.stride(0), target_logits.stride(1),
                          drafter_logits.data_ptr(), drafter_logits.stride(0), drafter_logits.stride(1),
                          temperature.data_ptr(), mass.data_ptr(), alpha_union.data_ptr(), alpha_tli.data_ptr(),
                          None if position_status is None else position_status.data_ptr(),
                          workspace.data_ptr(), workspace.numel() * workspace.element_size())


def tli_acceptance_rates(ctx: int, args: tli_rates_args, stream: Optional[int] = None) -> None:
    """tli_acceptance_rates() on ``stream`` (a cudaStream_t as int; default: torch's current stream)."""
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    rc = load().tli_acceptance_rates(ctx, ctypes.byref(args), ctypes.c_void_p(stream))
    if rc != TLI_OK:
        raise TLIError(rc, "tli_acceptance_rates")


def tli_draft_workspace_bytes(ctx: int, B: int, R: int, dtype: int) -> int:
    return int(load().tli_draft_workspace_bytes(ctx, B, R, dtype))


def make_draft_args(drafter_logits: torch.Tensor, temperature: torch.Tensor, uniforms: torch.Tensor,
                    draft_ids: torch.Tensor, workspace: torch.Tensor, q_draft: Optional[torch.Tensor] = None,
                    draft_status: Optional[torch.Tensor] = None) -> tli_draft_args:
    """Fill a tli_draft_args from device tensors (no copies; the tensors must outlive the call)."""
    B, R, _ = drafter_logits.shape
    dt = _logit_dtype(drafter_logits)
    if drafter_logits.stride(2) != 1:
        raise ValueError("the vocabulary axis must be contiguous")
    for name, t, dtype, shape in (("temperature", temperature, torch.float32, (B,)),
                                  ("uniforms", uniforms, torch.float32, (B, R)),
                                  ("draft_ids", draft_ids, torch.int32, (B, R))):
        if t.dtype != dtype or tuple(t.shape) != shape or not t.is_contiguous():
            raise ValueError("%s must be a contiguous %s tensor of shape %s" % (name, dtype, shape))
    opt = lambda t: None if t is None else t.data_ptr()
    return tli_draft_args(B, R, dt, drafter_logits.data_ptr(), drafter_logits.stride(0), drafter_logits.stride(1),
                          temperature.data_ptr(), uniforms.data_ptr(), draft_ids.data_ptr(), opt(q_draft),
                          opt(draft_status), workspace.data_ptr(), workspace.numel() * workspace.element_size())


def tli_draft_sample(ctx: int, args: tli_draft_args, stream: Optional[int] = None) -> None:
    """tli_draft_sample() on ``stream`` (a cudaStream_t as int; default: torch's current stream)."""
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    rc = load().tli_draft_sample(ctx, ctypes.byref(args), ctypes.c_void_p(stream))
    if rc != TLI_OK:
        raise TLIError(rc, "tli_draft_sample")


def tli_slem_workspace_bytes(ctx: int, B: int, M: int, dtype: int) -> int:
    return int(load().tli_slem_workspace_bytes(ctx, B, M, dtype))


def make_slem_args(target_logits: torch.Tensor, candidates: torch.Tensor, temperature: torch.Tensor,
                   uniforms: torch.Tensor, accepted: torch.Tensor, next_token: torch.Tensor, workspace: torch.Tensor,
                   lengths: Optional[torch.Tensor] = None, sampled: Optional[torch.Tensor] = None,
                   row_status: Optional[torch.Tensor] = None) -> tli_slem_args:
    """Fill a tli_slem_args from device tensors (no copies; the tensors must outlive the call)."""
    B, M1, _ = target_logits.shape
    M = M1 - 1
    dt = _logit_dtype(target_logits)
    if target_logits.stride(2) != 1:
        raise ValueError("the vocabulary axis must be contiguous")
    for name, t, dtype, shape in (("candidates", candidates, torch.int32, (B, M)),
                                  ("temperature", temperature, torch.float32, (B,)),
                                  ("uniforms", uniforms, torch.float32, (B, M + 1)),
                                  ("accepted", accepted, torch.int32, (B,)),
                                  ("next_token", next_token, torch.int32, (B,))):
        if t.dtype != dtype or tuple(t.shape) != shape or not t.is_contiguous():
            raise ValueError("%s must be a contiguous %s tensor of shape %s" % (name, dtype, shape))
    opt = lambda t: None if t is None else t.data_ptr()
    return tli_slem_args(B, M, dt, target_logits.data_ptr(), target_logits.stride(0), target_logits.stride(1),
                         candidates.data_ptr(), opt(lengths), temperature.data_ptr(), uniforms.data_ptr(),
                         accepted.data_ptr(), next_token.data_ptr(), opt(sampled), opt(row_status),
                         workspace.data_ptr(), workspace.numel() * workspace.element_size())


def tli_slem_verify(ctx: int, args: tli_slem_args, stream: Optional[int] = None) -> None:
    """tli_slem_verify() on ``stream`` (a cudaStream_t as int; default: torch's current stream)."""
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    rc = load().tli_slem_verify(ctx, ctypes.byref(args), ctypes.c_void_p(stream))
    if rc != TLI_OK:
        raise TLIError(rc, "tli_slem_verify")


def tli_verify_profile(ctx: int, args: tli_verify_args, stream: Optional[int] = None):
    """tli_verify_profile(): blocks; returns ms of (statistics kernel, decision kernel or 0, sampling kernel)."""
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    ms = (ctypes.c_float * 3)()
    rc = load().tli_verify_profile(ctx, ctypes.byref(args), ctypes.c_void_p(stream), ms)
    if rc != TLI_OK:
        raise TLIError(rc, "tli_verify_profile")
    return ms[0], ms[1], ms[2]


def tli_set_max_cluster(ctx: int, ctas: int) -> None:
    """tli_set_max_cluster(): widest cluster of the cluster kernel, 8 (portable) or 16 (where the device places it)."""
    rc = load().tli_set_max_cluster(ctx, int(ctas))
    if rc != TLI_OK:
        raise TLIError(rc, "tli_set_max_cluster")


def tli_set_tiled(ctx: int, enabled: bool) -> None:
    """tli_set_tiled(): the extra token by size (default) or always by the tile kernels."""
    rc = load().tli_set_tiled(ctx, 1 if enabled else 0)
    if rc != TLI_OK:
        raise TLIError(rc, "tli_set_tiled")


def tli_shard_create(device: int, V_t: int, V_d: int, id_map, n_shards: int, shard: int) -> int:
    """tli_shard_create(): the context of shard ``shard`` of ``n_shards``; returns the handle (an int)."""
    m = np.ascontiguousarray(id_map, dtype=np.int32)
    if m.shape != (V_d,):
        raise ValueError("id_map must have V_d entries")
    ctx = ctypes.c_void_p()
    rc = load().tli_shard_create(ctypes.byref(ctx), device, V_t, V_d, m.ctypes.data_as(ctypes.c_void_p), n_shards, shard)
    if rc != TLI_OK:
        raise TLIError(rc, "tli_shard_create")
    return ctx.value


def tli_shard_info(ctx: int) -> Dict[str, int]:
    """tli_shard_info(): the id ranges of a shard's context."""
    v = [ctypes.c_int32() for _ in range(6)]
    rc = load().tli_shard_info(ctx, *[ctypes.byref(x) for x in v])
    if rc != TLI_OK:
        raise TLIError(rc, "tli_shard_info")
    return dict(zip(("t_begin", "t_count", "d_begin", "d_count", "t_width", "d_width"), (x.value for x in v)))


def _shard_call(name: str, ctx: int, args: tli_verify_args, *buffers: torch.Tensor, stream: Optional[int] = None) -> None:
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    rc = getattr(load(), name)(ctx, ctypes.byref(args), *[ctypes.c_void_p(b.data_ptr()) for b in buffers], ctypes.c_void_p(stream))
    if rc != TLI_OK:
        raise TLIError(rc, name)


def tli_shard_stats(ctx: int, args: tli_verify_args, record: torch.Tensor, stream: Optional[int] = None) -> None:
    """tli_shard_stats(): this shard's statistics record."""
    _shard_call("tli_shard_stats", ctx, args, record, stream=stream)


def tli_shard_decide(ctx: int, args: tli_verify_args, records_all: torch.Tensor, rows: torch.Tensor,
                     stream: Optional[int] = None) -> None:
    """tli_shard_decide(): the decisions from all shards' records; packs this shard's slices of drafter row n."""
    _shard_call("tli_shard_decide", ctx, args, records_all, rows, stream=stream)


def tli_shard_weights(ctx: int, args: tli_verify_args, rows_all: torch.Tensor, mass: torch.Tensor,
                      stream: Optional[int] = None) -> None:
    """tli_shard_weights(): tile sums and totals of the extra token's weights over this shard's target ids."""
    _shard_call("tli_shard_weights", ctx, args, rows_all, mass, stream=stream)


def tli_shard_select(ctx: int, args: tli_verify_args, rows_all: torch.Tensor, masses_all: torch.Tensor,
                     stream: Optional[int] = None) -> None:
    """tli_shard_select(): the extra token on the shard that holds it, -1 elsewhere."""
    _shard_call("tli_shard_select", ctx, args, rows_all, masses_all, stream=stream)


def tli_verify_plan(ctx: int, B: int, K: int, dtype: int) -> Dict[str, int]:
    """tli_verify_plan(): how a batch of this shape will be run."""
    plan = (ctypes.c_int32 * 8)()
    rc = load().tli_verify_plan(ctx, B, K, dtype, plan)
    if rc != TLI_OK:
        raise TLIError(rc, "tli_verify_plan")
    return dict(zip(("launches", "cluster", "stats_ctas", "stage_bytes", "segment_bytes", "segments_per_target_row",
                     "segments_per_drafter_row", "cluster_smem_bytes"), plan))


def tli_launch_probe(ctx: int, B: int, K: int, dtype: int, stream: Optional[int] = None) -> None:
    """tli_launch_probe(): the launches of one call with kernels that do nothing."""
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    rc = load().tli_launch_probe(ctx, B, K, dtype, ctypes.c_void_p(stream))
    if rc != TLI_OK:
        raise TLIError(rc, "tli_launch_probe")


def tli_reset(ctx: int, stream: Optional[int] = None) -> None:
    """tli_reset(): the context's counters and its sticky time-out word back to zero, in stream order."""
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    rc = load().tli_reset(ctx, ctypes.c_void_p(stream))
    if rc != TLI_OK:
        raise TLIError(rc, "tli_reset")


def tli_selftest_bounded_wait(ctx: int, polls: int = 2000, stream: Optional[int] = None) -> bool:
    """tli_selftest_bounded_wait(): True if a wait on a barrier nothing completes gave up after `polls` polls."""
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    out = ctypes.c_int(0)
    rc = load().tli_selftest_bounded_wait(ctx, ctypes.c_void_p(stream), polls, ctypes.byref(out))
    if rc != TLI_OK:
        raise TLIError(rc, "tli_selftest_bounded_wait")
    return out.value == 1


class Verifier:
    """Convenience owner of one context plus its scratch and output tensors."""

    def __init__(self, V_t: int, V_d: int, id_map, device: int = 0, tiled: bool = False):
        self.device = torch.device("cuda", device)
        self.V_t, self.V_d = int(V_t), int(V_d)
        self.ctx = tli_create(device, V_t, V_d, id_map)
        if tiled:
            tli_set_tiled(self.ctx, True)
        self._ws: Optional[torch.Tensor] = None

    def close(self) -> None:
        if self.ctx:
            tli_destroy(self.ctx)
            self.ctx = 0

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def workspace(self, B: int, K: int, dtype: int) -> torch.Tensor:
        need = tli_workspace_bytes(self.ctx, B, K, dtype)
        if need == 0:
            raise TLIError(TLI_ERR_UNSUPPORTED, "tli_workspace_bytes")
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device=self.device)
        return self._ws

    def draft(self, drafter_logits, temperature, uniforms) -> Dict[str, torch.Tensor]:
        """Draw one drafter id per row of ``drafter_logits`` [B,R,V_d] from q'; returns device tensors."""
        B, R, _ = drafter_logits.shape
        dev = self.device
        out = {"draft_ids": torch.empty(B, R, dtype=torch.int32, device=dev),
               "q_draft": torch.empty(B, R, dtype=torch.float32, device=dev),
               "draft_status": torch.empty(B, R, dtype=torch.int32, device=dev)}
        need = tli_draft_workspace_bytes(self.ctx, B, R, _logit_dtype(drafter_logits))
        if need == 0:
            raise TLIError(TLI_ERR_UNSUPPORTED, "tli_draft_workspace_bytes")
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device=dev)
        args = make_draft_args(drafter_logits, temperature, uniforms, out["draft_ids"], self._ws,
                               out["q_draft"], out["draft_status"])
        tli_draft_sample(self.ctx, args)
        return out

    def rates(self, target_logits, drafter_logits, temperature) -> Dict[str, torch.Tensor]:
        """Expected acceptance rates per draft position (mass, alpha_union, alpha_tli); device tensors."""
        B, K, _ = drafter_logits.shape
        dev = self.device
        out = {k: torch.empty(B, K, dtype=torch.float32, device=dev) for k in ("mass", "alpha_union", "alpha_tli")}
        out["position_status"] = torch.empty(B, K, dtype=torch.int32, device=dev)
        need = tli_rates_workspace_bytes(self.ctx, B, K, _logit_dtype(target_logits))
        if need == 0:
            raise TLIError(TLI_ERR_UNSUPPORTED, "tli_rates_workspace_bytes")
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device=dev)
        args = make_rates_args(target_logits, drafter_logits, temperature, out["mass"], out["alpha_union"],
                               out["alpha_tli"], self._ws, out["position_status"])
        tli_acceptance_rates(self.ctx, args)
        return out

    def slem(self, target_logits, candidates, temperature, uniforms, lengths=None) -> Dict[str, torch.Tensor]:
        """Exact-match verification of re-tokenised drafts ``candidates`` [B,M] against tokens sampled
        from ``target_logits`` [B,M+1,V_t]; returns device tensors."""
        B, M1, _ = target_logits.shape
        dev = self.device
        out = {"accepted": torch.empty(B, dtype=torch.int32, device=dev),
               "next_token": torch.empty(B, dtype=torch.int32, device=dev),
               "sampled": torch.empty(B, M1, dtype=torch.int32, device=dev),
               "row_status": torch.empty(B, dtype=torch.int32, device=dev)}
        need = tli_slem_workspace_bytes(self.ctx, B, M1 - 1, _logit_dtype(target_logits))
        if need == 0:
            raise TLIError(TLI_ERR_UNSUPPORTED, "tli_slem_workspace_bytes")
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device=dev)
        args = make_slem_args(target_logits, candidates, temperature, uniforms, out["accepted"], out["next_token"],
                              self._ws, lengths, out["sampled"], out["row_status"])
        tli_slem_verify(self.ctx, args)
        return out

    def verify(self, target_logits, drafter_logits, draft_ids, temperature, uniforms,
               diagnostics: bool = True, draft_lengths=None) -> Dict[str, torch.Tensor]:
        """One call on torch's current stream; returns device tensors (no synchronisation)."""
        B, K1, _ = target_logits.shape
        K = K1 - 1
        dev = self.device
        out = {"accepted": torch.empty(B, dtype=torch.int32, device=dev),
               "next_token": torch.empty(B, dtype=torch.int32, device=dev),
               "row_status": torch.empty(B, dtype=torch.int32, device=dev)}
        if diagnostics:
            out["p_draft"] = torch.empty(B, K, dtype=torch.float32, device=dev)
            out["q_draft"] = torch.empty(B, K, dtype=torch.float32, device=dev)
        ws = self.workspace(B, K, _logit_dtype(target_logits))
        args = make_args(target_logits, drafter_logits, draft_ids, temperature, uniforms,
                         out["accepted"], out["next_token"], ws, out["row_status"],
                         out.get("p_draft"), out.get("q_draft"), draft_lengths)
        tli_verify(self.ctx, args)
        return out
