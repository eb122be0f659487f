"""Thin ctypes binding of ``libsgbv.so`` (declared in ``include/sgbv.h``).

Argument marshalling only: every step of the verify path runs in the CUDA kernels behind the C
ABI.  torch supplies device memory and the current stream.  There is no fallback of any kind: a
missing library or a non-CUDA tensor raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

from . import build as _build

OK = 0
STATUS_TOKEN_RANGE = 1
STATUS_NONFINITE_LOGIT = 2
STATUS_DEGENERATE_RESIDUAL = 4
STATUS_TIMEOUT = 8
DTYPE_F32 = 0
DTYPE_BF16 = 1

EXPORTS = ("sgbv_workspace_bytes", "sgbv_verify", "sgbv_verify_bf16", "sgbv_verify_ex",
           "sgbv_verify_host", "sgbv_last_launch_count", "sgbv_last_main_kernel", "sgbv_status_string",
           "sgbv_profile_begin",
           "sgbv_profile_end", "sgbv_verify_static", "sgbv_set_option", "sgbv_modify", "sgbv_verify_kseq",
           "sgbv_verify_token", "sgbv_verify_gbv", "sgbv_draw_tokens", "sgbv_shard_workspace_bytes",
           "sgbv_shard_stats", "sgbv_shard_sums", "sgbv_shard_decide", "sgbv_shard_draw")

_lib = None


class SgbvError(RuntimeError):
    def __init__(self, code: int):
        self.code = code
        super().__init__(status_string(code))


def lib_path() -> str:
    return _build.LIB


def load() -> ctypes.CDLL:
    """Load the in-tree CUDA library; raises if it has not been built."""
    global _lib
    if _lib is None:
        path = lib_path()
        if not os.path.exists(path):
            raise RuntimeError(f"{path} is missing: build it with `python -m paper_2604_25925_b200.build` "
                               "(there is no CPU fallback)")
        lib = ctypes.CDLL(path)
        vp, i32, f32, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
        lib.sgbv_workspace_bytes.restype = i32
        lib.sgbv_workspace_bytes.argtypes = [i32, i32, i32, i32, i32, ctypes.POINTER(sz)]
        dev_args = [vp, vp, vp, vp, i32, i32, i32, i32, f32, vp, vp, vp, vp]
        lib.sgbv_verify.restype = i32
        lib.sgbv_verify.argtypes = dev_args
        lib.sgbv_verify_bf16.restype = i32
        lib.sgbv_verify_bf16.argtypes = dev_args
        lib.sgbv_verify_ex.restype = i32
        lib.sgbv_verify_ex.argtypes = [vp, vp, i32, vp, vp, i32, i32, i32, i32, f32, vp, vp, vp, vp, sz,
                                       vp, vp, vp, vp]
        lib.sgbv_verify_static.restype = i32
        lib.sgbv_verify_static.argtypes = [vp, vp, i32, vp, vp, i32, i32, i32, i32, f32, vp, vp, vp, vp, vp, vp, vp]
        lib.sgbv_verify_host.restype = i32
        lib.sgbv_verify_host.argtypes = [vp, vp, i32, vp, vp, i32, i32, i32, i32, f32, vp, vp, vp, vp, vp]
        lib.sgbv_modify.restype = i32
        lib.sgbv_modify.argtypes = [vp, vp, i32, vp, vp, vp, i32, i32, i32, f32, vp, vp, vp, vp, vp, vp, sz, vp]
        lib.sgbv_verify_kseq.restype = i32
        lib.sgbv_verify_kseq.argtypes = [vp, vp, i32, vp, vp, i32, i32, i32, i32, f32, vp, vp, vp, vp, vp, vp, sz, vp]
        for fn in (lib.sgbv_verify_token, lib.sgbv_verify_gbv):
            fn.restype = i32
            fn.argtypes = [vp, vp, i32, vp, vp, i32, i32, i32, f32, vp, vp, vp, vp, vp, sz, vp]
        lib.sgbv_draw_tokens.restype = i32
        lib.sgbv_draw_tokens.argtypes = [vp, i32, vp, i32, i32, f32, vp, vp, vp, vp, sz, vp]
        lib.sgbv_shard_workspace_bytes.restype = i32
        lib.sgbv_shard_workspace_bytes.argtypes = [i32, i32, i32, i32, i32, ctypes.POINTER(sz)]
        lib.sgbv_shard_stats.restype = i32
        lib.sgbv_shard_stats.argtypes = [vp, vp, i32, vp, i32, i32, i32, i32, i32, i32, f32, vp, vp]
        lib.sgbv_shard_sums.restype = i32
        lib.sgbv_shard_sums.argtypes = [vp, vp, i32, i32, i32, i32, i32, f32, vp, i32, vp, sz, vp, vp]
        lib.sgbv_shard_decide.restype = i32
        lib.sgbv_shard_decide.argtypes = [vp, vp, i32, i32, i32, i32, f32, vp, vp, i32, vp, sz, vp, vp, vp, vp, vp, vp, vp]
        lib.sgbv_shard_draw.restype = i32
        lib.sgbv_shard_draw.argtypes = [vp, vp, i32, i32, i32, i32, i32, i32, f32, i32, vp, sz, vp, vp]
        lib.sgbv_last_launch_count.restype = i32
        lib.sgbv_last_launch_count.argtypes = []
        lib.sgbv_last_main_kernel.restype = ctypes.c_char_p
        lib.sgbv_last_main_kernel.argtypes = []
        lib.sgbv_profile_begin.restype = i32
        lib.sgbv_profile_begin.argtypes = [i32]
        lib.sgbv_profile_end.restype = i32
        lib.sgbv_profile_end.argtypes = [ctypes.POINTER(ctypes.c_double), ctypes.POINTER(i32)]
        lib.sgbv_set_option.restype = i32
        lib.sgbv_set_option.argtypes = [ctypes.c_char_p, i32]
        lib.sgbv_status_string.restype = ctypes.c_char_p
        lib.sgbv_status_string.argtypes = [i32]
        _lib = lib
    return _lib


def status_string(code: int) -> str:
    return load().sgbv_status_string(int(code)).decode()


def last_launch_count() -> int:
    return int(load().sgbv_last_launch_count())


def set_option(name: str, value: int) -> None:
    """Tuning knob for experiments (see include/sgbv.h); 0 restores the automatic choice."""
    rc = load().sgbv_set_option(name.encode(), int(value))
    if rc != OK:
        raise SgbvError(rc)


def last_main_kernel() -> str:
    return load().sgbv_last_main_kernel().decode()


def profile_begin(max_records: int) -> None:
    rc = load().sgbv_profile_begin(int(max_records))
    if rc != OK:
        raise SgbvError(rc)


def profile_end():
    """-> (summed milliseconds of the dominant kernel, number of recorded calls)."""
    ms, n = ctypes.c_double(0.0), ctypes.c_int(0)
    rc = load().sgbv_profile_end(ctypes.byref(ms), ctypes.byref(n))
    if rc != OK:
        raise SgbvError(rc)
    return ms.value, n.value


def workspace_bytes(B: int, K: int, gamma: int, V: int, dtype: int = DTYPE_F32) -> int:
    out = ctypes.c_size_t(0)
    rc = load().sgbv_workspace_bytes(B, K, gamma, V, dtype, ctypes.byref(out))
    if rc != OK:
        raise SgbvError(rc)
    return int(out.value)


@dataclass
class VerifyOutput:
    accept_len: torch.Tensor            # [B] int32
    draft_idx: torch.Tensor             # [B] int32
    tokens: torch.Tensor                # [B, gamma+1] int32
    h: Optional[torch.Tensor] = None        # [B,K,gamma] float64
    resmass: Optional[torch.Tensor] = None  # [B,K,gamma] float64
    status: Optional[torch.Tensor] = None   # [B] int32


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return DTYPE_F32
    if t.dtype == torch.bfloat16:
        return DTYPE_BF16
    raise TypeError(f"logits must be float32 or bfloat16, got {t.dtype}")


def _shapes(target_logits, draft_logits, draft_tokens, uniforms):
    B, K, g1, V = target_logits.shape
    gamma = g1 - 1
    if tuple(draft_logits.shape) != (B, K, gamma, V):
        raise ValueError(f"draft_logits shape {tuple(draft_logits.shape)} != {(B, K, gamma, V)}")
    if tuple(draft_tokens.shape) != (B, K, gamma) or draft_tokens.dtype != torch.int32:
        raise ValueError("draft_tokens must be int32 [B,K,gamma]")
    if tuple(uniforms.shape) != (B, K * gamma + 1) or uniforms.dtype != torch.float32:
        raise ValueError("uniforms must be float32 [B,K*gamma+1]")
    if draft_logits.dtype != target_logits.dtype:
        raise TypeError("target and draft logits must have the same dtype")
    for t in (target_logits, draft_logits, draft_tokens, uniforms):
        if not t.is_contiguous():
            raise ValueError("inputs must be contiguous")
    return B, K, gamma, V


def sgbv_verify(target_logits, draft_logits, draft_tokens, uniforms, temperature: float = 1.0,
                out: Optional[VerifyOutput] = None) -> VerifyOutput:
    """Plain entry point (``sgbv_verify`` / ``sgbv_verify_bf16``) on CUDA tensors, current stream."""
    B, K, gamma, V = _shapes(target_logits, draft_logits, draft_tokens, uniforms)
    for t in (target_logits, draft_logits, draft_tokens, uniforms):
        if not t.is_cuda:
            raise ValueError("sgbv_verify takes CUDA tensors (use sgbv_verify_host for host buffers)")
    dev = target_logits.device
    if out is None:
        out = VerifyOutput(torch.empty(B, dtype=torch.int32, device=dev),
                           torch.empty(B, dtype=torch.int32, device=dev),
                           torch.empty((B, gamma + 1), dtype=torch.int32, device=dev))
    fn = load().sgbv_verify if _dtype_code(target_logits) == DTYPE_F32 else load().sgbv_verify_bf16
    with torch.cuda.device(dev):
        rc = fn(target_logits.data_ptr(), draft_logits.data_ptr(), draft_tokens.data_ptr(),
                uniforms.data_ptr(), B, K, gamma, V, float(temperature), out.accept_len.data_ptr(),
                out.draft_idx.data_ptr(), out.tokens.data_ptr(), torch.cuda.current_stream(dev).cuda_stream)
    if rc != OK:
        raise SgbvError(rc)
    return out


def sgbv_verify_ex(target_logits, draft_logits, draft_tokens, uniforms, temperature: float = 1.0,
                   workspace: Optional[torch.Tensor] = None, diagnostics: bool = True,
                   out: Optional[VerifyOutput] = None) -> VerifyOutput:
    """Extended entry point: optional caller workspace (uint8 CUDA tensor) and diagnostics."""
    B, K, gamma, V = _shapes(target_logits, draft_logits, draft_tokens, uniforms)
    dev = target_logits.device
    if not target_logits.is_cuda:
        raise ValueError("sgbv_verify_ex takes CUDA tensors")
    if out is None:
        out = VerifyOutput(torch.empty(B, dtype=torch.int32, device=dev),
                           torch.empty(B, dtype=torch.int32, device=dev),
                           torch.empty((B, gamma + 1), dtype=torch.int32, device=dev))
    if diagnostics and out.h is None:
        out.h = torch.empty((B, K, gamma), dtype=torch.float64, device=dev)
        out.resmass = torch.empty((B, K, gamma), dtype=torch.float64, device=dev)
        out.status = torch.empty(B, dtype=torch.int32, device=dev)
    ws_ptr, ws_bytes = (workspace.data_ptr(), workspace.numel() * workspace.element_size()) \
        if workspace is not None else (None, 0)
    with torch.cuda.device(dev):
        rc = load().sgbv_verify_ex(
            target_logits.data_ptr(), draft_logits.data_ptr(), _dtype_code(target_logits),
            draft_tokens.data_ptr(), uniforms.data_ptr(), B, K, gamma, V, float(temperature),
            out.accept_len.data_ptr(), out.draft_idx.data_ptr(), out.tokens.data_ptr(), ws_ptr, ws_bytes,
            out.h.data_ptr() if out.h is not None else None,
            out.resmass.data_ptr() if out.resmass is not None else None,
            out.status.data_ptr() if out.status is not None else None,
            torch.cuda.current_stream(dev).cuda_stream)
    if rc != OK:
        raise SgbvError(rc)
    return out


STATIC_SCRATCH_BYTES = 32 * 1024 * 1024


def sgbv_verify_static(target_logits, draft_logits, draft_tokens, uniforms, temperature: float = 1.0,
                       out: Optional[VerifyOutput] = None) -> VerifyOutput:
    """Allocation-free entry point: scratch is the library's fixed device array, so the library
    itself never allocates.  For callers that cannot allocate device memory after start-up (all
    of it already belongs to their pool) or cannot take the device-wide stall of an allocation.
    Pass a pre-built ``out`` (with h, resmass, status tensors) to keep this wrapper from
    allocating too.  Shapes needing more than STATIC_SCRATCH_BYTES raise SGBV_ERR_WORKSPACE;
    calls that overlap on the GPU race on the shared scratch."""
    B, K, gamma, V = _shapes(target_logits, draft_logits, draft_tokens, uniforms)
    dev = target_logits.device
    if not target_logits.is_cuda:
        raise ValueError("sgbv_verify_static takes CUDA tensors")
    if out is None:
        out = VerifyOutput(torch.empty(B, dtype=torch.int32, device=dev),
                           torch.empty(B, dtype=torch.int32, device=dev),
                           torch.empty((B, gamma + 1), dtype=torch.int32, device=dev),
                           torch.empty((B, K, gamma), dtype=torch.float64, device=dev),
                           torch.empty((B, K, gamma), dtype=torch.float64, device=dev),
                           torch.empty(B, dtype=torch.int32, device=dev))
    with torch.cuda.device(dev):
        rc = load().sgbv_verify_static(
            target_logits.data_ptr(), draft_logits.data_ptr(), _dtype_code(target_logits),
            draft_tokens.data_ptr(), uniforms.data_ptr(), B, K, gamma, V, float(temperature),
            out.accept_len.data_ptr(), out.draft_idx.data_ptr(), out.tokens.data_ptr(),
            out.h.data_ptr() if out.h is not None else None,
            out.resmass.data_ptr() if out.resmass is not None else None,
            out.status.data_ptr() if out.status is not None else None,
            torch.cuda.current_stream(dev).cuda_stream)
    if rc != OK:
        raise SgbvError(rc)
    return out


def sgbv_verify_host(target_logits, draft_logits, draft_tokens, uniforms, temperature: float = 1.0,
                     out: Optional[VerifyOutput] = None, device: int = 0) -> VerifyOutput:
    """Host-buffer entry point: CPU tensors in (pinned for asynchronous copies), CPU tensors out.
    Returns after the stream has been synchronised."""
    B, K, gamma, V = _shapes(target_logits, draft_logits, draft_tokens, uniforms)
    for t in (target_logits, draft_logits, draft_tokens, uniforms):
        if t.is_cuda:
            raise ValueError("sgbv_verify_host takes host tensors")
    if out is None:
        out = VerifyOutput(torch.empty(B, dtype=torch.int32).pin_memory(),
                           torch.empty(B, dtype=torch.int32).pin_memory(),
                           torch.empty((B, gamma + 1), dtype=torch.int32).pin_memory(),
                           status=torch.empty(B, dtype=torch.int32).pin_memory())
    with torch.cuda.device(device):
        rc = load().sgbv_verify_host(
            target_logits.data_ptr(), draft_logits.data_ptr(), _dtype_code(target_logits),
            draft_tokens.data_ptr(), uniforms.data_ptr(), B, K, gamma, V, float(temperature),
            out.accept_len.data_ptr(), out.draft_idx.data_ptr(), out.tokens.data_ptr(),
            out.status.data_ptr() if out.status is not None else None,
            torch.cuda.current_stream(device).cuda_stream)
    if rc != OK:
        raise SgbvError(rc)
    return out


@dataclass
class ModifyOutput:
    token: torch.Tensor      # [B] int32
    log_a: torch.Tensor      # [B] float64 log q(s, token)
    log_b: torch.Tensor      # [B] float64 log p(s, token)
    resmass: torch.Tensor    # [B] float64 normaliser over q(s)
    status: torch.Tensor     # [B] int32


def sgbv_modify(target_logits, draft_logits, log_a, log_b, uniforms, K: int, temperature: float = 1.0,
                workspace: Optional[torch.Tensor] = None) -> ModifyOutput:
    """One position of Algorithm 2 per batch row: target/draft logits [B,V], carried joint logs [B] (float64),
    uniforms [B]; returns the drawn tokens and the carried logs with them appended."""
    B, V = target_logits.shape
    if tuple(draft_logits.shape) != (B, V) or draft_logits.dtype != target_logits.dtype:
        raise ValueError("draft_logits must match target_logits")
    for t, dt in ((log_a, torch.float64), (log_b, torch.float64), (uniforms, torch.float32)):
        if tuple(t.shape) != (B,) or t.dtype != dt or not t.is_cuda or not t.is_contiguous():
            raise ValueError("log_a, log_b must be float64 [B], uniforms float32 [B], CUDA, contiguous")
    if not (target_logits.is_cuda and target_logits.is_contiguous() and draft_logits.is_contiguous()):
        raise ValueError("logits must be contiguous CUDA tensors")
    dev = target_logits.device
    out = ModifyOutput(torch.empty(B, dtype=torch.int32, device=dev), torch.empty(B, dtype=torch.float64, device=dev),
                       torch.empty(B, dtype=torch.float64, device=dev), torch.empty(B, dtype=torch.float64, device=dev),
                       torch.empty(B, dtype=torch.int32, device=dev))
    ws_ptr, ws_bytes = (workspace.data_ptr(), workspace.numel() * workspace.element_size()) \
        if workspace is not None else (None, 0)
    with torch.cuda.device(dev):
        rc = load().sgbv_modify(target_logits.data_ptr(), draft_logits.data_ptr(), _dtype_code(target_logits),
                                log_a.data_ptr(), log_b.data_ptr(), uniforms.data_ptr(), B, int(K), V,
                                float(temperature), out.token.data_ptr(), out.log_a.data_ptr(), out.log_b.data_ptr(),
                                out.resmass.data_ptr(), out.status.data_ptr(), ws_ptr, ws_bytes,
                                torch.cuda.current_stream(dev).cuda_stream)
    if rc != OK:
        raise SgbvError(rc)
    return out


@dataclass
class PositionwiseOutput:
    accept_len: torch.Tensor            # [B] int32
    tokens: torch.Tensor                # [B, gamma+1] int32
    rho: Optional[torch.Tensor]         # [B, gamma] float64 (K-SEQ only)
    accept_prob: torch.Tensor           # [B, K, gamma] float64 (NaN where a token was not tried)
    status: torch.Tensor                # [B] int32


def sgbv_verify_kseq(target_logits, draft_logits, draft_tokens, uniforms, temperature: float = 1.0) -> PositionwiseOutput:
    """SpecTr's K-SEQ on the verify step's tensors ([B,K,gamma+1,V], [B,K,gamma,V], [B,K,gamma], [B,K*gamma+1])."""
    B, K, gamma, V = _shapes(target_logits, draft_logits, draft_tokens, uniforms)
    dev = target_logits.device
    out = PositionwiseOutput(torch.empty(B, dtype=torch.int32, device=dev),
                             torch.empty((B, gamma + 1), dtype=torch.int32, device=dev),
                             torch.empty((B, gamma), dtype=torch.float64, device=dev),
                             torch.empty((B, K, gamma), dtype=torch.float64, device=dev),
                             torch.empty(B, dtype=torch.int32, device=dev))
    with torch.cuda.device(dev):
        rc = load().sgbv_verify_kseq(target_logits.data_ptr(), draft_logits.data_ptr(), _dtype_code(target_logits),
                                     draft_tokens.data_ptr(), uniforms.data_ptr(), B, K, gamma, V, float(temperature),
                                     out.accept_len.data_ptr(), out.tokens.data_ptr(), out.rho.data_ptr(),
                                     out.accept_prob.data_ptr(), out.status.data_ptr(), None, 0,
                                     torch.cuda.current_stream(dev).cuda_stream)
    if rc != OK:
        raise SgbvError(rc)
    return out


def _single_draft(name, target_logits, draft_logits, draft_tokens, uniforms, temperature):
    B, g1, V = target_logits.shape
    gamma = g1 - 1
    if tuple(draft_logits.shape) != (B, gamma, V) or tuple(draft_tokens.shape) != (B, gamma) or \
            tuple(uniforms.shape) != (B, gamma + 1):
        raise ValueError("single-draft tensors: target [B,gamma+1,V], draft [B,gamma,V], tokens [B,gamma], uniforms [B,gamma+1]")
    dev = target_logits.device
    out = PositionwiseOutput(torch.empty(B, dtype=torch.int32, device=dev),
                             torch.empty((B, gamma + 1), dtype=torch.int32, device=dev), None,
                             torch.empty((B, 1, gamma), dtype=torch.float64, device=dev),
                             torch.empty(B, dtype=torch.int32, device=dev))
    with torch.cuda.device(dev):
        rc = getattr(load(), name)(target_logits.data_ptr(), draft_logits.data_ptr(), _dtype_code(target_logits),
                                   draft_tokens.data_ptr(), uniforms.data_ptr(), B, gamma, V, float(temperature),
                                   out.accept_len.data_ptr(), out.tokens.data_ptr(), out.accept_prob.data_ptr(),
                                   out.status.data_ptr(), None, 0, torch.cuda.current_stream(dev).cuda_stream)
    if rc != OK:
        raise SgbvError(rc)
    return out


def sgbv_verify_token(target_logits, draft_logits, draft_tokens, uniforms, temperature: float = 1.0) -> PositionwiseOutput:
    """Token-level speculative sampling, one draft per batch row."""
    return _single_draft("sgbv_verify_token", target_logits, draft_logits, draft_tokens, uniforms, temperature)


def sgbv_verify_gbv(target_logits, draft_logits, draft_tokens, uniforms, temperature: float = 1.0) -> PositionwiseOutput:
    """Single-draft greedy block verification (the block verifier with K = 1)."""
    return _single_draft("sgbv_verify_gbv", target_logits, draft_logits, draft_tokens, uniforms, temperature)


def sgbv_draw_tokens(logits, uniforms, temperature: float = 1.0):
    """One token per row of logits [N,V] from softmax(logits/T) by inverse CDF. -> (tokens int32 [N], logprob float64 [N],
    status int32 [N])"""
    N, V = logits.shape
    if tuple(uniforms.shape) != (N,) or uniforms.dtype != torch.float32 or not (logits.is_cuda and uniforms.is_cuda):
        raise ValueError("uniforms must be float32 [N] on the device of the logits")
    if not logits.is_contiguous():
        raise ValueError("logits must be contiguous")
    dev = logits.device
    tok = torch.empty(N, dtype=torch.int32, device=dev)
    lp = torch.empty(N, dtype=torch.float64, device=dev)
    st = torch.empty(N, dtype=torch.int32, device=dev)
    with torch.cuda.device(dev):
        rc = load().sgbv_draw_tokens(logits.data_ptr(), _dtype_code(logits), uniforms.data_ptr(), N, V, float(temperature),
                                     tok.data_ptr(), lp.data_ptr(), st.data_ptr(), None, 0,
                                     torch.cuda.current_stream(dev).cuda_stream)
    if rc != OK:
        raise SgbvError(rc)
    return tok, lp, st


# ---- vocabulary-sharded verify step: the four local phases (the exchanges between them are the caller's) ----------

def _shard_shapes(target_shard, draft_shard):
    B, K, g1, Vs = target_shard.shape
    gamma = g1 - 1
    if tuple(draft_shard.shape) != (B, K, gamma, Vs) or draft_shard.dtype != target_shard.dtype:
        raise ValueError(f"draft shard must be {(B, K, gamma, Vs)} of the target shard's dtype")
    if not (target_shard.is_cuda and draft_shard.is_cuda and target_shard.is_contiguous() and draft_shard.is_contiguous()):
        raise ValueError("shards must be contiguous CUDA tensors")
    return B, K, gamma, Vs


def sgbv_shard_workspace_bytes(B: int, K: int, gamma: int, shard_V: int, dtype: int = DTYPE_F32) -> int:
    out = ctypes.c_size_t(0)
    rc = load().sgbv_shard_workspace_bytes(B, K, gamma, shard_V, dtype, ctypes.byref(out))
    if rc != OK:
        raise SgbvError(rc)
    return int(out.value)


def sgbv_shard_stats(target_shard, draft_shard, draft_tokens, v_begin: int, V: int, temperature: float) -> torch.Tensor:
    """-> this shard's statistics records, float32 [B,K,gamma+1,8]."""
    B, K, gamma, Vs = _shard_shapes(target_shard, draft_shard)
    dev = target_shard.device
    out = torch.empty((B, K, gamma + 1, 8), dtype=torch.float32, device=dev)
    with torch.cuda.device(dev):
        rc = load().sgbv_shard_stats(target_shard.data_ptr(), draft_shard.data_ptr(), _dtype_code(target_shard),
                                     draft_tokens.data_ptr(), B, K, gamma, Vs, int(v_begin), int(V), float(temperature),
                                     out.data_ptr(), torch.cuda.current_stream(dev).cuda_stream)
    if rc != OK:
        raise SgbvError(rc)
    return out


def sgbv_shard_sums(target_shard, draft_shard, temperature: float, stats_all, workspace) -> torch.Tensor:
    """stats_all: float32 [n_ranks,B,K,gamma+1,8] in rank order. -> this shard's row sums, float64 [B,K,gamma,3]."""
    B, K, gamma, Vs = _shard_shapes(target_shard, draft_shard)
    dev = target_shard.device
    if tuple(stats_all.shape[1:]) != (B, K, gamma + 1, 8) or stats_all.dtype != torch.float32 or not stats_all.is_contiguous():
        raise ValueError("stats_all must be contiguous float32 [n_ranks,B,K,gamma+1,8]")
    out = torch.empty((B, K, gamma, 3), dtype=torch.float64, device=dev)
    with torch.cuda.device(dev):
        rc = load().sgbv_shard_sums(target_shard.data_ptr(), draft_shard.data_ptr(), _dtype_code(target_shard), B, K, gamma,
                                    Vs, float(temperature), stats_all.data_ptr(), int(stats_all.shape[0]),
                                    workspace.data_ptr(), workspace.numel(), out.data_ptr(),
                                    torch.cuda.current_stream(dev).cuda_stream)
    if rc != OK:
        raise SgbvError(rc)
    return out


def sgbv_shard_decide(draft_tokens, uniforms, shard_V: int, temperature: float, stats_all, sums_all, workspace) -> VerifyOutput:
    """Decisions from the gathered sums (identical on every rank); tokens hold the accepted prefix, -1 elsewhere."""
    B, K, gamma = draft_tokens.shape
    dev = draft_tokens.device
    if tuple(sums_all.shape[1:]) != (B, K, gamma, 3) or sums_all.dtype != torch.float64 or not sums_all.is_contiguous() \
            or sums_all.shape[0] != stats_all.shape[0]:
        raise ValueError("sums_all must be contiguous float64 [n_ranks,B,K,gamma,3]")
    if tuple(uniforms.shape) != (B, K * gamma + 1) or uniforms.dtype != torch.float32 or draft_tokens.dtype != torch.int32:
        raise ValueError("draft_tokens int32 [B,K,gamma], uniforms float32 [B,K*gamma+1]")
    out = VerifyOutput(torch.empty(B, dtype=torch.int32, device=dev), torch.empty(B, dtype=torch.int32, device=dev),
                       torch.empty((B, gamma + 1), dtype=torch.int32, device=dev),
                       torch.empty((B, K, gamma), dtype=torch.float64, device=dev),
                       torch.empty((B, K, gamma), dtype=torch.float64, device=dev),
                       torch.empty(B, dtype=torch.int32, device=dev))
    with torch.cuda.device(dev):
        rc = load().sgbv_shard_decide(draft_tokens.data_ptr(), uniforms.data_ptr(), B, K, gamma, int(shard_V),
                                      float(temperature), stats_all.data_ptr(), sums_all.data_ptr(), int(stats_all.shape[0]),
                                      workspace.data_ptr(), workspace.numel(), out.accept_len.data_ptr(),
                                      out.draft_idx.data_ptr(), out.tokens.data_ptr(), out.h.data_ptr(),
                                      out.resmass.data_ptr(), out.status.data_ptr(),
                                      torch.cuda.current_stream(dev).cuda_stream)
    if rc != OK:
        raise SgbvError(rc)
    return out


def sgbv_shard_draw(target_shard, draft_shard, v_begin: int, temperature: float, rank: int, workspace, tokens) -> None:
    """The owning rank writes the extra token's global id into tokens[b, accept_len] (in place)."""
    B, K, gamma, Vs = _shard_shapes(target_shard, draft_shard)
    dev = target_shard.device
    with torch.cuda.device(dev):
        rc = load().sgbv_shard_draw(target_shard.data_ptr(), draft_shard.data_ptr(), _dtype_code(target_shard), B, K, gamma,
                                    Vs, int(v_begin), float(temperature), int(rank), workspace.data_ptr(), workspace.numel(),
                                    tokens.data_ptr(), torch.cuda.current_stream(dev).cuda_stream)
    if rc != OK:
        raise SgbvError(rc)
