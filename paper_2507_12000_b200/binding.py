"""Thin Python binding of libdssd.so (see include/dssd.h for the contract of every call).

Only argument marshalling happens here: torch tensors supply device memory and the CUDA
stream; every step of the verification round runs inside the library's kernels.  There is no
CPU path: if the library cannot be loaded the import fails.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libdssd.so")

DSSD_OK = 0
DSSD_ERR_INVALID_ARG = 1
DSSD_ERR_UNSUPPORTED = 2
DSSD_ERR_WORKSPACE = 3
DSSD_ERR_CUDA = 4
DSSD_F32 = 0
DSSD_BF16 = 1

EDGE_FLAG_BAD_TOKEN = 1
EDGE_FLAG_NONFINITE = 2
EDGE_FLAG_TIMEOUT = 4
RS_FLAG_BONUS = 1
RS_FLAG_FALLBACK = 2
RS_FLAG_INVALID = 4
RS_FLAG_TIMEOUT = 8


class DssdError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        name = lib.dssd_status_string(status).decode()
        extra = f" (cudaError {lib.dssd_last_cuda_error()})" if status == DSSD_ERR_CUDA else ""
        super().__init__(f"{where}: {name}{extra}")


def _load(path: Optional[str] = None) -> ctypes.CDLL:
    path = path or LIB_PATH
    if not os.path.exists(path):
        raise ImportError(
            f"{path} is missing: build it with `python -m paper_2507_12000_b200.build` "
            "(needs nvcc); this package has no CPU fallback")
    c = ctypes
    L = c.CDLL(path)
    L.dssd_status_string.restype = c.c_char_p
    L.dssd_status_string.argtypes = [c.c_int]
    L.dssd_version.restype = c.c_int
    L.dssd_last_cuda_error.restype = c.c_int
    for f in (L.dssd_edge_verify_workspace_bytes, L.dssd_device_resample_workspace_bytes):
        f.restype = c.c_size_t
        f.argtypes = [c.c_int, c.c_int, c.c_int]
    L.dssd_round_host_arena_bytes.restype = c.c_size_t
    L.dssd_round_host_arena_bytes.argtypes = [c.c_int, c.c_int, c.c_int, c.c_int]
    L.dssd_edge_verify.restype = c.c_int
    L.dssd_edge_verify.argtypes = [
        c.c_void_p, c.c_int, c.c_int64, c.c_void_p, c.c_void_p, c.c_void_p, c.c_float,
        c.c_int, c.c_int, c.c_int, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p,
        c.c_void_p, c.c_size_t, c.c_void_p]
    L.dssd_device_resample.restype = c.c_int
    L.dssd_device_resample.argtypes = [
        c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_int, c.c_int, c.c_int,
        c.c_void_p, c.c_void_p, c.c_void_p, c.c_size_t, c.c_void_p]
    L.dssd_device_resample_static.restype = c.c_int
    L.dssd_device_resample_static.argtypes = [
        c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_int, c.c_int, c.c_int,
        c.c_void_p, c.c_void_p, c.c_void_p]
    L.dssd_edge_verify_topk_workspace_bytes.restype = c.c_size_t
    L.dssd_edge_verify_topk_workspace_bytes.argtypes = [c.c_int, c.c_int, c.c_int, c.c_int]
    L.dssd_edge_verify_topk.restype = c.c_int
    L.dssd_edge_verify_topk.argtypes = [
        c.c_void_p, c.c_int, c.c_int64, c.c_void_p, c.c_void_p, c.c_void_p, c.c_float,
        c.c_int, c.c_int, c.c_int, c.c_int, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p,
        c.c_void_p, c.c_size_t, c.c_void_p]
    L.dssd_device_resample_topk.restype = c.c_int
    L.dssd_device_resample_topk.argtypes = [
        c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p,
        c.c_int, c.c_int, c.c_int, c.c_void_p, c.c_void_p, c.c_void_p]
    L.dssd_edge_verify_p16.restype = c.c_int
    L.dssd_edge_verify_p16.argtypes = L.dssd_edge_verify.argtypes
    L.dssd_device_resample_p16.restype = c.c_int
    L.dssd_device_resample_p16.argtypes = L.dssd_device_resample.argtypes
    L.dssd_dsd_verify_workspace_bytes.restype = c.c_size_t
    L.dssd_dsd_verify_workspace_bytes.argtypes = [c.c_int, c.c_int, c.c_int]
    L.dssd_dsd_verify.restype = c.c_int
    L.dssd_dsd_verify.argtypes = [
        c.c_void_p, c.c_int, c.c_int64, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_float,
        c.c_int, c.c_int, c.c_int, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_size_t, c.c_void_p]
    L.dssd_edge_verify_bonus_workspace_bytes.restype = c.c_size_t
    L.dssd_edge_verify_bonus_workspace_bytes.argtypes = [c.c_int, c.c_int, c.c_int]
    L.dssd_edge_verify_bonus.restype = c.c_int
    L.dssd_edge_verify_bonus.argtypes = [
        c.c_void_p, c.c_int, c.c_int64, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_float,
        c.c_int, c.c_int, c.c_int, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p,
        c.c_void_p, c.c_void_p, c.c_size_t, c.c_void_p]
    L.dssd_device_resample_rejected.restype = c.c_int
    L.dssd_device_resample_rejected.argtypes = L.dssd_device_resample.argtypes
    for f in (L.dssd_edge_partial_workspace_bytes, L.dssd_resample_shard_workspace_bytes):
        f.restype = c.c_size_t
        f.argtypes = [c.c_int, c.c_int, c.c_int]
    L.dssd_edge_partial.restype = c.c_int
    L.dssd_edge_partial.argtypes = [
        c.c_void_p, c.c_int, c.c_int64, c.c_void_p, c.c_int, c.c_float, c.c_int, c.c_int, c.c_int,
        c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_size_t, c.c_void_p]
    L.dssd_edge_combine.restype = c.c_int
    L.dssd_edge_combine.argtypes = [
        c.c_void_p, c.c_void_p, c.c_void_p, c.c_int, c.c_void_p, c.c_void_p, c.c_void_p, c.c_float,
        c.c_int, c.c_int, c.c_int, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p]
    L.dssd_edge_emit_shard.restype = c.c_int
    L.dssd_edge_emit_shard.argtypes = [
        c.c_void_p, c.c_int, c.c_int64, c.c_void_p, c.c_void_p, c.c_float, c.c_int, c.c_int, c.c_int,
        c.c_void_p, c.c_int64, c.c_void_p]
    L.dssd_resample_shard_mass.restype = c.c_int
    L.dssd_resample_shard_mass.argtypes = [
        c.c_void_p, c.c_int64, c.c_void_p, c.c_int64, c.c_void_p, c.c_int, c.c_int, c.c_int,
        c.c_void_p, c.c_void_p, c.c_size_t, c.c_void_p]
    L.dssd_resample_shard_draw.restype = c.c_int
    L.dssd_resample_shard_draw.argtypes = [
        c.c_void_p, c.c_int, c.c_int, c.c_int, c.c_void_p, c.c_int64, c.c_void_p, c.c_int64,
        c.c_void_p, c.c_void_p, c.c_int, c.c_int, c.c_int, c.c_void_p, c.c_void_p,
        c.c_void_p, c.c_size_t, c.c_void_p]
    L.dssd_round_host.restype = c.c_int
    L.dssd_round_host.argtypes = [
        c.c_void_p, c.c_int, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_float,
        c.c_int, c.c_int, c.c_int, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p,
        c.c_void_p, c.c_size_t, c.c_void_p]
    L.dssd_round_host_topk_arena_bytes.restype = c.c_size_t
    L.dssd_round_host_topk_arena_bytes.argtypes = [c.c_int, c.c_int, c.c_int, c.c_int, c.c_int]
    L.dssd_round_host_topk.restype = c.c_int
    L.dssd_round_host_topk.argtypes = [
        c.c_void_p, c.c_int, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_float,
        c.c_int, c.c_int, c.c_int, c.c_int, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p,
        c.c_void_p, c.c_size_t, c.c_void_p]
    return L


lib = _load()


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None or t.numel() == 0 else t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return DSSD_BF16
    if t.dtype == torch.float32:
        return DSSD_F32
    raise TypeError(f"target_logits must be float32 or bfloat16, got {t.dtype}")


def _row_stride(target_logits: torch.Tensor) -> int:
    """Elements between consecutive rows of a [B, gamma+1, V] tensor with unit stride along V."""
    B, g1, V = target_logits.shape
    assert target_logits.stride(2) == 1 or V == 1
    row_stride = target_logits.stride(1) if g1 > 1 else max(V, target_logits.stride(0))
    if B > 1 and target_logits.stride(0) != g1 * row_stride:
        raise ValueError("rows of target_logits must be equally spaced")
    return row_stride


def _workspace(nbytes: int, device) -> torch.Tensor:
    return torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device)


def dssd_edge_verify_workspace_bytes(B: int, gamma: int, V: int) -> int:
    return int(lib.dssd_edge_verify_workspace_bytes(B, gamma, V))


def dssd_device_resample_workspace_bytes(B: int, gamma: int, V: int) -> int:
    return int(lib.dssd_device_resample_workspace_bytes(B, gamma, V))


def dssd_round_host_arena_bytes(B: int, gamma: int, V: int, dtype: int) -> int:
    return int(lib.dssd_round_host_arena_bytes(B, gamma, V, dtype))


def dssd_edge_verify(target_logits: torch.Tensor, draft_tokens: torch.Tensor, draft_q_tok: torch.Tensor,
                     uniforms: torch.Tensor, temperature: float, *, out: Optional[Dict[str, torch.Tensor]] = None,
                     want_p_tok: bool = True, want_lse: bool = True, workspace: Optional[torch.Tensor] = None,
                     stream=None, payload: str = "f32") -> Dict[str, torch.Tensor]:
    """Edge half of one round.  target_logits: CUDA tensor [B, gamma+1, V], float32 or bfloat16,
    unit stride along V and a common stride between rows.  Returns accept_len, p_row, flags and,
    if asked, p_tok and lse.  Pass `out` (a previous result) and `workspace` to allocate nothing.
    payload="f16" writes p_row as float16 (dssd_edge_verify_p16)."""
    assert target_logits.is_cuda and target_logits.dim() == 3
    B, g1, V = target_logits.shape
    gamma = g1 - 1
    row_stride = _row_stride(target_logits)
    dev = target_logits.device
    if out is None:
        out = {
            "accept_len": torch.empty(B, dtype=torch.int32, device=dev),
            "p_row": torch.empty(B, V, dtype=torch.float16 if payload == "f16" else torch.float32, device=dev),
            "flags": torch.empty(B, dtype=torch.int32, device=dev),
            "p_tok": torch.empty(B, gamma, dtype=torch.float32, device=dev) if want_p_tok else None,
            "lse": torch.empty(B, g1, dtype=torch.float32, device=dev) if want_lse else None,
        }
    assert out["p_row"].dtype == (torch.float16 if payload == "f16" else torch.float32)
    need = dssd_edge_verify_workspace_bytes(B, gamma, V)
    if workspace is None:
        workspace = _workspace(need, dev)
    fn = lib.dssd_edge_verify_p16 if payload == "f16" else lib.dssd_edge_verify
    st = fn(
        target_logits.data_ptr(), _dtype_code(target_logits), row_stride,
        _ptr(draft_tokens), _ptr(draft_q_tok), _ptr(uniforms), ctypes.c_float(temperature), B, gamma, V,
        out["accept_len"].data_ptr(), out["p_row"].data_ptr(), _ptr(out.get("p_tok")), _ptr(out.get("lse")),
        _ptr(out.get("flags")), workspace.data_ptr(), workspace.numel(), _stream(stream))
    if st != DSSD_OK:
        raise DssdError(st, "dssd_edge_verify")
    return out


def dssd_device_resample(p_row: torch.Tensor, draft_q: Optional[torch.Tensor], accept_len: torch.Tensor,
                         uniforms_rs: torch.Tensor, gamma: int, *, out: Optional[Dict[str, torch.Tensor]] = None,
                         workspace: Optional[torch.Tensor] = None, stream=None) -> Dict[str, torch.Tensor]:
    """Device half of one round.  p_row [B, V] float32 (or float16: dssd_device_resample_p16),
    draft_q [B, gamma, V] float32 (contiguous)."""
    assert p_row.is_cuda and p_row.dim() == 2 and p_row.is_contiguous() and p_row.dtype in (torch.float32, torch.float16)
    B, V = p_row.shape
    if gamma > 0:
        assert draft_q.is_contiguous() and draft_q.dtype == torch.float32 and draft_q.numel() == B * gamma * V
    dev = p_row.device
    if out is None:
        out = {"token": torch.empty(B, dtype=torch.int32, device=dev),
               "flags": torch.empty(B, dtype=torch.int32, device=dev)}
    need = dssd_device_resample_workspace_bytes(B, gamma, V)
    if workspace is None:
        workspace = _workspace(need, dev)
    fn = lib.dssd_device_resample_p16 if p_row.dtype == torch.float16 else lib.dssd_device_resample
    st = fn(
        p_row.data_ptr(), _ptr(draft_q) if gamma > 0 else None, accept_len.data_ptr(), uniforms_rs.data_ptr(),
        B, gamma, V, out["token"].data_ptr(), _ptr(out.get("flags")), workspace.data_ptr(), workspace.numel(),
        _stream(stream))
    if st != DSSD_OK:
        raise DssdError(st, "dssd_device_resample")
    return out


STATIC_SCRATCH_BYTES = 1 << 20


def dssd_device_resample_static(p_row: torch.Tensor, draft_q: Optional[torch.Tensor], accept_len: torch.Tensor,
                                uniforms_rs: torch.Tensor, gamma: int, *, out: Dict[str, torch.Tensor],
                                stream=None) -> Dict[str, torch.Tensor]:
    """Device half of one round for callers that cannot allocate: the scratch is a fixed array
    inside the library, and `out` (token, flags: int32 [B]) must be passed in, so that neither
    the library nor this wrapper allocates anything.  Sizes beyond the built-in scratch raise
    DssdError(DSSD_ERR_UNSUPPORTED).  Calls that overlap on the GPU race on the shared scratch."""
    assert p_row.is_cuda and p_row.dim() == 2 and p_row.is_contiguous() and p_row.dtype == torch.float32
    B, V = p_row.shape
    st = lib.dssd_device_resample_static(
        p_row.data_ptr(), _ptr(draft_q) if gamma > 0 else None, accept_len.data_ptr(), uniforms_rs.data_ptr(),
        B, gamma, V, out["token"].data_ptr(), _ptr(out.get("flags")), _stream(stream))
    if st != DSSD_OK:
        raise DssdError(st, "dssd_device_resample_static")
    return out


TOPK_MAX = 32


def dssd_edge_verify_topk_workspace_bytes(B: int, gamma: int, V: int, k: int) -> int:
    return int(lib.dssd_edge_verify_topk_workspace_bytes(B, gamma, V, k))


def dssd_edge_verify_topk(target_logits: torch.Tensor, draft_tokens: torch.Tensor, draft_q_tok: torch.Tensor,
                          uniforms: torch.Tensor, temperature: float, k: int, *,
                          out: Optional[Dict[str, torch.Tensor]] = None, want_p_tok: bool = True,
                          workspace: Optional[torch.Tensor] = None, stream=None) -> Dict[str, torch.Tensor]:
    """Edge half of one round on target distributions truncated to their k largest entries.
    Returns accept_len [B], p_idx / p_val [B, k], flags and, if asked, p_tok."""
    assert target_logits.is_cuda and target_logits.dim() == 3
    B, g1, V = target_logits.shape
    gamma = g1 - 1
    row_stride = _row_stride(target_logits)
    dev = target_logits.device
    if out is None:
        kk = max(0, min(k, TOPK_MAX))
        out = {
            "accept_len": torch.empty(B, dtype=torch.int32, device=dev),
            "p_idx": torch.empty(B, kk, dtype=torch.int32, device=dev),
            "p_val": torch.empty(B, kk, dtype=torch.float32, device=dev),
            "flags": torch.empty(B, dtype=torch.int32, device=dev),
            "p_tok": torch.empty(B, gamma, dtype=torch.float32, device=dev) if want_p_tok else None,
        }
    if workspace is None:
        workspace = _workspace(dssd_edge_verify_topk_workspace_bytes(B, gamma, V, k), dev)
    st = lib.dssd_edge_verify_topk(
        target_logits.data_ptr(), _dtype_code(target_logits), row_stride,
        _ptr(draft_tokens), _ptr(draft_q_tok), _ptr(uniforms), ctypes.c_float(temperature), B, gamma, V, k,
        out["accept_len"].data_ptr(), out["p_idx"].data_ptr(), out["p_val"].data_ptr(), _ptr(out.get("p_tok")),
        _ptr(out.get("flags")), workspace.data_ptr(), workspace.numel(), _stream(stream))
    if st != DSSD_OK:
        raise DssdError(st, "dssd_edge_verify_topk")
    return out


def dssd_device_resample_topk(p_idx: torch.Tensor, p_val: torch.Tensor, q_idx: Optional[torch.Tensor],
                              q_val: Optional[torch.Tensor], accept_len: torch.Tensor,
                              uniforms_rs: torch.Tensor, gamma: int, *,
                              out: Optional[Dict[str, torch.Tensor]] = None, stream=None) -> Dict[str, torch.Tensor]:
    """Device half on truncated distributions: p_* [B, k], q_* [B, gamma, k] (contiguous)."""
    assert p_idx.is_cuda and p_idx.dim() == 2 and p_idx.is_contiguous() and p_idx.dtype == torch.int32
    assert p_val.is_contiguous() and p_val.dtype == torch.float32 and p_val.shape == p_idx.shape
    B, k = p_idx.shape
    if gamma > 0:
        assert q_idx.is_contiguous() and q_idx.dtype == torch.int32 and q_idx.numel() == B * gamma * k
        assert q_val.is_contiguous() and q_val.dtype == torch.float32 and q_val.numel() == B * gamma * k
    dev = p_idx.device
    if out is None:
        out = {"token": torch.empty(B, dtype=torch.int32, device=dev),
               "flags": torch.empty(B, dtype=torch.int32, device=dev)}
    st = lib.dssd_device_resample_topk(
        p_idx.data_ptr(), p_val.data_ptr(), _ptr(q_idx) if gamma > 0 else None,
        _ptr(q_val) if gamma > 0 else None, accept_len.data_ptr(), uniforms_rs.data_ptr(), B, gamma, k,
        out["token"].data_ptr(), _ptr(out.get("flags")), _stream(stream))
    if st != DSSD_OK:
        raise DssdError(st, "dssd_device_resample_topk")
    return out


def dssd_dsd_verify_workspace_bytes(B: int, gamma: int, V: int) -> int:
    return int(lib.dssd_dsd_verify_workspace_bytes(B, gamma, V))


def dssd_dsd_verify(target_logits: torch.Tensor, draft_q: Optional[torch.Tensor], draft_tokens: torch.Tensor,
                    uniforms: torch.Tensor, uniforms_rs: torch.Tensor, temperature: float, *,
                    out: Optional[Dict[str, torch.Tensor]] = None, workspace: Optional[torch.Tensor] = None,
                    stream=None) -> Dict[str, torch.Tensor]:
    """Fused verification of Algorithm 1: acceptance tests with q_i(x_i) read from the draft rows and
    the corrected / bonus draw, without any row P_n in memory.  Returns accept_len, token, edge_flags, rs_flags."""
    assert target_logits.is_cuda and target_logits.dim() == 3
    B, g1, V = target_logits.shape
    gamma = g1 - 1
    row_stride = _row_stride(target_logits)
    if gamma > 0:
        assert draft_q.is_contiguous() and draft_q.dtype == torch.float32 and draft_q.numel() == B * gamma * V
    dev = target_logits.device
    if out is None:
        out = {k: torch.empty(B, dtype=torch.int32, device=dev) for k in ("accept_len", "token", "edge_flags", "rs_flags")}
    if workspace is None:
        workspace = _workspace(dssd_dsd_verify_workspace_bytes(B, gamma, V), dev)
    st = lib.dssd_dsd_verify(
        target_logits.data_ptr(), _dtype_code(target_logits), row_stride, _ptr(draft_q) if gamma > 0 else None,
        _ptr(draft_tokens), _ptr(uniforms), uniforms_rs.data_ptr(), ctypes.c_float(temperature), B, gamma, V,
        out["accept_len"].data_ptr(), out["token"].data_ptr(), _ptr(out.get("edge_flags")), _ptr(out.get("rs_flags")),
        workspace.data_ptr(), workspace.numel(), _stream(stream))
    if st != DSSD_OK:
        raise DssdError(st, "dssd_dsd_verify")
    return out


def dssd_edge_verify_bonus_workspace_bytes(B: int, gamma: int, V: int) -> int:
    return int(lib.dssd_edge_verify_bonus_workspace_bytes(B, gamma, V))


def dssd_edge_verify_bonus(target_logits: torch.Tensor, draft_tokens: torch.Tensor, draft_q_tok: torch.Tensor,
                           uniforms: torch.Tensor, uniforms_bonus: torch.Tensor, temperature: float, *,
                           out: Optional[Dict[str, torch.Tensor]] = None, want_p_tok: bool = True,
                           want_lse: bool = True, workspace: Optional[torch.Tensor] = None,
                           stream=None) -> Dict[str, torch.Tensor]:
    """Edge half with the bonus token drawn at the edge (Algorithm 2 as printed): p_row is written only
    for sequences with a rejection; `token` holds the bonus token of fully accepted sequences (-1
    elsewhere) and `token_flags` its flags.  Returns accept_len, p_row, token, token_flags, flags and,
    if asked, p_tok and lse.  A fresh p_row starts out as zeros so that unwritten rows are defined."""
    assert target_logits.is_cuda and target_logits.dim() == 3
    B, g1, V = target_logits.shape
    gamma = g1 - 1
    row_stride = _row_stride(target_logits)
    dev = target_logits.device
    if out is None:
        out = {
            "accept_len": torch.empty(B, dtype=torch.int32, device=dev),
            "p_row": torch.zeros(B, V, dtype=torch.float32, device=dev),
            "token": torch.empty(B, dtype=torch.int32, device=dev),
            "token_flags": torch.empty(B, dtype=torch.int32, device=dev),
            "flags": torch.empty(B, dtype=torch.int32, device=dev),
            "p_tok": torch.empty(B, gamma, dtype=torch.float32, device=dev) if want_p_tok else None,
            "lse": torch.empty(B, g1, dtype=torch.float32, device=dev) if want_lse else None,
        }
    if workspace is None:
        workspace = _workspace(dssd_edge_verify_bonus_workspace_bytes(B, gamma, V), dev)
    st = lib.dssd_edge_verify_bonus(
        target_logits.data_ptr(), _dtype_code(target_logits), row_stride,
        _ptr(draft_tokens), _ptr(draft_q_tok), _ptr(uniforms), uniforms_bonus.data_ptr(), ctypes.c_float(temperature),
        B, gamma, V, out["accept_len"].data_ptr(), out["p_row"].data_ptr(), out["token"].data_ptr(),
        _ptr(out.get("p_tok")), _ptr(out.get("lse")), _ptr(out.get("flags")), _ptr(out.get("token_flags")),
        workspace.data_ptr(), workspace.numel(), _stream(stream))
    if st != DSSD_OK:
        raise DssdError(st, "dssd_edge_verify_bonus")
    return out


def dssd_device_resample_rejected(p_row: torch.Tensor, draft_q: Optional[torch.Tensor], accept_len: torch.Tensor,
                                  uniforms_rs: torch.Tensor, gamma: int, *, out: Dict[str, torch.Tensor],
                                  workspace: Optional[torch.Tensor] = None, stream=None) -> Dict[str, torch.Tensor]:
    """Device half for the rejected sequences only: out["token"] / out["flags"] (int32 [B], as
    dssd_edge_verify_bonus left them) are written where accept_len < gamma and kept elsewhere."""
    assert p_row.is_cuda and p_row.dim() == 2 and p_row.is_contiguous() and p_row.dtype == torch.float32
    B, V = p_row.shape
    if gamma > 0:
        assert draft_q.is_contiguous() and draft_q.dtype == torch.float32 and draft_q.numel() == B * gamma * V
    if workspace is None:
        workspace = _workspace(dssd_device_resample_workspace_bytes(B, gamma, V), p_row.device)
    st = lib.dssd_device_resample_rejected(
        p_row.data_ptr(), _ptr(draft_q) if gamma > 0 else None, accept_len.data_ptr(), uniforms_rs.data_ptr(),
        B, gamma, V, out["token"].data_ptr(), _ptr(out.get("flags")), workspace.data_ptr(), workspace.numel(),
        _stream(stream))
    if st != DSSD_OK:
        raise DssdError(st, "dssd_device_resample_rejected")
    return out


def dssd_round_host(host: Dict[str, torch.Tensor], temperature: float, arena: torch.Tensor, *,
                    out: Optional[Dict[str, torch.Tensor]] = None, want_p_row: bool = False,
                    stream=None) -> Dict[str, torch.Tensor]:
    """Both halves on HOST tensors (pinned for asynchronous copies); `arena` is CUDA scratch of
    dssd_round_host_arena_bytes(...) bytes.  Results land in host tensors once the stream is done."""
    tl = host["target_logits"]
    assert not tl.is_cuda and tl.is_contiguous() and tl.dim() == 3
    B, g1, V = tl.shape
    gamma = g1 - 1
    if out is None:
        pin = torch.cuda.is_available()
        out = {k: torch.empty(B, dtype=torch.int32, pin_memory=pin)
               for k in ("accept_len", "token", "edge_flags", "rs_flags")}
        out["p_row"] = torch.empty(B, V, dtype=torch.float32, pin_memory=pin) if want_p_row else None
    st = lib.dssd_round_host(
        tl.data_ptr(), _dtype_code(tl), _ptr(host.get("draft_tokens")), _ptr(host.get("draft_q_tok")),
        _ptr(host.get("uniforms")), _ptr(host.get("draft_q")), host["uniforms_rs"].data_ptr(),
        ctypes.c_float(temperature), B, gamma, V, out["accept_len"].data_ptr(), out["token"].data_ptr(),
        _ptr(out.get("edge_flags")), _ptr(out.get("rs_flags")), _ptr(out.get("p_row")),
        arena.data_ptr(), arena.numel(), _stream(stream))
    if st != DSSD_OK:
        raise DssdError(st, "dssd_round_host")
    return out


def dssd_round_host_topk_arena_bytes(B: int, gamma: int, V: int, k: int, dtype: int) -> int:
    return int(lib.dssd_round_host_topk_arena_bytes(B, gamma, V, k, dtype))


def dssd_round_host_topk(host: Dict[str, torch.Tensor], temperature: float, k: int, arena: torch.Tensor, *,
                         out: Optional[Dict[str, torch.Tensor]] = None, want_pairs: bool = False,
                         stream=None) -> Dict[str, torch.Tensor]:
    """The truncated-support round on HOST tensors (pinned for asynchronous copies); `arena` is CUDA
    scratch of dssd_round_host_topk_arena_bytes(...) bytes.  Results land in host tensors once the stream is done."""
    tl = host["target_logits"]
    assert not tl.is_cuda and tl.is_contiguous() and tl.dim() == 3
    B, g1, V = tl.shape
    gamma = g1 - 1
    if out is None:
        pin = torch.cuda.is_available()
        out = {n: torch.empty(B, dtype=torch.int32, pin_memory=pin)
               for n in ("accept_len", "token", "edge_flags", "rs_flags")}
        out["p_idx"] = torch.empty(B, k, dtype=torch.int32, pin_memory=pin) if want_pairs else None
        out["p_val"] = torch.empty(B, k, dtype=torch.float32, pin_memory=pin) if want_pairs else None
    st = lib.dssd_round_host_topk(
        tl.data_ptr(), _dtype_code(tl), _ptr(host.get("draft_tokens")), _ptr(host.get("draft_q_tok")),
        _ptr(host.get("uniforms")), _ptr(host.get("q_idx")), _ptr(host.get("q_val")), host["uniforms_rs"].data_ptr(),
        ctypes.c_float(temperature), B, gamma, V, k, out["accept_len"].data_ptr(), out["token"].data_ptr(),
        _ptr(out.get("edge_flags")), _ptr(out.get("rs_flags")), _ptr(out.get("p_idx")), _ptr(out.get("p_val")),
        arena.data_ptr(), arena.numel(), _stream(stream))
    if st != DSSD_OK:
        raise DssdError(st, "dssd_round_host_topk")
    return out


# ---- the vocabulary-sharded round: five calls per shard, two small exchanges between them ----


def dssd_edge_partial_workspace_bytes(B: int, gamma: int, V_shard: int) -> int:
    return int(lib.dssd_edge_partial_workspace_bytes(B, gamma, V_shard))


def dssd_resample_shard_workspace_bytes(B: int, gamma: int, V_shard: int) -> int:
    return int(lib.dssd_resample_shard_workspace_bytes(B, gamma, V_shard))


def dssd_edge_partial(logits_shard: torch.Tensor, draft_tokens: torch.Tensor, v_begin: int, temperature: float, *,
                      out: Optional[Dict[str, torch.Tensor]] = None, workspace: Optional[torch.Tensor] = None,
                      stream=None) -> Dict[str, torch.Tensor]:
    """One shard's partial sums.  logits_shard [B, gamma+1, V_shard]: this shard's slice of every row (a
    view into whole rows works), vocabulary ids v_begin .. v_begin + V_shard - 1.  Returns part_ref
    [B, gamma+1] float32, part_sum [B, gamma+1] float64, tok_logit [B, gamma] float32."""
    assert logits_shard.is_cuda and logits_shard.dim() == 3
    B, g1, Vs = logits_shard.shape
    gamma = g1 - 1
    row_stride = _row_stride(logits_shard)
    dev = logits_shard.device
    if out is None:
        out = {"part_ref": torch.empty(B, g1, dtype=torch.float32, device=dev),
               "part_sum": torch.empty(B, g1, dtype=torch.float64, device=dev),
               "tok_logit": torch.empty(B, gamma, dtype=torch.float32, device=dev)}
    if workspace is None:
        workspace = _workspace(dssd_edge_partial_workspace_bytes(B, gamma, Vs), dev)
    st = lib.dssd_edge_partial(
        logits_shard.data_ptr(), _dtype_code(logits_shard), row_stride, _ptr(draft_tokens), v_begin,
        ctypes.c_float(temperature), B, gamma, Vs, out["part_ref"].data_ptr(), out["part_sum"].data_ptr(),
        _ptr(out["tok_logit"]), workspace.data_ptr(), workspace.numel(), _stream(stream))
    if st != DSSD_OK:
        raise DssdError(st, "dssd_edge_partial")
    return out


def dssd_edge_combine(part_ref: torch.Tensor, part_sum: torch.Tensor, tok_logit: torch.Tensor,
                      draft_tokens: torch.Tensor, draft_q_tok: torch.Tensor, uniforms: torch.Tensor,
                      temperature: float, V: int, *, out: Optional[Dict[str, torch.Tensor]] = None,
                      stream=None) -> Dict[str, torch.Tensor]:
    """part_ref, part_sum [G, B, gamma+1] and tok_logit [G, B, gamma], gathered from the G shards ->
    accept_len [B], row_scale [B, 2], p_tok, lse, flags.  V is the size of the whole vocabulary."""
    assert part_ref.is_cuda and part_ref.dim() == 3 and part_ref.is_contiguous() and part_ref.dtype == torch.float32
    assert part_sum.shape == part_ref.shape and part_sum.is_contiguous() and part_sum.dtype == torch.float64
    G, B, g1 = part_ref.shape
    gamma = g1 - 1
    assert tok_logit.is_contiguous() and tok_logit.dtype == torch.float32 and tok_logit.numel() == G * B * gamma
    dev = part_ref.device
    if out is None:
        out = {"accept_len": torch.empty(B, dtype=torch.int32, device=dev),
               "row_scale": torch.empty(B, 2, dtype=torch.float32, device=dev),
               "p_tok": torch.empty(B, gamma, dtype=torch.float32, device=dev),
               "lse": torch.empty(B, g1, dtype=torch.float32, device=dev),
               "flags": torch.empty(B, dtype=torch.int32, device=dev)}
    st = lib.dssd_edge_combine(
        part_ref.data_ptr(), part_sum.data_ptr(), _ptr(tok_logit), G, _ptr(draft_tokens), _ptr(draft_q_tok),
        _ptr(uniforms), ctypes.c_float(temperature), B, gamma, V, out["accept_len"].data_ptr(),
        out["row_scale"].data_ptr(), _ptr(out.get("p_tok")), _ptr(out.get("lse")), _ptr(out.get("flags")),
        _stream(stream))
    if st != DSSD_OK:
        raise DssdError(st, "dssd_edge_combine")
    return out


def _rows_2d(t: torch.Tensor) -> int:
    """Elements between consecutive rows of a [B, V] float32 tensor with unit stride along V."""
    assert t.is_cuda and t.dim() == 2 and t.dtype == torch.float32 and (t.stride(1) == 1 or t.shape[1] == 1)
    return max(t.shape[1], t.stride(0)) if t.shape[0] > 1 else t.shape[1]


def dssd_edge_emit_shard(logits_shard: torch.Tensor, accept_len: torch.Tensor, row_scale: torch.Tensor,
                         temperature: float, *, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """This shard's slice of the downlink row: [B, V_shard] float32 (`out` may be a view into whole rows)."""
    assert logits_shard.is_cuda and logits_shard.dim() == 3
    B, g1, Vs = logits_shard.shape
    if out is None:
        out = torch.empty(B, Vs, dtype=torch.float32, device=logits_shard.device)
    assert out.shape == (B, Vs)
    st = lib.dssd_edge_emit_shard(
        logits_shard.data_ptr(), _dtype_code(logits_shard), _row_stride(logits_shard), accept_len.data_ptr(),
        row_scale.data_ptr(), ctypes.c_float(temperature), B, g1 - 1, Vs, out.data_ptr(), _rows_2d(out),
        _stream(stream))
    if st != DSSD_OK:
        raise DssdError(st, "dssd_edge_emit_shard")
    return out


def _q_stride(draft_q_shard: Optional[torch.Tensor], B: int, gamma: int, Vs: int) -> int:
    if gamma == 0 or draft_q_shard is None:
        return Vs
    q = draft_q_shard
    assert q.is_cuda and q.dtype == torch.float32 and q.shape == (B, gamma, Vs) and (q.stride(2) == 1 or Vs == 1)
    stride = q.stride(1) if gamma > 1 else max(Vs, q.stride(0))
    if B > 1 and q.stride(0) != gamma * stride:
        raise ValueError("rows of draft_q_shard must be equally spaced")
    return stride


def dssd_resample_shard_mass(p_row_shard: torch.Tensor, draft_q_shard: Optional[torch.Tensor],
                             accept_len: torch.Tensor, gamma: int, *, out: Optional[torch.Tensor] = None,
                             workspace: Optional[torch.Tensor] = None, stream=None):
    """This shard's residual mass and plain mass per sequence: ([B, 2] float64, the workspace that
    dssd_resample_shard_draw needs next)."""
    B, Vs = p_row_shard.shape
    dev = p_row_shard.device
    if out is None:
        out = torch.empty(B, 2, dtype=torch.float64, device=dev)
    if workspace is None:
        workspace = _workspace(dssd_resample_shard_workspace_bytes(B, gamma, Vs), dev)
    st = lib.dssd_resample_shard_mass(
        p_row_shard.data_ptr(), _rows_2d(p_row_shard), _ptr(draft_q_shard) if gamma > 0 else None,
        _q_stride(draft_q_shard, B, gamma, Vs), accept_len.data_ptr(), B, gamma, Vs, out.data_ptr(),
        workspace.data_ptr(), workspace.numel(), _stream(stream))
    if st != DSSD_OK:
        raise DssdError(st, "dssd_resample_shard_mass")
    return out, workspace


def dssd_resample_shard_draw(masses: torch.Tensor, g: int, v_begin: int, p_row_shard: torch.Tensor,
                             draft_q_shard: Optional[torch.Tensor], accept_len: torch.Tensor,
                             uniforms_rs: torch.Tensor, gamma: int, workspace: torch.Tensor, *,
                             out: Optional[Dict[str, torch.Tensor]] = None, stream=None) -> Dict[str, torch.Tensor]:
    """The draw as shard g sees it; masses [G, B, 2] float64 gathered from all shards.  token is the id
    in the whole vocabulary on the owning shard and -1 on the others; flags are the sequence's."""
    assert masses.is_cuda and masses.dim() == 3 and masses.is_contiguous() and masses.dtype == torch.float64
    G = masses.shape[0]
    B, Vs = p_row_shard.shape
    dev = p_row_shard.device
    if out is None:
        out = {"token": torch.empty(B, dtype=torch.int32, device=dev),
               "flags": torch.empty(B, dtype=torch.int32, device=dev)}
    st = lib.dssd_resample_shard_draw(
        masses.data_ptr(), G, g, v_begin, p_row_shard.data_ptr(), _rows_2d(p_row_shard),
        _ptr(draft_q_shard) if gamma > 0 else None, _q_stride(draft_q_shard, B, gamma, Vs), accept_len.data_ptr(),
        uniforms_rs.data_ptr(), B, gamma, Vs, out["token"].data_ptr(), _ptr(out.get("flags")),
        workspace.data_ptr(), workspace.numel(), _stream(stream))
    if st != DSSD_OK:
        raise DssdError(st, "dssd_resample_shard_draw")
    return out
