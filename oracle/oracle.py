"""ctypes front end of the CPU oracle (dssd_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA library and its Python binding never
import this module.

The arithmetic lives in dssd_oracle.c; this file compiles it with gcc, passes
numpy arrays through and, when asked, runs disjoint slices of the batch on
several host threads (sequences are independent, so this changes no result).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor
from typing import Dict, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dssd_oracle.c")
_LIB = os.path.join(_HERE, "libdssd_oracle.so")

F32 = 0
BF16 = 1

FLAG_BAD_TOKEN = 1
FLAG_NONFINITE = 2
RS_FLAG_BONUS = 1
RS_FLAG_FALLBACK = 2
RS_FLAG_INVALID = 4

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle (plain C, strict IEEE semantics: no fast-math, no contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-ffp-contract=off",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        c = ctypes
        lib.dssd_oracle_edge_verify.restype = c.c_int
        lib.dssd_oracle_edge_verify.argtypes = [
            c.c_void_p, c.c_int, c.c_int64, c.c_void_p, c.c_void_p, c.c_void_p, c.c_float,
            c.c_int, c.c_int, c.c_int,
            c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p]
        lib.dssd_oracle_device_resample.restype = c.c_int
        lib.dssd_oracle_device_resample.argtypes = [
            c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_int, c.c_int, c.c_int,
            c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p]
        lib.dssd_oracle_dsd_verify.restype = c.c_int
        lib.dssd_oracle_dsd_verify.argtypes = [
            c.c_void_p, c.c_int, c.c_int64, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_float,
            c.c_int, c.c_int, c.c_int, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p,
            c.c_void_p]
        lib.dssd_oracle_edge_verify_topk.restype = c.c_int
        lib.dssd_oracle_edge_verify_topk.argtypes = [
            c.c_void_p, c.c_int, c.c_int64, c.c_void_p, c.c_void_p, c.c_void_p, c.c_float,
            c.c_int, c.c_int, c.c_int, c.c_int,
            c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p]
        lib.dssd_oracle_device_resample_topk.restype = c.c_int
        lib.dssd_oracle_device_resample_topk.argtypes = [
            c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p,
            c.c_int, c.c_int, c.c_int, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p]
        _lib = lib
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _chunks(B: int, threads: int):
    threads = max(1, min(threads, B))
    edges = np.linspace(0, B, threads + 1).astype(int)
    return [(int(edges[i]), int(edges[i + 1])) for i in range(threads) if edges[i + 1] > edges[i]]


def edge_verify(target_logits: np.ndarray, draft_tokens: np.ndarray, draft_q_tok: np.ndarray,
                uniforms: np.ndarray, temperature: float, want_p_row64: bool = False,
                threads: int = 1) -> Dict[str, np.ndarray]:
    """Edge half of the round.  target_logits: [B, gamma+1, V] float32, or uint16 = bf16 bits."""
    lib = _load()
    tl = np.ascontiguousarray(target_logits)
    assert tl.ndim == 3 and tl.dtype in (np.float32, np.uint16)
    dtype = BF16 if tl.dtype == np.uint16 else F32
    B, g1, V = tl.shape
    gamma = g1 - 1
    tok = np.ascontiguousarray(draft_tokens, dtype=np.int32).reshape(B, gamma)
    qt = np.ascontiguousarray(draft_q_tok, dtype=np.float32).reshape(B, gamma)
    u = np.ascontiguousarray(uniforms, dtype=np.float32).reshape(B, gamma)
    out = {
        "accept_len": np.zeros(B, np.int32),
        "p_row": np.zeros((B, V), np.float32),
        "p_row64": np.zeros((B, V), np.float64) if want_p_row64 else None,
        "p_tok": np.zeros((B, gamma), np.float64),
        "lse": np.zeros((B, gamma + 1), np.float64),
        "flags": np.zeros(B, np.uint32),
        "margin_acc": np.zeros(B, np.float64),
    }

    def run(rng):
        b0, b1 = rng
        rc = lib.dssd_oracle_edge_verify(
            _ptr(tl[b0:b1]), dtype, V, _ptr(tok[b0:b1]), _ptr(qt[b0:b1]), _ptr(u[b0:b1]),
            ctypes.c_float(temperature), b1 - b0, gamma, V,
            _ptr(out["accept_len"][b0:b1]), _ptr(out["p_row"][b0:b1]),
            _ptr(out["p_row64"][b0:b1]) if want_p_row64 else None,
            _ptr(out["p_tok"][b0:b1]), _ptr(out["lse"][b0:b1]), _ptr(out["flags"][b0:b1]),
            _ptr(out["margin_acc"][b0:b1]))
        if rc != 0:
            raise ValueError("dssd_oracle_edge_verify: invalid arguments")

    parts = _chunks(B, threads)
    if len(parts) == 1:
        run(parts[0])
    else:
        with ThreadPoolExecutor(len(parts)) as ex:
            list(ex.map(run, parts))
    return out


def device_resample(p_row: np.ndarray, draft_q: Optional[np.ndarray], accept_len: np.ndarray,
                    uniforms_rs: np.ndarray, gamma: int, threads: int = 1) -> Dict[str, np.ndarray]:
    """Device half of the round.  p_row: [B, V] float32; draft_q: [B, gamma, V] float32."""
    lib = _load()
    p = np.ascontiguousarray(p_row, dtype=np.float32)
    B, V = p.shape
    if gamma > 0:
        q = np.ascontiguousarray(draft_q, dtype=np.float32).reshape(B, gamma, V)
    else:
        q = np.zeros((B, 0, V), np.float32)
    n = np.ascontiguousarray(accept_len, dtype=np.int32).reshape(B)
    u = np.ascontiguousarray(uniforms_rs, dtype=np.float32).reshape(B)
    out = {
        "token": np.zeros(B, np.int32),
        "flags": np.zeros(B, np.uint32),
        "margin_cdf": np.zeros(B, np.float64),
        "Z": np.zeros(B, np.float64),
    }

    def run(rng):
        b0, b1 = rng
        rc = lib.dssd_oracle_device_resample(
            _ptr(p[b0:b1]), _ptr(q[b0:b1]) if gamma > 0 else None, _ptr(n[b0:b1]), _ptr(u[b0:b1]),
            b1 - b0, gamma, V, _ptr(out["token"][b0:b1]), _ptr(out["flags"][b0:b1]),
            _ptr(out["margin_cdf"][b0:b1]), _ptr(out["Z"][b0:b1]))
        if rc != 0:
            raise ValueError("dssd_oracle_device_resample: invalid arguments")

    parts = _chunks(B, threads)
    if len(parts) == 1:
        run(parts[0])
    else:
        with ThreadPoolExecutor(len(parts)) as ex:
            list(ex.map(run, parts))
    return out


def to_payload16(p_row64: np.ndarray) -> np.ndarray:
    """The downlink row at b_prob = 16 bits (Section 2.2 allows 16 or 32): every probability
    rounded once, from float64, to IEEE binary16 (nearest, ties to even; values below 2**-25
    become 0, those below 2**-14 lose precision as subnormals).  Returns float16."""
    return np.asarray(p_row64, dtype=np.float64).astype(np.float16)


def verify_round(inputs: Dict[str, np.ndarray], temperature: float, threads: int = 1,
                 payload: str = "f32") -> Dict[str, np.ndarray]:
    """Both halves on one generated batch: the device half consumes the row that the edge half
    emitted, as it would after the downlink: float32, or with payload="f16" the 16-bit row
    (widened exactly to float32 for the draw)."""
    ev = edge_verify(inputs["target_logits"], inputs["draft_tokens"], inputs["draft_q_tok"],
                     inputs["uniforms"], temperature, want_p_row64=(payload == "f16"), threads=threads)
    gamma = inputs["target_logits"].shape[1] - 1
    if payload == "f16":
        ev["p_row16"] = to_payload16(ev["p_row64"])
        ev["p_row"] = ev["p_row16"].astype(np.float32)
        ev["p_row64"] = None
    rs = device_resample(ev["p_row"], inputs["draft_q"], ev["accept_len"], inputs["uniforms_rs"],
                         gamma, threads=threads)
    out = dict(ev)
    out["token"] = rs["token"]
    out["rs_flags"] = rs["flags"]
    out["margin_cdf"] = rs["margin_cdf"]
    out["Z"] = rs["Z"]
    return out


RS_FLAG_BONUS, RS_FLAG_FALLBACK, RS_FLAG_INVALID = 1, 2, 4


def bonus_draw(p_row64: np.ndarray, u: float):
    """x_{gamma+1} ~ P_{gamma+1} at the edge (Algorithm 2, the branch j = gamma + 1): inverse CDF in
    index order on the float64 row, token = min{k : sum_{v<=k} p_v > u * sum_v p_v}, clamped to the
    last entry with mass.  Returns (token, flags, margin relative to the row's sum)."""
    p = np.asarray(p_row64, dtype=np.float64)
    C = np.cumsum(p)  # sequential, in index order
    Z = C[-1]
    if not (np.isfinite(Z) and Z > 0.0):
        return -1, RS_FLAG_BONUS | RS_FLAG_INVALID, 0.0
    t = float(np.float64(np.float32(u))) * Z
    k = int(np.searchsorted(C, t, side="right"))
    if k >= p.size:
        k = int(np.nonzero(p > 0.0)[0][-1])
        return k, RS_FLAG_BONUS, 0.0
    below = C[k - 1] if k > 0 else 0.0
    return k, RS_FLAG_BONUS, float(min(t - below, C[k] - t) / Z)


def verify_round_bonus_at_edge(inputs: Dict[str, np.ndarray], temperature: float,
                               threads: int = 1) -> Dict[str, np.ndarray]:
    """One round as Algorithm 2 prints it: after gamma acceptances the edge itself draws the bonus
    token from P_{gamma+1} (in float64: nothing is rounded for a transmission that does not take
    place) and the downlink carries that token (Section 3, "Downlink Transmission"; a = 0 in Section
    3.1); after a rejection the float32 row P_n goes down and the device draws from the residual.
    `bonus_token` is what the edge sends (-1 for rejected sequences), `token` the round's result."""
    ev = edge_verify(inputs["target_logits"], inputs["draft_tokens"], inputs["draft_q_tok"],
                     inputs["uniforms"], temperature, want_p_row64=True, threads=threads)
    gamma = inputs["target_logits"].shape[1] - 1
    n = ev["accept_len"]
    rs = device_resample(ev["p_row"], inputs["draft_q"], n, inputs["uniforms_rs"], gamma, threads=threads)
    B = n.shape[0]
    out = dict(ev)
    out["token"] = rs["token"].copy()
    out["rs_flags"] = rs["flags"].copy()
    out["margin_cdf"] = rs["margin_cdf"].copy()
    out["Z"] = rs["Z"].copy()
    out["bonus_token"] = np.full(B, -1, np.int32)
    out["bonus_flags"] = np.zeros(B, np.uint32)
    for b in np.nonzero(n == gamma)[0]:
        tok, fl, margin = bonus_draw(ev["p_row64"][b], inputs["uniforms_rs"][b])
        out["bonus_token"][b] = out["token"][b] = tok
        out["bonus_flags"][b] = out["rs_flags"][b] = fl
        out["margin_cdf"][b] = margin
    out["p_row64"] = None
    return out


TOPK_MAX = 32


def edge_verify_topk(target_logits: np.ndarray, draft_tokens: np.ndarray, draft_q_tok: np.ndarray,
                     uniforms: np.ndarray, temperature: float, k: int,
                     threads: int = 1) -> Dict[str, np.ndarray]:
    """Edge half on distributions truncated to their k largest entries (Section 4, top-k sampling)."""
    lib = _load()
    tl = np.ascontiguousarray(target_logits)
    assert tl.ndim == 3 and tl.dtype in (np.float32, np.uint16)
    dtype = BF16 if tl.dtype == np.uint16 else F32
    B, g1, V = tl.shape
    gamma = g1 - 1
    tok = np.ascontiguousarray(draft_tokens, dtype=np.int32).reshape(B, gamma)
    qt = np.ascontiguousarray(draft_q_tok, dtype=np.float32).reshape(B, gamma)
    u = np.ascontiguousarray(uniforms, dtype=np.float32).reshape(B, gamma)
    out = {
        "accept_len": np.zeros(B, np.int32),
        "p_idx": np.zeros((B, k), np.int32),
        "p_val": np.zeros((B, k), np.float32),
        "p_val64": np.zeros((B, k), np.float64),
        "p_tok": np.zeros((B, gamma), np.float64),
        "flags": np.zeros(B, np.uint32),
        "margin_acc": np.zeros(B, np.float64),
    }

    def run(rng):
        b0, b1 = rng
        rc = lib.dssd_oracle_edge_verify_topk(
            _ptr(tl[b0:b1]), dtype, V, _ptr(tok[b0:b1]), _ptr(qt[b0:b1]), _ptr(u[b0:b1]),
            ctypes.c_float(temperature), b1 - b0, gamma, V, k,
            _ptr(out["accept_len"][b0:b1]), _ptr(out["p_idx"][b0:b1]), _ptr(out["p_val"][b0:b1]),
            _ptr(out["p_val64"][b0:b1]), _ptr(out["p_tok"][b0:b1]), _ptr(out["flags"][b0:b1]),
            _ptr(out["margin_acc"][b0:b1]))
        if rc != 0:
            raise ValueError("dssd_oracle_edge_verify_topk: invalid arguments")

    parts = _chunks(B, threads)
    if len(parts) == 1:
        run(parts[0])
    else:
        with ThreadPoolExecutor(len(parts)) as ex:
            list(ex.map(run, parts))
    return out


def device_resample_topk(p_idx: np.ndarray, p_val: np.ndarray, q_idx: Optional[np.ndarray],
                         q_val: Optional[np.ndarray], accept_len: np.ndarray,
                         uniforms_rs: np.ndarray, gamma: int) -> Dict[str, np.ndarray]:
    """Device half on truncated distributions: p_* [B, k], q_* [B, gamma, k]."""
    lib = _load()
    pi = np.ascontiguousarray(p_idx, dtype=np.int32)
    pv = np.ascontiguousarray(p_val, dtype=np.float32)
    B, k = pi.shape
    if gamma > 0:
        qi = np.ascontiguousarray(q_idx, dtype=np.int32).reshape(B, gamma, k)
        qv = np.ascontiguousarray(q_val, dtype=np.float32).reshape(B, gamma, k)
    else:
        qi = qv = None
    n = np.ascontiguousarray(accept_len, dtype=np.int32).reshape(B)
    u = np.ascontiguousarray(uniforms_rs, dtype=np.float32).reshape(B)
    out = {
        "token": np.zeros(B, np.int32),
        "flags": np.zeros(B, np.uint32),
        "margin_cdf": np.zeros(B, np.float64),
        "Z": np.zeros(B, np.float64),
    }
    rc = lib.dssd_oracle_device_resample_topk(
        _ptr(pi), _ptr(pv), _ptr(qi), _ptr(qv), _ptr(n), _ptr(u), B, gamma, k,
        _ptr(out["token"]), _ptr(out["flags"]), _ptr(out["margin_cdf"]), _ptr(out["Z"]))
    if rc != 0:
        raise ValueError("dssd_oracle_device_resample_topk: invalid arguments")
    return out


def verify_round_topk(inputs: Dict[str, np.ndarray], temperature: float, k: int,
                      threads: int = 1) -> Dict[str, np.ndarray]:
    """Both halves on one generated truncated-support batch."""
    ev = edge_verify_topk(inputs["target_logits"], inputs["draft_tokens"], inputs["draft_q_tok"],
                          inputs["uniforms"], temperature, k, threads=threads)
    gamma = inputs["target_logits"].shape[1] - 1
    rs = device_resample_topk(ev["p_idx"], ev["p_val"], inputs["q_idx"], inputs["q_val"],
                              ev["accept_len"], inputs["uniforms_rs"], gamma)
    out = dict(ev)
    out["token"] = rs["token"]
    out["rs_flags"] = rs["flags"]
    out["margin_cdf"] = rs["margin_cdf"]
    out["Z"] = rs["Z"]
    return out


def dsd_verify(inputs: Dict[str, np.ndarray], temperature: float, threads: int = 1) -> Dict[str, np.ndarray]:
    """Algorithm 1 (DSD) on one generated batch: the edge holds the full draft rows, tests with
    q_i(x_i) read from them, and draws the corrected or bonus token itself."""
    lib = _load()
    tl = np.ascontiguousarray(inputs["target_logits"])
    assert tl.ndim == 3 and tl.dtype in (np.float32, np.uint16)
    dtype = BF16 if tl.dtype == np.uint16 else F32
    B, g1, V = tl.shape
    gamma = g1 - 1
    q = (np.ascontiguousarray(inputs["draft_q"], dtype=np.float32).reshape(B, gamma, V) if gamma > 0
         else np.zeros((B, 0, V), np.float32))
    tok = np.ascontiguousarray(inputs["draft_tokens"], dtype=np.int32).reshape(B, gamma)
    u = np.ascontiguousarray(inputs["uniforms"], dtype=np.float32).reshape(B, gamma)
    urs = np.ascontiguousarray(inputs["uniforms_rs"], dtype=np.float32).reshape(B)
    out = {
        "accept_len": np.zeros(B, np.int32), "token": np.zeros(B, np.int32),
        "flags": np.zeros(B, np.uint32), "rs_flags": np.zeros(B, np.uint32),
        "margin_acc": np.zeros(B, np.float64), "margin_cdf": np.zeros(B, np.float64),
        "Z": np.zeros(B, np.float64),
    }

    def run(rng):
        b0, b1 = rng
        rc = lib.dssd_oracle_dsd_verify(
            _ptr(tl[b0:b1]), dtype, V, _ptr(q[b0:b1]) if gamma > 0 else None, _ptr(tok[b0:b1]), _ptr(u[b0:b1]),
            _ptr(urs[b0:b1]), ctypes.c_float(temperature), b1 - b0, gamma, V,
            _ptr(out["accept_len"][b0:b1]), _ptr(out["token"][b0:b1]), _ptr(out["flags"][b0:b1]),
            _ptr(out["rs_flags"][b0:b1]), _ptr(out["margin_acc"][b0:b1]), _ptr(out["margin_cdf"][b0:b1]),
            _ptr(out["Z"][b0:b1]))
        if rc != 0:
            raise ValueError("dssd_oracle_dsd_verify: invalid arguments")

    parts = _chunks(B, threads)
    if len(parts) == 1:
        run(parts[0])
    else:
        with ThreadPoolExecutor(len(parts)) as ex:
            list(ex.map(run, parts))
    return out
