"""Seeded synthetic inputs for one round of split speculative verification.

This module only manufactures inputs: target logits, the draft model's
distributions, drafted tokens and the uniforms that the verification rule
consumes.  It performs none of the verification arithmetic (no acceptance test,
no first-rejection scan, no residual sampling) and imports neither the CPU
oracle nor the CUDA library, so both can be fed from it without sharing code.

What it stands in for: the paper's experiments run OPT-family models on a
narrative prompt (Section 4).  Neither weights nor prompt are available, so the
draft process (Algorithm 2, "Draft Process": Q_i <- M_q, x_i ~ Q_i) is replaced
by a noise model: the draft logits are the target logits plus Gaussian noise,
and the drafted token is drawn from the resulting distribution.

Recipe (per sequence b, position i, vocabulary entry v):
  target logit  l = sigma_t * g + beta_v          g ~ N(0,1) i.i.d.
  beta_v        = -1.1 * ln(1 + pi(v)) when the workload has the Zipf bias
                  (pi = one seeded permutation of [0,V) per workload), else 0
  stored target = l rounded to the workload's dtype (bf16: round-to-nearest-even)
  draft logit   = l (before rounding) + sigma_d * g'
  Q_i           = softmax(draft logit / T), computed in float64, stored float32
  x_i           ~ Q_i by inverse CDF with one generator uniform
  q_i(x_i)      = the stored float32 entry of Q_i at x_i
  u_i, u'       = (32 random bits >> 8) * 2**-24, i.e. uniform on [0,1)

Truncated-support batches (the experiments' top-k sampler, Section 4, k = 10): the draft side
keeps only the k largest entries of each Q_i (equal entries: lower index first), renormalises
them in float64, stores them as float32 (index, value) pairs and draws x_i from those; the
target logits, the uniforms and their streams are the ones of the dense batch.

Every array has its own counter-based (Philox) stream keyed by
(seed, array id, sequence index), so changing B or gamma never perturbs the
leading values of another array.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, List, Optional

import numpy as np

BASE_SEED = 20250712

_ARR_PERM = 0
_ARR_TARGET = 1
_ARR_DRAFT = 2
_ARR_DRAFT_U = 3
_ARR_ACCEPT_U = 4
_ARR_RESAMPLE_U = 5


@dataclass(frozen=True)
class Workload:
    """Shape and noise parameters of one synthetic verification batch."""

    name: str
    B: int
    gamma: int
    V: int
    dtype: str  # "f32" or "bf16": storage type of the target logits
    temperature: float
    sigma_t: float
    sigma_d: float
    zipf: bool
    seed: int

    @property
    def rows(self) -> int:
        return self.B * (self.gamma + 1)

    @property
    def logit_bytes(self) -> int:
        return 2 if self.dtype == "bf16" else 4


def _seed(config_index: int, point_index: int = 0) -> int:
    return BASE_SEED + 1000 * config_index + point_index


PRESETS: Dict[str, Workload] = {
    "c1": Workload("c1", B=1, gamma=4, V=1024, dtype="f32", temperature=1.0,
                   sigma_t=2.0, sigma_d=0.5, zipf=False, seed=_seed(0)),
    "c2": Workload("c2", B=8, gamma=4, V=32000, dtype="bf16", temperature=1.0,
                   sigma_t=3.0, sigma_d=0.7, zipf=True, seed=_seed(1)),
    "c3": Workload("c3", B=64, gamma=8, V=128256, dtype="bf16", temperature=0.8,
                   sigma_t=3.0, sigma_d=1.0, zipf=True, seed=_seed(2)),
    "c4": Workload("c4", B=256, gamma=4, V=151936, dtype="bf16", temperature=0.7,
                   sigma_t=3.0, sigma_d=0.4, zipf=True, seed=_seed(3)),
}

SWEEP_B = (1, 16, 128, 1024)
SWEEP_GAMMA = (1, 2, 4, 8, 16)
SWEEP_SIGMA = (0.2, 0.6, 1.2)


def sweep_points() -> List[Workload]:
    """The 60 points of the V=50272 fp32 sweep, in (B, gamma, sigma) order."""
    pts = []
    idx = 0
    for B in SWEEP_B:
        for gamma in SWEEP_GAMMA:
            for sigma in SWEEP_SIGMA:
                pts.append(Workload(f"c5_B{B}_g{gamma}_s{sigma}", B=B, gamma=gamma,
                                    V=50272, dtype="f32", temperature=1.0, sigma_t=3.0,
                                    sigma_d=sigma, zipf=True, seed=_seed(4, idx)))
                idx += 1
    return pts


def sweep_max() -> Workload:
    """Largest sweep point by bytes: B=1024, gamma=16, middle noise level."""
    for w in sweep_points():
        if w.B == 1024 and w.gamma == 16 and w.sigma_d == 0.6:
            return replace(w, name="c5max")
    raise AssertionError


def get_workload(name: str) -> Workload:
    if name in PRESETS:
        return PRESETS[name]
    if name == "c5max":
        return sweep_max()
    for w in sweep_points():
        if w.name == name:
            return w
    raise KeyError(name)


def custom(B: int, gamma: int, V: int, dtype: str = "f32", temperature: float = 1.0,
           sigma_t: float = 3.0, sigma_d: float = 0.7, zipf: bool = True,
           seed: int = 1234, name: str = "custom") -> Workload:
    return Workload(name, B, gamma, V, dtype, temperature, sigma_t, sigma_d, zipf, seed)


def _rng(seed: int, arr: int, b: int) -> np.random.Generator:
    key = np.array([np.uint64(seed), (np.uint64(arr) << np.uint64(40)) | np.uint64(b)],
                   dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def _unit_uniform(rng: np.random.Generator, n: int) -> np.ndarray:
    bits = rng.integers(0, 2 ** 32, size=n, dtype=np.uint32)
    return ((bits >> np.uint32(8)).astype(np.float32) * np.float32(2.0 ** -24)).astype(np.float32)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest, ties to even); returns the 16-bit patterns."""
    bits = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = bits + np.uint32(0x7FFF) + ((bits >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def zipf_bias(w: Workload) -> Optional[np.ndarray]:
    if not w.zipf:
        return None
    perm = _rng(w.seed, _ARR_PERM, 0).permutation(w.V)
    return (-1.1 * np.log1p(perm.astype(np.float64))).astype(np.float32)


def _gen_sequence(w: Workload, b: int, beta: Optional[np.ndarray], out: Dict[str, np.ndarray], slot: int) -> None:
    g, V = w.gamma, w.V
    tl = _rng(w.seed, _ARR_TARGET, b).standard_normal(size=(g + 1, V), dtype=np.float32)
    tl *= np.float32(w.sigma_t)
    if beta is not None:
        tl += beta[None, :]
    if w.dtype == "bf16":
        out["target_logits"][slot] = f32_to_bf16_bits(tl)
    else:
        out["target_logits"][slot] = tl
    if g > 0:
        noise = _rng(w.seed, _ARR_DRAFT, b).standard_normal(size=(g, V), dtype=np.float32)
        d = tl[:g].astype(np.float64) + np.float64(w.sigma_d) * noise.astype(np.float64)
        d /= np.float64(np.float32(w.temperature))
        d -= d.max(axis=1, keepdims=True)
        np.exp(d, out=d)
        d /= d.sum(axis=1, keepdims=True)
        q32 = d.astype(np.float32)
        out["draft_q"][slot] = q32
        ud = _unit_uniform(_rng(w.seed, _ARR_DRAFT_U, b), g)
        for i in range(g):
            cs = np.cumsum(q32[i], dtype=np.float64)
            k = int(np.searchsorted(cs, np.float64(ud[i]) * cs[-1], side="right"))
            k = min(k, V - 1)
            out["draft_tokens"][slot, i] = k
            out["draft_q_tok"][slot, i] = q32[i, k]
        out["uniforms"][slot] = _unit_uniform(_rng(w.seed, _ARR_ACCEPT_U, b), g)
    out["uniforms_rs"][slot] = _unit_uniform(_rng(w.seed, _ARR_RESAMPLE_U, b), 1)[0]


def generate(w: Workload, b0: int = 0, b1: Optional[int] = None, threads: int = 1) -> Dict[str, np.ndarray]:
    """Generate sequences [b0, b1) of workload `w`.

    Returns host arrays:
      target_logits [n, gamma+1, V]  float32, or uint16 holding bf16 bit patterns
      draft_q       [n, gamma, V]    float32   (device-side Q_i)
      draft_tokens  [n, gamma]       int32     x_i
      draft_q_tok   [n, gamma]       float32   q_i(x_i)
      uniforms      [n, gamma]       float32   u_i
      uniforms_rs   [n]              float32   u'
    """
    if b1 is None:
        b1 = w.B
    n = b1 - b0
    g, V = w.gamma, w.V
    ldt = np.uint16 if w.dtype == "bf16" else np.float32
    out = {
        "target_logits": np.empty((n, g + 1, V), dtype=ldt),
        "draft_q": np.empty((n, g, V), dtype=np.float32),
        "draft_tokens": np.zeros((n, g), dtype=np.int32),
        "draft_q_tok": np.zeros((n, g), dtype=np.float32),
        "uniforms": np.zeros((n, g), dtype=np.float32),
        "uniforms_rs": np.zeros((n,), dtype=np.float32),
    }
    beta = zipf_bias(w)
    if threads <= 1 or n <= 1:
        for s in range(n):
            _gen_sequence(w, b0 + s, beta, out, s)
    else:
        from concurrent.futures import ThreadPoolExecutor

        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(lambda s: _gen_sequence(w, b0 + s, beta, out, s), range(n)))
    return out


def generate_topk(w: Workload, k: int, b0: int = 0, b1: Optional[int] = None,
                  threads: int = 1) -> Dict[str, np.ndarray]:
    """Sequences [b0, b1) of workload `w` with the draft side truncated to its top k.

    Returns target_logits, uniforms, uniforms_rs as `generate` does, and
      q_idx        [n, gamma, k]  int32    support of the truncated Q_i, most likely first
      q_val        [n, gamma, k]  float32  its renormalised probabilities
      draft_tokens [n, gamma]     int32    x_i drawn from the truncated Q_i
      draft_q_tok  [n, gamma]     float32  the stored q_val entry of x_i
    """
    if b1 is None:
        b1 = w.B
    n, g = b1 - b0, w.gamma
    assert 1 <= k <= w.V
    out = {
        "q_idx": np.zeros((n, g, k), dtype=np.int32),
        "q_val": np.zeros((n, g, k), dtype=np.float32),
        "draft_tokens": np.zeros((n, g), dtype=np.int32),
        "draft_q_tok": np.zeros((n, g), dtype=np.float32),
    }
    ldt = np.uint16 if w.dtype == "bf16" else np.float32
    out["target_logits"] = np.empty((n, g + 1, w.V), dtype=ldt)
    out["uniforms"] = np.zeros((n, g), dtype=np.float32)
    out["uniforms_rs"] = np.zeros((n,), dtype=np.float32)
    beta = zipf_bias(w)

    def one(s: int) -> None:
        dense = {
            "target_logits": out["target_logits"][s:s + 1],
            "draft_q": np.empty((1, g, w.V), dtype=np.float32),
            "draft_tokens": np.zeros((1, g), dtype=np.int32),
            "draft_q_tok": np.zeros((1, g), dtype=np.float32),
            "uniforms": out["uniforms"][s:s + 1],
            "uniforms_rs": out["uniforms_rs"][s:s + 1],
        }
        _gen_sequence(w, b0 + s, beta, dense, 0)
        if g == 0:
            return
        ud = _unit_uniform(_rng(w.seed, _ARR_DRAFT_U, b0 + s), g)
        for i in range(g):
            q = dense["draft_q"][0, i]
            # the k largest entries, equal entries by increasing index
            cand = np.argpartition(-q, min(k, w.V - 1))[:k] if k < w.V else np.arange(w.V)
            kth = q[cand].min()
            pool = np.flatnonzero(q >= kth)
            order = pool[np.argsort(-q[pool], kind="stable")][:k]
            vals = q[order].astype(np.float64)
            vals /= vals.sum()
            v32 = vals.astype(np.float32)
            out["q_idx"][s, i] = order
            out["q_val"][s, i] = v32
            cs = np.cumsum(v32, dtype=np.float64)
            r = int(np.searchsorted(cs, np.float64(ud[i]) * cs[-1], side="right"))
            r = min(r, k - 1)
            out["draft_tokens"][s, i] = order[r]
            out["draft_q_tok"][s, i] = v32[r]

    if threads <= 1 or n <= 1:
        for s in range(n):
            one(s)
    else:
        from concurrent.futures import ThreadPoolExecutor

        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(one, range(n)))
    return out
