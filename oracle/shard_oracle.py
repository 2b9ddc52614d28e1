"""CPU oracle of the vocabulary-sharded verification round (numpy, float64).

TEST INFRASTRUCTURE ONLY: imported by the tests and by the benchmark's CPU-baseline leg; the
CUDA library and its binding never import this module, and it shares no code with them.

The vocabulary is cut into G contiguous shards [v_0, v_1), [v_1, v_2), ... (a tensor-parallel
LM head leaves each GPU with such a slice of every logit row).  Algorithm 2 of the paper
("Verification Process", "Downlink Transmission", "Resample"; Section 3) is unchanged; only the
sums over the vocabulary are formed shard by shard and combined:

  edge, per shard g and row (b, i):    m_g = max_{v in g} z_v,  S_g = sum_{v in g} exp(z_v - m_g),
                                       z = l / T; and z_{x_i} where the shard holds token x_i
  combine over shards:                 M = max_g m_g,  lse = M + ln sum_g S_g exp(m_g - M),
                                       p_i(x_i) = exp(z_{x_i} - lse), the acceptance test
                                       u_i < min(1, p_i(x_i) / q_i(x_i)) and the first rejection n
  edge, per shard:                     its slice of the row P_n(v) = exp(z_v - lse_n), as float32
  resample, per shard:                 R_g = sum_{v in g} max(0, p_v - q_v)  (p_v alone for the bonus draw)
                                       and the plain mass sum_{v in g} p_v (for the fall-back)
  resample, draw:                      Z = sum_g R_g, t = u' Z; the shard whose running total first
                                       exceeds t walks its slice for min{k : C_k > t}

Every function is plain index-order float64 arithmetic on whole arrays; nothing is blocked or
fused beyond the sharding that defines the method.  The non-finite, bad-token, fall-back and
clamping rules are those of the dense oracle (dssd_oracle.c), restated for shards.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

FLAG_BAD_TOKEN = 1
FLAG_NONFINITE = 2
RS_FLAG_BONUS = 1
RS_FLAG_FALLBACK = 2
RS_FLAG_INVALID = 4


def shard_bounds(V: int, G: int) -> List[Tuple[int, int]]:
    """G contiguous slices of [0, V) whose lengths differ by at most one (the first V % G are longer)."""
    base, extra = divmod(V, G)
    out, v = [], 0
    for g in range(G):
        n = base + (1 if g < extra else 0)
        out.append((v, v + n))
        v += n
    return out


def _widen(logits: np.ndarray) -> np.ndarray:
    """float32, or uint16 holding bfloat16 bit patterns, to float64 (exact)."""
    if logits.dtype == np.uint16:
        return (logits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return np.asarray(logits, dtype=np.float32).astype(np.float64)


def edge_partial(logits_shard: np.ndarray, draft_tokens: np.ndarray, v_begin: int,
                 temperature: float) -> Dict[str, np.ndarray]:
    """One shard's share of every row's log-sum-exp (Section 3, "Verification Process").
    logits_shard [B, gamma+1, Vs]; draft_tokens [B, gamma] are ids in the whole vocabulary.
    Returns m, S [B, gamma+1] (m = -inf, S = 0 for a slice of -inf only; m = NaN when the slice
    holds a NaN) and z_tok [B, gamma]: z of the drafted token where this shard holds it, else NaN."""
    T = float(np.float32(temperature))
    z = _widen(logits_shard) / T
    B, g1, Vs = z.shape
    m = np.max(z, axis=2) if Vs else np.full((B, g1), -np.inf)  # NaN propagates
    with np.errstate(invalid="ignore", over="ignore"):
        S = np.zeros((B, g1))
        for b in range(B):
            for i in range(g1):
                if np.isfinite(m[b, i]):
                    S[b, i] = np.sum(np.exp(z[b, i] - m[b, i]))  # index order within the slice
                elif m[b, i] == np.inf or np.isnan(m[b, i]):
                    S[b, i] = np.nan
    gamma = g1 - 1
    z_tok = np.full((B, gamma), np.nan)
    x = np.asarray(draft_tokens, dtype=np.int64).reshape(B, gamma) - v_begin
    for b in range(B):
        for i in range(gamma):
            if 0 <= x[b, i] < Vs:
                z_tok[b, i] = z[b, i, x[b, i]]
    return {"m": m, "S": S, "z_tok": z_tok}


def edge_combine(parts: Sequence[Dict[str, np.ndarray]], draft_tokens: np.ndarray, draft_q_tok: np.ndarray,
                 uniforms: np.ndarray, V: int) -> Dict[str, np.ndarray]:
    """The shards' partial sums -> every row's log-sum-exp, p_i(x_i), the acceptance test
    u_i < min(1, p_i(x_i)/q_i(x_i)) and the first rejection n (Algorithm 2, "Verification Process").
    V is the size of the whole vocabulary (token ids outside [0, V) are rejected and flagged)."""
    m = np.stack([p["m"] for p in parts])  # [G, B, gamma+1]
    S = np.stack([p["S"] for p in parts])
    zt = np.stack([p["z_tok"] for p in parts])  # [G, B, gamma]
    G, B, g1 = m.shape
    gamma = g1 - 1
    tok = np.asarray(draft_tokens, dtype=np.int64).reshape(B, gamma)
    q_tok = np.asarray(draft_q_tok, dtype=np.float32).astype(np.float64).reshape(B, gamma)
    u = np.asarray(uniforms, dtype=np.float32).astype(np.float64).reshape(B, gamma)
    lse = np.full((B, g1), np.nan)
    p_tok = np.full((B, gamma), np.nan)
    accept_len = np.zeros(B, np.int32)
    flags = np.zeros(B, np.uint32)
    margin = np.full(B, np.inf)
    for b in range(B):
        for i in range(g1):
            M = -np.inf
            bad = False
            for g in range(G):
                if np.isnan(m[g, b, i]):
                    bad = True
                elif m[g, b, i] > M:
                    M = m[g, b, i]
            if bad or not np.isfinite(M):
                flags[b] |= FLAG_NONFINITE
                continue
            tot = 0.0
            for g in range(G):  # shard order
                if m[g, b, i] > -np.inf:
                    tot += S[g, b, i] * np.exp(m[g, b, i] - M)
            val = M + np.log(tot)
            if np.isfinite(val):
                lse[b, i] = val
            else:
                flags[b] |= FLAG_NONFINITE
        n, open_ = gamma, True
        for i in range(gamma):
            x = tok[b, i]
            if x < 0 or x >= V:
                flags[b] |= FLAG_BAD_TOKEN
                ratio, accept = np.nan, False
            else:
                zx = np.nan
                for g in range(G):  # the one shard that holds x reports its z
                    if not np.isnan(zt[g, b, i]):
                        zx = zt[g, b, i]
                with np.errstate(invalid="ignore", over="ignore"):
                    p = np.exp(zx - lse[b, i])
                p_tok[b, i] = p
                q = q_tok[b, i]
                if np.isnan(q) or np.isnan(p):
                    ratio = np.nan
                elif q <= 0.0:
                    ratio = np.inf if p > 0.0 else 0.0
                else:
                    ratio = p / q
                accept = (not np.isnan(ratio)) and (u[b, i] < min(ratio, 1.0))
            if open_:
                if not np.isnan(ratio):
                    margin[b] = min(margin[b], abs(u[b, i] - min(ratio, 1.0)))
                if not accept:
                    n, open_ = i, False
        accept_len[b] = n
    return {"accept_len": accept_len, "lse": lse, "p_tok": p_tok, "flags": flags, "margin_acc": margin}


def edge_emit_shard(logits_shard: np.ndarray, accept_len: np.ndarray, lse: np.ndarray,
                    temperature: float) -> np.ndarray:
    """This shard's slice of the downlink row P_n(v) = exp(z_v - lse_n), rounded to float32
    (Section 3, "Downlink Transmission"; NaN where row n has no finite log-sum-exp)."""
    T = float(np.float32(temperature))
    z = _widen(logits_shard) / T
    B = z.shape[0]
    out = np.empty((B, z.shape[2]), np.float32)
    with np.errstate(invalid="ignore", over="ignore"):
        for b in range(B):
            n = int(accept_len[b])
            out[b] = np.exp(z[b, n] - lse[b, n]).astype(np.float32)
    return out


def _residual(p_row_shard: np.ndarray, q_shard: Optional[np.ndarray], n: int, gamma: int, b: int) -> np.ndarray:
    # max(0, p - q) as C's fmax forms it in the dense oracle: a NaN difference counts as no mass
    p = p_row_shard[b].astype(np.float64)
    if n < gamma:
        return np.fmax(0.0, p - q_shard[b, n].astype(np.float64))
    return p


def resample_shard_mass(p_row_shard: np.ndarray, draft_q_shard: Optional[np.ndarray], accept_len: np.ndarray,
                        gamma: int) -> np.ndarray:
    """[B, 2]: this shard's residual mass sum_v max(0, p_v - q_v) (sum_v p_v for a bonus draw,
    n == gamma) and its plain mass sum_v p_v (Section 3, "Resample").  Rows with n outside
    [0, gamma] get NaN."""
    B = p_row_shard.shape[0]
    out = np.zeros((B, 2))
    for b in range(B):
        n = int(accept_len[b])
        if n < 0 or n > gamma:
            out[b] = np.nan
            continue
        r = _residual(p_row_shard, draft_q_shard, n, gamma, b)
        out[b, 0] = np.cumsum(r)[-1] if r.size else 0.0  # sequential, index order
        pp = p_row_shard[b].astype(np.float64)
        out[b, 1] = np.cumsum(pp)[-1] if pp.size else 0.0
    return out


def resample_shard_draw(masses: np.ndarray, g: int, v_begin: int, p_row_shard: np.ndarray,
                        draft_q_shard: Optional[np.ndarray], accept_len: np.ndarray, uniforms_rs: np.ndarray,
                        gamma: int) -> Dict[str, np.ndarray]:
    """The draw as shard g sees it, given every shard's masses [G, B, 2].  All shards reach the
    same verdict on Z, the fall-back and the owning shard; the owner returns the token's id in
    the whole vocabulary, the others -1.  flags are the sequence's (identical on every shard)."""
    G, B, _ = masses.shape
    token = np.full(B, -1, np.int32)
    flags = np.zeros(B, np.uint32)
    margin = np.full(B, np.inf)
    Zs = np.zeros(B)
    owner = np.full(B, -1, np.int32)
    u = np.asarray(uniforms_rs, dtype=np.float32).astype(np.float64)
    for b in range(B):
        n = int(accept_len[b])
        if n < 0 or n > gamma:
            flags[b] = RS_FLAG_INVALID
            margin[b] = 0.0
            continue
        fl = RS_FLAG_BONUS if n == gamma else 0
        col, Z = 0, 0.0
        for h in range(G):
            Z += masses[h, b, 0]
        use_q = n < gamma
        if not (Z > 0.0 and np.isfinite(Z)):
            if n == gamma:
                flags[b] = fl | RS_FLAG_INVALID
                margin[b] = 0.0
                continue
            fl |= RS_FLAG_FALLBACK
            col, use_q, Z = 1, False, 0.0
            for h in range(G):
                Z += masses[h, b, 1]
            if not (Z > 0.0 and np.isfinite(Z)):
                flags[b] = fl | RS_FLAG_INVALID
                margin[b] = 0.0
                continue
        t = u[b] * Z
        C, own, before, beyond = 0.0, -1, 0.0, False
        for h in range(G):
            if C + masses[h, b, col] > t:
                own, before = h, C
                break
            C += masses[h, b, col]
        if own < 0:  # rounding left no shard above t: the last shard with mass, its last positive entry
            beyond = True
            for h in range(G):
                if masses[h, b, col] > 0.0:
                    own = h
        flags[b] = fl
        Zs[b] = Z
        owner[b] = own
        if own != g:
            continue
        p = p_row_shard[b].astype(np.float64)
        r = np.fmax(0.0, p - draft_q_shard[b, n].astype(np.float64)) if use_q else p
        c = np.cumsum(r)
        pos = np.nonzero(r > 0.0)[0]
        k = r.size if beyond else int(np.searchsorted(c, t - before, side="right"))
        if k >= r.size:
            token[b] = v_begin + int(pos[-1]) if pos.size else -1
            margin[b] = 0.0
        else:
            below = c[k - 1] if k > 0 else 0.0
            token[b] = v_begin + k
            margin[b] = min((t - before) - below, c[k] - (t - before)) / Z
    return {"token": token, "flags": flags, "margin_cdf": margin, "Z": Zs, "owner": owner}


def verify_round_sharded(inputs: Dict[str, np.ndarray], temperature: float,
                         bounds: Sequence[Tuple[int, int]]) -> Dict[str, np.ndarray]:
    """The whole round over the given shards: what G ranks compute, with the two exchanges
    (partial sums, masses) written as plain stacking."""
    tl, dq = inputs["target_logits"], inputs.get("draft_q")
    B, g1, V = tl.shape
    gamma = g1 - 1
    parts = [edge_partial(tl[:, :, a:b_], inputs["draft_tokens"], a, temperature) for a, b_ in bounds]
    ev = edge_combine(parts, inputs["draft_tokens"], inputs["draft_q_tok"], inputs["uniforms"], V)
    rows = [edge_emit_shard(tl[:, :, a:b_], ev["accept_len"], ev["lse"], temperature) for a, b_ in bounds]
    qs = [dq[:, :, a:b_] if gamma else None for a, b_ in bounds]
    masses = np.stack([resample_shard_mass(rows[g], qs[g], ev["accept_len"], gamma) for g in range(len(bounds))])
    draws = [resample_shard_draw(masses, g, bounds[g][0], rows[g], qs[g], ev["accept_len"], inputs["uniforms_rs"], gamma)
             for g in range(len(bounds))]
    out = dict(ev)
    out["parts"] = parts
    out["p_row"] = np.concatenate(rows, axis=1)
    out["masses"] = masses
    out["token"] = np.max(np.stack([d["token"] for d in draws]), axis=0)  # -1 everywhere but on the owner
    out["rs_flags"] = draws[0]["flags"]
    out["shard_tokens"] = np.stack([d["token"] for d in draws])
    out["shard_flags"] = np.stack([d["flags"] for d in draws])
    out["margin_cdf"] = np.min(np.stack([d["margin_cdf"] for d in draws]), axis=0)
    out["Z"] = draws[0]["Z"]
    out["owner"] = draws[0]["owner"]
    return out
