"""Closed forms the paper states for the accept/reject statistics (test infrastructure only).

Section 3.1: with acceptance rate alpha per draft token, all gamma drafts are
accepted with probability alpha**gamma, so a downlink row is sent with probability
1 - alpha**gamma and the expected communication time is
T_comm = (1 - alpha**gamma) * |V| b_prob / R_down + T_NTT.
"""
from __future__ import annotations

import numpy as np


def acceptance_rate(p: np.ndarray, q: np.ndarray) -> float:
    """alpha = sum_v min(p_v, q_v): probability that a token drawn from q passes u < min(1, p/q)."""
    return float(np.minimum(np.asarray(p, np.float64), np.asarray(q, np.float64)).sum())


def prob_rejection(alpha: float, gamma: int) -> float:
    """1 - alpha**gamma (Section 3.1)."""
    return 1.0 - alpha ** gamma


def expected_accept_len(alpha: float, gamma: int) -> float:
    """E[n] = sum_{k=1..gamma} alpha**k = alpha (1 - alpha**gamma) / (1 - alpha)."""
    if alpha == 1.0:
        return float(gamma)
    return alpha * (1.0 - alpha ** gamma) / (1.0 - alpha)


def t_comm_ms(alpha: float, gamma: int, t_ntt_ms: float, payload_ms: float) -> float:
    """Expected DSSD communication time (Section 3.1), payload_ms = |V| b_prob / R_down."""
    return prob_rejection(alpha, gamma) * payload_ms + t_ntt_ms


def batch_acceptance_rate(target_logits: np.ndarray, draft_q: np.ndarray, temperature: float, n_seq: int = 32) -> float:
    """Mean over the first n_seq sequences and their gamma draft positions of alpha = sum_v min(p_v, q_v)
    (Section 3.1's alpha), p = softmax(l / T) in float64.  Logits are float32, or uint16 holding bfloat16."""
    tl = target_logits[:n_seq]
    if tl.dtype == np.uint16:
        tl = (tl.astype(np.uint32) << 16).view(np.float32)
    gamma = tl.shape[1] - 1
    if gamma == 0:
        return float("nan")
    T = float(np.float32(temperature))
    total, count = 0.0, 0
    for b in range(tl.shape[0]):
        z = tl[b, :gamma].astype(np.float64) / T
        z -= z.max(axis=1, keepdims=True)
        p = np.exp(z)
        p /= p.sum(axis=1, keepdims=True)
        for i in range(gamma):
            total += acceptance_rate(p[i], draft_q[b, i])
            count += 1
    return total / count
