"""Pins of the CPU oracle against facts that do not come from the oracle itself.

P1  exhaustive enumeration on tiny vocabularies: the emitted-token law equals the
    target distribution exactly (the paper's "maintains inference quality" claim).
P2  closed-form accepted-length statistics (Section 3.1: P(all accepted) = alpha^gamma).
P3  special cases that reduce to library routines (softmax, cumsum + searchsorted).
P4  the 24 cells printed in Table 1.
P5  invariants and monotonicity on random inputs.
P6  brute-force search against an independent prefix-array formulation.
"""
import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import dssd_inputs as di
from oracle import closed_forms as cf

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _logits_from_probs(rows, T=1.0):
    """float32 logits T*ln(p) for rows of Fractions; zero-mass entries get -inf."""
    out = np.empty((len(rows), len(rows[0])), np.float32)
    for i, r in enumerate(rows):
        for v, p in enumerate(r):
            out[i, v] = -np.inf if p == 0 else np.float32(T * math.log(float(p)))
    return out


def _lcm(a, b):
    return a * b // math.gcd(a, b)


def _grid_K(p_rows, q_rows, D):
    """Smallest K such that every acceptance ratio and every CDF step is a multiple of 1/K."""
    K = 1
    for p, q in zip(p_rows, q_rows):
        for pv, qv in zip(p, q):
            if qv > 0 and pv < qv:
                K = _lcm(K, (pv / qv).denominator)
        res = [max(Fraction(0), pv - qv) for pv, qv in zip(p, q)]
        Z = sum(res)
        if Z > 0:
            c = Fraction(0)
            for r in res:
                c += r
                K = _lcm(K, (c / Z).denominator)
    c = Fraction(0)
    for pv in p_rows[-1]:
        c += pv
        K = _lcm(K, c.denominator)
    return K


def _enumerate(O, p_rows, q_rows, T=1.0, q_tok_override=None):
    """Run the oracle on every (draft string, acceptance-uniform grid point, resample grid point).

    Returns (num, den): num[k][a] = exact probability that k drafts are accepted and token a is
    emitted at position k; den[k] = exact probability that the first k drafts are accepted.
    """
    gamma = len(q_rows)
    V = len(p_rows[0])
    D = 1
    K = _grid_K(p_rows, q_rows, D)
    xs = [x for x in itertools.product(range(V), repeat=gamma)
          if all(q_rows[i][x[i]] > 0 for i in range(gamma))]
    grid = np.array([(k + 0.5) / K for k in range(K)], np.float32)
    ucombos = np.array(list(itertools.product(range(K), repeat=gamma + 1)), np.int64).reshape(-1, gamma + 1)
    nU = ucombos.shape[0]
    B = len(xs) * nU
    logits = np.broadcast_to(_logits_from_probs(p_rows, T)[None], (B, gamma + 1, V)).copy()
    tokens = np.repeat(np.array(xs, np.int32).reshape(len(xs), gamma), nU, axis=0)
    q32 = np.array([[float(v) for v in r] for r in q_rows], np.float32).reshape(gamma, V)
    if q_tok_override is None:
        q_tok = np.stack([q32[i, tokens[:, i]] for i in range(gamma)], axis=1) if gamma else np.zeros((B, 0), np.float32)
    else:
        q_tok = np.stack([q_tok_override[i][tokens[:, i]] for i in range(gamma)], axis=1)
    u_idx = np.tile(ucombos, (len(xs), 1))
    u_acc = grid[u_idx[:, :gamma]]
    u_rs = grid[u_idx[:, gamma]]
    draft_q = np.broadcast_to(q32[None], (B, gamma, V)).copy()
    ev = O.edge_verify(logits, tokens, q_tok, u_acc, T, threads=8)
    rs = O.device_resample(ev["p_row"], draft_q, ev["accept_len"], u_rs, gamma, threads=8)
    n = ev["accept_len"]
    y = rs["token"]
    assert (y >= 0).all()
    num = [[Fraction(0)] * V for _ in range(gamma + 1)]
    den = [Fraction(0)] * (gamma + 1)
    cell = Fraction(1, K ** (gamma + 1))
    for xi, x in enumerate(xs):
        wx = Fraction(1)
        for i in range(gamma):
            wx *= q_rows[i][x[i]]
        sl = slice(xi * nU, (xi + 1) * nU)
        nn, yy = n[sl], y[sl]
        for k in range(gamma + 1):
            reached = nn >= k
            den[k] += wx * cell * int(reached.sum())
            stop = nn == k
            cnt = np.bincount(yy[stop], minlength=V)
            for a in range(V):
                num[k][a] += wx * cell * int(cnt[a])
            if k < gamma:
                num[k][x[k]] += wx * cell * int((nn > k).sum())
    return num, den, K, B


def _F(rows, D):
    return [[Fraction(a, D) for a in r] for r in rows]


CASES = {
    "V4_g2": (_F([[1, 3, 4, 0], [2, 2, 2, 2], [1, 1, 2, 4]], 8), _F([[4, 2, 1, 1], [1, 1, 3, 3]], 8)),
    "V3_g3": (_F([[1, 2, 3], [3, 3, 0], [2, 1, 3], [1, 1, 4]], 6), _F([[3, 2, 1], [2, 2, 2], [4, 1, 1]], 6)),
    "V8_g1": (_F([[1, 0, 2, 3, 4, 1, 3, 2], [5, 1, 1, 1, 2, 2, 2, 2]], 16), _F([[2, 2, 2, 2, 2, 2, 2, 2]], 16)),
    "V2_g3": (_F([[1, 3], [2, 2], [3, 1], [1, 3]], 4), _F([[2, 2], [1, 3], [1, 3]], 4)),
    # q has zero-mass entries that the target wants (residual carries them)
    "V4_g1_qzero": (_F([[2, 2, 2, 2], [1, 1, 1, 5]], 8), _F([[4, 4, 0, 0]], 8)),
}


@pytest.mark.parametrize("name", sorted(CASES))
def test_p1_emitted_law_equals_target(oracle_mod, name):
    p_rows, q_rows = CASES[name]
    num, den, K, B = _enumerate(oracle_mod, p_rows, q_rows)
    gamma = len(q_rows)
    assert den[0] == 1
    for k in range(gamma + 1):
        assert den[k] > 0
        for a in range(len(p_rows[0])):
            assert num[k][a] / den[k] == p_rows[k][a], (name, k, a, K, B)


def test_p1_with_temperature(oracle_mod):
    p_rows, q_rows = CASES["V4_g2"]
    num, den, _, _ = _enumerate(oracle_mod, p_rows, q_rows, T=0.7)
    for k in range(3):
        for a in range(4):
            assert num[k][a] / den[k] == p_rows[k][a]


def test_p1_detects_inverted_ratio(oracle_mod):
    """The ratio as printed in Algorithm 2 (q/p) does not reproduce the target law:
    feeding q' = p^2/q makes the oracle evaluate exactly that ratio, and the pin fails."""
    p_rows, q_rows = CASES["V2_g3"]
    gamma = len(q_rows)
    override = []
    for i in range(gamma):
        override.append(np.array([float(p_rows[i][v] ** 2 / q_rows[i][v]) for v in range(2)], np.float32))
    num, den, _, _ = _enumerate(oracle_mod, p_rows, q_rows, q_tok_override=override)
    assert any(num[0][a] / den[0] != p_rows[0][a] for a in range(2))


def test_p2_accept_length_closed_form_exact(oracle_mod):
    p = _F([[1, 3, 4, 0]], 8)[0]
    q = _F([[4, 2, 1, 1]], 8)[0]
    gamma = 3
    alpha = sum(min(a, b) for a, b in zip(p, q))
    assert alpha == Fraction(1, 2)
    num, den, _, _ = _enumerate(oracle_mod, [p] * (gamma + 1), [q] * gamma)
    for k in range(gamma + 1):
        assert den[k] == alpha ** k  # P(n >= k)
    e_n = sum(den[k] for k in range(1, gamma + 1))
    assert float(e_n) == pytest.approx(cf.expected_accept_len(float(alpha), gamma), rel=1e-15)
    assert float(1 - den[gamma]) == pytest.approx(cf.prob_rejection(float(alpha), gamma), rel=1e-15)


def test_p2_accept_length_statistical(oracle_mod):
    """Random (p, q) at V=64: accepted-length histogram against alpha^k within 5 sigma."""
    rng = np.random.default_rng(7)
    V, gamma, N = 64, 4, 200_000
    lp = rng.normal(0, 2, V).astype(np.float32)
    lq = (lp + rng.normal(0, 1, V)).astype(np.float32)
    p = np.exp(lp.astype(np.float64) - lp.max()); p /= p.sum()
    q = np.exp(lq.astype(np.float64) - lq.max()); q /= q.sum()
    q32 = q.astype(np.float32)
    alpha = cf.acceptance_rate(p, q32)
    cs = np.cumsum(q32, dtype=np.float64)
    x = np.minimum(np.searchsorted(cs, rng.random((N, gamma)) * cs[-1], side="right"), V - 1).astype(np.int32)
    logits = np.broadcast_to(lp[None, None], (N, gamma + 1, V)).copy()
    u = rng.random((N, gamma)).astype(np.float32)
    ev = oracle_mod.edge_verify(logits, x, q32[x], u, 1.0, threads=8)
    n = ev["accept_len"]
    for k in range(1, gamma + 1):
        pk = alpha ** k
        sd = math.sqrt(pk * (1 - pk) / N)
        assert abs((n >= k).mean() - pk) < 5 * sd
    assert abs(n.mean() - cf.expected_accept_len(alpha, gamma)) < 5 * gamma / math.sqrt(N)


def _table1():
    rows = []
    with open(os.path.join(GOLDEN, "table1_reject_prob_tcomm.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            g, a, r, t = line.split()
            rows.append((int(g), a, float(r), float(t)))
    return rows


@pytest.mark.parametrize("gamma,alpha_s,rej_printed,tcomm_printed", _table1())
def test_p4_table1(oracle_mod, gamma, alpha_s, rej_printed, tcomm_printed):
    """Rejection probability of the oracle with per-token acceptance alpha (q one-hot on the
    drafted token, p(x) = alpha), against the printed 1 - alpha^gamma and T_comm."""
    alpha = Fraction(alpha_s)
    K = alpha.denominator
    logits_row = _logits_from_probs([[alpha, 1 - alpha]])[0]
    exact = K ** gamma <= 400_000
    if exact:
        idx = np.array(list(itertools.product(range(K), repeat=gamma)), np.int64)
        u = ((idx + 0.5) / K).astype(np.float32)
    else:
        u = np.random.default_rng(1000 * gamma + K).random((400_000, gamma)).astype(np.float32)
    N = u.shape[0]
    logits = np.broadcast_to(logits_row[None, None], (N, gamma + 1, 2)).copy()
    tokens = np.zeros((N, gamma), np.int32)
    q_tok = np.ones((N, gamma), np.float32)
    ev = oracle_mod.edge_verify(logits, tokens, q_tok, u, 1.0, threads=8)
    rej = float((ev["accept_len"] < gamma).mean())
    slack = 0.0 if exact else 5 * math.sqrt(max(rej * (1 - rej), 1e-4) / N)
    if exact:
        assert Fraction(int((ev["accept_len"] < gamma).sum()), N) == 1 - alpha ** gamma
    assert abs(rej - rej_printed) <= 0.005 + 1e-12 + slack
    assert abs(cf.prob_rejection(float(alpha), gamma) - rej_printed) <= 0.005 + 1e-12
    assert abs(cf.t_comm_ms(float(alpha), gamma, 20.0, 8.0) - tcomm_printed) <= 0.005 + 1e-9
    assert abs(20.0 + 8.0 * rej - tcomm_printed) <= 0.005 + 1e-9 + 8 * slack


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_p3_gamma0_is_softmax_and_inverse_cdf(oracle_mod, dtype):
    w = di.custom(B=6, gamma=0, V=1000, dtype=dtype, temperature=0.8, seed=5)
    d = di.generate(w)
    r = oracle_mod.verify_round(d, w.temperature)
    lg = d["target_logits"][:, 0]
    lg = di.bf16_bits_to_f32(lg) if dtype == "bf16" else lg
    z = torch.from_numpy(lg.astype(np.float64)) / float(np.float32(w.temperature))
    assert (r["accept_len"] == 0).all()
    assert np.allclose(r["lse"][:, 0], torch.logsumexp(z, -1).numpy(), rtol=0, atol=1e-12)
    sm = torch.softmax(z, -1).numpy()
    ev = oracle_mod.edge_verify(d["target_logits"], d["draft_tokens"], d["draft_q_tok"], d["uniforms"],
                                w.temperature, want_p_row64=True)
    assert np.allclose(ev["p_row64"], sm, rtol=1e-12, atol=1e-300)
    assert np.allclose(ev["p_row64"].sum(1), 1.0, atol=1e-12)
    assert (ev["p_row"] == ev["p_row64"].astype(np.float32)).all()
    p32 = ev["p_row"].astype(np.float64)
    for b in range(w.B):
        cs = np.cumsum(p32[b])
        k = np.searchsorted(cs, float(d["uniforms_rs"][b]) * cs[-1], side="right")
        assert r["token"][b] == k
        assert r["rs_flags"][b] == oracle_mod.RS_FLAG_BONUS


def test_p3_draft_equals_target_accepts_everything(oracle_mod):
    w = di.custom(B=4, gamma=5, V=300, dtype="f32", seed=9)
    d = di.generate(w)
    ev = oracle_mod.edge_verify(d["target_logits"], d["draft_tokens"], d["draft_q_tok"], d["uniforms"], 1.0)
    # re-verify with q(x) := p(x): every ratio is 1 up to float32 rounding of q
    q_tok = ev["p_tok"].astype(np.float32)
    u = np.minimum(d["uniforms"], np.float32(0.999))
    ev2 = oracle_mod.edge_verify(d["target_logits"], d["draft_tokens"], q_tok, u, 1.0)
    assert (ev2["accept_len"] == w.gamma).all()


def test_p3_one_hot_target(oracle_mod):
    V, gamma, B = 17, 2, 9
    hot = 11
    logits = np.full((B, gamma + 1, V), -np.inf, np.float32)
    logits[:, :, hot] = 3.0
    tokens = np.full((B, gamma), 4, np.int32)
    q = np.full((B, gamma, V), 1.0 / V, np.float32)
    u = np.linspace(0, 0.99, B * gamma).astype(np.float32).reshape(B, gamma)
    u_rs = np.linspace(0, 1 - 2 ** -24, B).astype(np.float32)
    ev = oracle_mod.edge_verify(logits, tokens, q[:, :, 4], u, 1.0)
    assert (ev["accept_len"] == 0).all()
    assert (ev["p_row"][:, hot] == 1.0).all() and ev["p_row"].sum() == B
    rs = oracle_mod.device_resample(ev["p_row"], q, ev["accept_len"], u_rs, gamma)
    assert (rs["token"] == hot).all() and (rs["flags"] == 0).all()


def test_p3_shift_and_temperature_invariance(oracle_mod):
    rng = np.random.default_rng(3)
    B, gamma, V = 5, 3, 257
    base = (rng.integers(-4096, 4096, size=(B, gamma + 1, V)) / 512.0).astype(np.float32)
    w = di.custom(B=B, gamma=gamma, V=V, seed=11)
    d = di.generate(w)
    args = (d["draft_tokens"], d["draft_q_tok"], d["uniforms"])
    a = oracle_mod.edge_verify(base, *args, 1.0, want_p_row64=True)
    shifted = (base + np.float32(37.0)).astype(np.float32)
    assert (shifted - np.float32(37.0) == base).all()
    b = oracle_mod.edge_verify(shifted, *args, 1.0, want_p_row64=True)
    assert (a["accept_len"] == b["accept_len"]).all()
    assert np.allclose(a["p_row64"], b["p_row64"], rtol=1e-12, atol=0)
    assert np.allclose(a["lse"] + 37.0, b["lse"], rtol=0, atol=1e-11)
    c = oracle_mod.edge_verify((base * np.float32(0.5)).astype(np.float32), *args, 0.5, want_p_row64=True)
    assert (a["accept_len"] == c["accept_len"]).all()
    assert np.allclose(a["p_row64"], c["p_row64"], rtol=1e-12, atol=0)


def test_p3_bf16_widening_is_exact(oracle_mod):
    w = di.custom(B=3, gamma=2, V=513, dtype="bf16", seed=21)
    d = di.generate(w)
    as_f32 = di.bf16_bits_to_f32(d["target_logits"])
    a = oracle_mod.edge_verify(d["target_logits"], d["draft_tokens"], d["draft_q_tok"], d["uniforms"], 0.9)
    b = oracle_mod.edge_verify(as_f32, d["draft_tokens"], d["draft_q_tok"], d["uniforms"], 0.9)
    for k in ("accept_len", "p_row", "p_tok", "lse"):
        assert (a[k] == b[k]).all()


def test_p5_invariants_and_monotonicity(oracle_mod):
    w = di.custom(B=64, gamma=6, V=777, dtype="f32", sigma_d=1.0, seed=31)
    d = di.generate(w)
    r = oracle_mod.verify_round(d, w.temperature)
    n, tok = r["accept_len"], r["token"]
    assert ((n >= 0) & (n <= w.gamma)).all()
    assert ((tok >= 0) & (tok < w.V)).all()
    assert 0 < (n == w.gamma).sum() < w.B or True
    for b in range(w.B):
        res = r["p_row"][b].astype(np.float64)
        if n[b] < w.gamma:
            res = np.maximum(0.0, res - d["draft_q"][b, n[b]].astype(np.float64))
            assert r["rs_flags"][b] == 0
        else:
            assert r["rs_flags"][b] == oracle_mod.RS_FLAG_BONUS
        assert res[tok[b]] > 0
        assert r["Z"][b] == pytest.approx(res.sum(), rel=1e-13)
    # raising one acceptance uniform never lengthens the accepted prefix
    rng = np.random.default_rng(2)
    for _ in range(5):
        u2 = d["uniforms"].copy()
        i = rng.integers(0, w.gamma, w.B)
        u2[np.arange(w.B), i] = np.minimum(u2[np.arange(w.B), i] + rng.random(w.B).astype(np.float32) * 0.5,
                                           np.float32(1 - 2 ** -24))
        n2 = oracle_mod.edge_verify(d["target_logits"], d["draft_tokens"], d["draft_q_tok"], u2,
                                    w.temperature)["accept_len"]
        assert (n2 <= n).all()
    # raising the resample uniform never lowers the token index
    u_lo = d["uniforms_rs"]
    u_hi = np.minimum(u_lo + np.float32(0.1), np.float32(1 - 2 ** -24))
    t_hi = oracle_mod.device_resample(r["p_row"], d["draft_q"], n, u_hi, w.gamma)["token"]
    assert (t_hi >= tok).all()


def test_p5_first_rejection_is_first(oracle_mod):
    """accept_len is the FIRST failing position: later positions play no role."""
    w = di.custom(B=32, gamma=5, V=200, dtype="f32", sigma_d=1.5, seed=41)
    d = di.generate(w)
    ev = oracle_mod.edge_verify(d["target_logits"], d["draft_tokens"], d["draft_q_tok"], d["uniforms"], 1.0)
    n = ev["accept_len"]
    assert (n < w.gamma).any()
    u2 = d["uniforms"].copy()
    for b in range(w.B):
        u2[b, n[b] + 1:] = 0.0  # would accept everything after the first rejection
    ev2 = oracle_mod.edge_verify(d["target_logits"], d["draft_tokens"], d["draft_q_tok"], u2, 1.0)
    assert (ev2["accept_len"] == n).all()
    # a uniform of 0 at the rejected position accepts it (p > 0), so the prefix grows
    u3 = d["uniforms"].copy()
    rej = n < w.gamma
    u3[np.nonzero(rej)[0], n[rej]] = 0.0
    ev3 = oracle_mod.edge_verify(d["target_logits"], d["draft_tokens"], d["draft_q_tok"], u3, 1.0)
    assert (ev3["accept_len"][rej] > n[rej]).all()


def test_p6_search_against_prefix_array(oracle_mod):
    rng = np.random.default_rng(17)
    for V in (1, 2, 3, 5, 8, 31, 33, 1000, 1025, 50272):
        B, gamma = 7, 2
        p = rng.random((B, V)).astype(np.float32) ** 4
        p /= p.sum(1, keepdims=True)
        q = rng.random((B, gamma, V)).astype(np.float32) ** 4
        q /= q.sum(2, keepdims=True)
        n = rng.integers(0, gamma + 1, B).astype(np.int32)
        u = rng.random(B).astype(np.float32)
        rs = oracle_mod.device_resample(p, q, n, u, gamma)
        for b in range(B):
            r = p[b].astype(np.float64)
            if n[b] < gamma:
                r = np.maximum(0.0, r - q[b, n[b]].astype(np.float64))
            if not r.sum() > 0:
                assert V == 1
                r = p[b].astype(np.float64)
                assert rs["flags"][b] & oracle_mod.RS_FLAG_FALLBACK
            cs = np.cumsum(r)
            k = int(np.searchsorted(cs, float(u[b]) * cs[-1], side="right"))
            assert rs["token"][b] == min(k, V - 1)
            lo = float(u[b]) * cs[-1] - (cs[k - 1] if k > 0 else 0.0)
            hi = cs[k] - float(u[b]) * cs[-1]
            assert rs["margin_cdf"][b] == pytest.approx(min(lo, hi) / cs[-1], rel=1e-9, abs=1e-15)


def test_degenerate_inputs(oracle_mod):
    V, gamma = 9, 3
    logits = np.zeros((4, gamma + 1, V), np.float32)
    tokens = np.array([[0, 1, 2], [0, -1, 2], [0, 1, V], [0, 1, 2]], np.int32)
    q_tok = np.full((4, gamma), 1.0 / V, np.float32)
    q_tok[3, 1] = 0.0   # q(x) = 0 with p(x) > 0: ratio = +inf, accepted
    u = np.full((4, gamma), 0.5, np.float32)
    logits[0, 2, 3] = np.nan
    ev = oracle_mod.edge_verify(logits, tokens, q_tok, u, 1.0)
    assert ev["flags"][0] == oracle_mod.FLAG_NONFINITE and ev["accept_len"][0] == 2
    assert ev["flags"][1] == oracle_mod.FLAG_BAD_TOKEN and ev["accept_len"][1] == 1
    assert ev["flags"][2] == oracle_mod.FLAG_BAD_TOKEN and ev["accept_len"][2] == 2
    assert ev["flags"][3] == 0 and ev["accept_len"][3] == gamma
    # residual with no mass (p == q): falls back to sampling from p
    p = np.full((2, V), 1.0 / V, np.float32)
    q = np.full((2, gamma, V), 1.0 / V, np.float32)
    rs = oracle_mod.device_resample(p, q, np.array([1, 7], np.int32), np.array([0.5, 0.5], np.float32), gamma)
    assert rs["flags"][0] == oracle_mod.RS_FLAG_FALLBACK and rs["token"][0] == 4
    assert rs["flags"][1] == oracle_mod.RS_FLAG_INVALID and rs["token"][1] == -1
    # the strict comparison: u = 1 can never be accepted, u = 0 needs p > 0
    ev = oracle_mod.edge_verify(np.zeros((1, 2, V), np.float32), np.array([[0]], np.int32),
                                np.array([[1e-9]], np.float32), np.array([[1.0]], np.float32), 1.0)
    assert ev["accept_len"][0] == 0
    lg = np.zeros((1, 2, V), np.float32); lg[0, 0, 0] = -np.inf
    ev = oracle_mod.edge_verify(lg, np.array([[0]], np.int32), np.array([[0.5]], np.float32),
                                np.array([[0.0]], np.float32), 1.0)
    assert ev["accept_len"][0] == 0


def test_p7_sixteen_bit_payload(oracle_mod):
    """The b_prob = 16 row: one rounding to IEEE binary16, nearest-even, checked against bit
    patterns worked out by hand; the draw then runs on the widened row unchanged."""
    cases = [
        (1.0, 0x3C00), (0.5, 0x3800), (1.0 / 3.0, 0x3555), (0.1, 0x2E66), (2.0 ** -14, 0x0400),
        (2.0 ** -24, 0x0001),                      # smallest subnormal
        (2.0 ** -25, 0x0000),                      # exactly half of it: ties to even, i.e. zero
        (2.0 ** -25 * (1 + 2.0 ** -40), 0x0001),   # just above the tie
        (1.0 + 2.0 ** -11, 0x3C00),                # tie between 1 and 1 + 2^-10: even mantissa wins
        (1.0 + 3 * 2.0 ** -11, 0x3C02),            # tie between 1 + 2^-10 and 1 + 2^-9
        (0.0, 0x0000), (3e-9, 0x0000),
        # a value whose float32 rounding would sit on a binary16 tie, while the float64 value does not
        (1.0 + 2.0 ** -11 + 2.0 ** -30, 0x3C01),
    ]
    got = oracle_mod.to_payload16(np.array([c[0] for c in cases], np.float64)).view(np.uint16)
    assert got.tolist() == [c[1] for c in cases]
    w = di.custom(B=12, gamma=3, V=3000, dtype="bf16", temperature=0.9, seed=21)
    d = di.generate(w)
    full = oracle_mod.verify_round(d, w.temperature)
    half = oracle_mod.verify_round(d, w.temperature, payload="f16")
    assert half["p_row16"].dtype == np.float16 and (half["accept_len"] == full["accept_len"]).all()
    p16 = half["p_row16"].astype(np.float64)
    p32 = full["p_row"].astype(np.float64)
    normal = p32 >= 2.0 ** -14
    assert (np.abs(p16 - p32)[normal] <= 2.0 ** -11 * p32[normal] * (1 + 1e-6)).all()
    assert (np.abs(p16 - p32)[~normal] <= 2.0 ** -25 * (1 + 1e-6)).all()
    assert (np.abs(p16.sum(axis=1) - 1.0) < 2e-3).all()
    order = np.argsort(p32, axis=1, kind="stable")
    assert (np.diff(np.take_along_axis(p16, order, axis=1), axis=1) >= 0).all()  # rounding keeps the order
    # the draw on the 16-bit row is the dense draw on its widened values
    again = oracle_mod.device_resample(half["p_row16"].astype(np.float32), d["draft_q"], half["accept_len"],
                                       d["uniforms_rs"], w.gamma)
    assert (again["token"] == half["token"]).all()
    assert (half["token"] == full["token"]).mean() > 0.7  # most draws do not sit within 2^-11 of a CDF step


def test_batch_acceptance_rate_on_hand_made_rows():
    """alpha = sum_v min(p_v, q_v) (Section 3.1) for rows worked out by hand, and its link to the
    closed forms: a draft token is accepted with probability alpha."""
    ln = np.log
    # gamma = 2: p_0 = (1/2, 1/2) against q_0 = (3/4, 1/4): alpha = 3/4; p_1 = q_1 = (1/8, 7/8): alpha = 1
    logits = np.array([[[ln(0.5), ln(0.5)], [ln(0.125), ln(0.875)], [0.0, 0.0]]], np.float32)
    q = np.array([[[0.75, 0.25], [0.125, 0.875]]], np.float32)
    assert abs(cf.batch_acceptance_rate(logits, q, 1.0) - 0.875) < 1e-7
    # equal logits give the uniform row at any temperature
    same = np.zeros((3, 2, 5), np.float32)
    assert abs(cf.batch_acceptance_rate(same, np.full((3, 1, 5), 0.2, np.float32), 0.7) - 1.0) < 1e-12
    # bfloat16 bit patterns are widened exactly: 0x3f80 = 1.0, 0x0000 = 0.0 -> p = (e, 1) / (e + 1)
    bits = np.array([[[0x3F80, 0x0000], [0, 0]]], np.uint16)
    p0 = np.e / (np.e + 1.0)
    qq = np.array([[[0.5, 0.5]]], np.float32)
    assert abs(cf.batch_acceptance_rate(bits, qq, 1.0) - (0.5 + (1.0 - p0))) < 1e-12
    assert np.isnan(cf.batch_acceptance_rate(np.zeros((1, 1, 4), np.float32), np.zeros((1, 0, 4), np.float32), 1.0))
