"""Pins of the truncated-support (top-k) oracle against facts that do not come from it.

K1  brute force: the support equals Python's sort by (logit descending, index ascending).
K2  closed forms: equal logits share the mass equally; a gap of T ln 2 halves a probability.
K3  reduction to the dense oracle (itself pinned in test_oracle_pins.py): with every logit
    outside the brute-force support set to -inf, the dense round gives the same decisions.
K4  k = V is the dense round.
K5  the truncated draw equals the dense draw on the scattered vectors.
K6  exhaustive enumeration: the emitted-token law is the truncated target distribution exactly.
K7  invalid arguments are refused.
"""
from fractions import Fraction

import numpy as np
import pytest

import dssd_inputs as di
from test_oracle_pins import _F, _enumerate


def _as_f64(logits):
    return di.bf16_bits_to_f32(logits).astype(np.float64) if logits.dtype == np.uint16 else logits.astype(np.float64)


def _brute_support(row64, k):
    return sorted(range(len(row64)), key=lambda v: (-row64[v], v))[:k]


def _tie_heavy(rng, B, g1, V, dtype):
    l = rng.integers(-3, 4, size=(B, g1, V)).astype(np.float32) * np.float32(0.5)
    l[rng.random(size=l.shape) < 0.05] = -np.inf
    l[:, :, 0] = np.maximum(l[:, :, 0], -1.0)  # at least one finite entry per row
    return di.f32_to_bf16_bits(l) if dtype == "bf16" else l


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V,k", [(7, 1), (7, 7), (40, 3), (64, 10), (200, 32)])
def test_k1_support_is_the_sorted_prefix(oracle_mod, dtype, V, k):
    rng = np.random.default_rng(1000 * V + k)
    B = 24
    for logits in (_tie_heavy(rng, B, 1, V, dtype),
                   (lambda x: di.f32_to_bf16_bits(x) if dtype == "bf16" else x)(
                       rng.standard_normal((B, 1, V)).astype(np.float32) * 3)):
        ev = oracle_mod.edge_verify_topk(logits, np.zeros((B, 0), np.int32), np.zeros((B, 0), np.float32),
                                         np.zeros((B, 0), np.float32), 0.9, k)
        l64 = _as_f64(logits)
        for b in range(B):
            assert ev["accept_len"][b] == 0
            want = _brute_support(l64[b, 0], k)
            assert ev["p_idx"][b].tolist() == want
            z = l64[b, 0, want] / np.float64(np.float32(0.9))
            e = np.exp(z - z.max())
            np.testing.assert_allclose(ev["p_val64"][b], e / e.sum(), rtol=1e-14, atol=0)
            assert abs(ev["p_val64"][b].sum() - 1.0) < 1e-14
            np.testing.assert_array_equal(ev["p_val"][b], ev["p_val64"][b].astype(np.float32))


def test_k2_closed_forms(oracle_mod):
    T = 0.5
    c = 1.25
    step = np.float32(T * np.log(2.0))
    # entries 1, 4, 6 tie at the top; 2 and 5 sit T ln 2 below; the rest far below
    row = np.full(9, -20.0, np.float32)
    row[[1, 4, 6]] = c
    row[[2, 5]] = np.float32(c) - step
    logits = row[None, None, :]
    none = (np.zeros((1, 0), np.int32), np.zeros((1, 0), np.float32), np.zeros((1, 0), np.float32))
    ev = oracle_mod.edge_verify_topk(logits, *none, T, 3)
    assert ev["p_idx"][0].tolist() == [1, 4, 6]
    np.testing.assert_allclose(ev["p_val64"][0], [1 / 3] * 3, rtol=1e-15)
    ev = oracle_mod.edge_verify_topk(logits, *none, T, 2)
    assert ev["p_idx"][0].tolist() == [1, 4]  # the tie is cut toward the lower index
    np.testing.assert_allclose(ev["p_val64"][0], [0.5, 0.5], rtol=1e-15)
    ev = oracle_mod.edge_verify_topk(logits, *none, T, 5)
    assert ev["p_idx"][0].tolist() == [1, 4, 6, 2, 5]
    np.testing.assert_allclose(ev["p_val64"][0], [0.25, 0.25, 0.25, 0.125, 0.125], rtol=1e-6)
    # acceptance: x inside the support with p/q = 0.25/0.5, x outside it has p = 0
    tok = np.array([[4, 0]], np.int32)
    two = np.repeat(logits, 3, axis=1)
    for u0, want_n in ((0.49, 1), (0.51, 0)):
        ev = oracle_mod.edge_verify_topk(two, tok, np.array([[0.5, 0.3]], np.float32),
                                         np.array([[u0, 0.0]], np.float32), T, 5)
        assert ev["accept_len"][0] == want_n
        np.testing.assert_allclose(ev["p_tok"][0], [0.25, 0.0], rtol=1e-6)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_k3_reduces_to_the_dense_round_on_masked_logits(oracle_mod, dtype):
    k = 10
    w = di.custom(B=48, gamma=4, V=700, dtype=dtype, temperature=0.8, sigma_d=0.5, seed=77)
    inp = di.generate_topk(w, k)
    ev = oracle_mod.edge_verify_topk(inp["target_logits"], inp["draft_tokens"], inp["draft_q_tok"],
                                     inp["uniforms"], w.temperature, k)
    l64 = _as_f64(inp["target_logits"])
    masked = np.full(l64.shape, -np.inf, np.float32)
    for b in range(w.B):
        for i in range(w.gamma + 1):
            s = _brute_support(l64[b, i], k)
            masked[b, i, s] = l64[b, i, s].astype(np.float32)
    dense = oracle_mod.edge_verify(masked, inp["draft_tokens"], inp["draft_q_tok"], inp["uniforms"],
                                   w.temperature, want_p_row64=True)
    assert (dense["margin_acc"] > 1e-9).all()  # no decision sits on a rounding edge
    np.testing.assert_array_equal(ev["accept_len"], dense["accept_len"])
    np.testing.assert_allclose(ev["p_tok"], dense["p_tok"], rtol=1e-13, atol=0)
    assert len(set(ev["accept_len"].tolist())) >= 3
    for b in range(w.B):
        row = np.zeros(w.V)
        row[ev["p_idx"][b]] = ev["p_val64"][b]
        np.testing.assert_allclose(row, dense["p_row64"][b], rtol=1e-13, atol=0)


def test_k4_k_equal_to_V_is_the_dense_round(oracle_mod):
    w = di.custom(B=16, gamma=3, V=24, dtype="f32", temperature=1.0, sigma_d=0.6, seed=5)
    inp = di.generate(w)
    ev = oracle_mod.edge_verify_topk(inp["target_logits"], inp["draft_tokens"], inp["draft_q_tok"],
                                     inp["uniforms"], w.temperature, w.V)
    dense = oracle_mod.edge_verify(inp["target_logits"], inp["draft_tokens"], inp["draft_q_tok"],
                                   inp["uniforms"], w.temperature, want_p_row64=True)
    np.testing.assert_array_equal(ev["accept_len"], dense["accept_len"])
    np.testing.assert_allclose(ev["p_tok"], dense["p_tok"], rtol=1e-13)
    for b in range(w.B):
        assert sorted(ev["p_idx"][b].tolist()) == list(range(w.V))
        row = np.zeros(w.V)
        row[ev["p_idx"][b]] = ev["p_val64"][b]
        np.testing.assert_allclose(row, dense["p_row64"][b], rtol=1e-13)


def _scatter(idx, val, V):
    out = np.zeros(idx.shape[:-1] + (V,), np.float32)
    np.put_along_axis(out, idx.astype(np.int64), val, axis=-1)
    return out


def test_k5_truncated_draw_equals_dense_draw_on_scattered_rows(oracle_mod):
    rng = np.random.default_rng(11)
    B, gamma, V, k = 400, 3, 50, 6
    p_idx = np.stack([rng.permutation(V)[:k] for _ in range(B)]).astype(np.int32)
    p_val = rng.random((B, k)).astype(np.float32)
    p_val /= p_val.sum(axis=1, keepdims=True)
    q_idx = np.stack([[rng.permutation(V)[:k] for _ in range(gamma)] for _ in range(B)]).astype(np.int32)
    # make the supports overlap: half of q's entries are copied from p's
    q_idx[:, :, : k // 2] = p_idx[:, None, : k // 2]
    for b in range(B):  # keep q's indices unique
        for i in range(gamma):
            seen = set(q_idx[b, i, : k // 2].tolist())
            for e in range(k // 2, k):
                while int(q_idx[b, i, e]) in seen:
                    q_idx[b, i, e] = (q_idx[b, i, e] + 1) % V
                seen.add(int(q_idx[b, i, e]))
    q_val = rng.random((B, gamma, k)).astype(np.float32)
    q_val /= q_val.sum(axis=2, keepdims=True)
    n = rng.integers(0, gamma + 1, size=B).astype(np.int32)
    n[:4] = [-1, gamma + 1, gamma, 0]
    # rows 4..7: q equals p on p's support, so the residual is empty and the draw falls back to p
    for b in range(4, 8):
        n[b] = 1
        q_idx[b, 1] = p_idx[b][::-1]
        q_val[b, 1] = p_val[b][::-1]
    # row 8: p without mass at all
    p_val[8] = 0
    u = rng.random(B).astype(np.float32)
    got = oracle_mod.device_resample_topk(p_idx, p_val, q_idx, q_val, n, u, gamma)
    want = oracle_mod.device_resample(_scatter(p_idx, p_val, V), _scatter(q_idx, q_val, V), n, u, gamma)
    np.testing.assert_array_equal(got["token"], want["token"])
    np.testing.assert_array_equal(got["flags"], want["flags"])
    np.testing.assert_allclose(got["Z"], want["Z"], rtol=1e-15, atol=0)
    assert got["flags"][0] == oracle_mod.RS_FLAG_INVALID and got["token"][0] == -1
    assert got["flags"][2] == oracle_mod.RS_FLAG_BONUS
    assert all(got["flags"][b] & oracle_mod.RS_FLAG_FALLBACK for b in range(4, 8))
    assert got["flags"][8] & oracle_mod.RS_FLAG_INVALID and got["token"][8] == -1
    # a sequence without a row (negative index) gets no token
    p_bad = p_idx.copy()
    p_bad[9, 2] = -1
    got = oracle_mod.device_resample_topk(p_bad, p_val, q_idx, q_val, n, u, gamma)
    assert got["token"][9] == -1 and got["flags"][9] == oracle_mod.RS_FLAG_INVALID


class _Truncated:
    """Presents the truncated oracle through the dense oracle's two calls, for _enumerate."""

    def __init__(self, O, k, q_rows):
        self.O, self.k = O, k
        q32 = np.array([[float(v) for v in r] for r in q_rows], np.float32)
        order = np.argsort(-q32, axis=1, kind="stable")[:, :k]
        self.q_idx = order.astype(np.int32)
        self.q_val = np.take_along_axis(q32, order, axis=1)

    def edge_verify(self, logits, tokens, q_tok, u, T, threads=1):
        ev = self.O.edge_verify_topk(logits, tokens, q_tok, u, T, self.k, threads=threads)
        ev["p_row"] = (ev["p_idx"], ev["p_val"])
        return ev

    def device_resample(self, p_row, draft_q, n, u_rs, gamma, threads=1):
        p_idx, p_val = p_row
        B = p_idx.shape[0]
        qi = np.broadcast_to(self.q_idx[None], (B,) + self.q_idx.shape).copy()
        qv = np.broadcast_to(self.q_val[None], (B,) + self.q_val.shape).copy()
        return self.O.device_resample_topk(p_idx, p_val, qi, qv, n, u_rs, gamma)


def _truncate(row, k):
    keep = sorted(range(len(row)), key=lambda v: (-row[v], v))[:k]
    Z = sum(row[v] for v in keep)
    return [row[v] / Z if v in keep else Fraction(0) for v in range(len(row))]


TRUNC_CASES = {
    # (raw P rows, raw Q rows, k); the ties in P row 1 and Q row 0 are cut toward the lower index
    "V4_g2_k2": (_F([[1, 3, 4, 2], [1, 3, 3, 3], [1, 1, 2, 6]], 10), _F([[4, 4, 1, 1], [1, 2, 3, 4]], 10), 2),
    "V5_g1_k3": (_F([[1, 5, 2, 4, 4], [6, 1, 5, 2, 2]], 16), _F([[3, 5, 5, 2, 1]], 16), 3),
}


@pytest.mark.parametrize("name", sorted(TRUNC_CASES))
def test_k6_emitted_law_is_the_truncated_target(oracle_mod, name):
    p_raw, q_raw, k = TRUNC_CASES[name]
    p_rows = [_truncate(r, k) for r in p_raw]
    q_rows = [_truncate(r, k) for r in q_raw]
    shim = _Truncated(oracle_mod, k, q_rows)
    # the edge sees the raw target rows (it truncates them itself); drafts come from truncated Q
    import test_oracle_pins as tp

    orig = tp._logits_from_probs
    try:
        tp._logits_from_probs = lambda rows, T=1.0: orig(p_raw, T)
        num, den, K, B = _enumerate(shim, p_rows, q_rows)
    finally:
        tp._logits_from_probs = orig
    gamma = len(q_rows)
    for j in range(gamma + 1):
        assert den[j] > 0
        for a in range(len(p_rows[0])):
            assert num[j][a] / den[j] == p_rows[j][a], (name, j, a, K, B)


def test_k7_invalid_arguments(oracle_mod):
    l = np.zeros((1, 1, 8), np.float32)
    none = (np.zeros((1, 0), np.int32), np.zeros((1, 0), np.float32), np.zeros((1, 0), np.float32))
    for k in (0, 9, 33):
        with pytest.raises(ValueError):
            oracle_mod.edge_verify_topk(np.zeros((1, 1, 40), np.float32) if k == 33 else l, *none, 1.0, k)
    # a row with a NaN or +inf has no distribution: flagged, nothing accepted, no support
    for bad in (np.nan, np.inf):
        l2 = np.zeros((1, 2, 8), np.float32)
        l2[0, 0, 3] = bad
        ev = oracle_mod.edge_verify_topk(l2, np.array([[1]], np.int32), np.array([[0.1]], np.float32),
                                         np.array([[0.0]], np.float32), 1.0, 4)
        assert ev["flags"][0] & oracle_mod.FLAG_NONFINITE
        assert ev["accept_len"][0] == 0 and (ev["p_idx"][0] == -1).all() and np.isnan(ev["p_val"][0]).all()
