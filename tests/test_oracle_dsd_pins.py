"""Pins of the Algorithm 1 (DSD, fused verify) oracle against facts that do not come from it.

D1  exhaustive enumeration: the emitted-token law equals the target law exactly.
D2  it agrees with the split round (Algorithm 2) wherever the float32 rounding of the downlink
    row cannot matter: the two algorithms compute the same thing (Section 3: "maintains
    inference quality").
D3  gamma = 0 is softmax + cumsum + searchsorted.
D4  a draft row that dominates the target row everywhere leaves no residual: fallback to P_n.
"""
import numpy as np
import pytest

import dssd_inputs as di
from test_oracle_pins import CASES, _enumerate


class _Fused:
    """Presents dsd_verify through the two calls _enumerate makes: the first call only records
    its arguments, the second runs the fused oracle and fills in the accepted lengths."""

    def __init__(self, O):
        self.O = O

    def edge_verify(self, logits, tokens, q_tok, u, T, threads=1):
        self.args = (logits, tokens, u, T, threads)
        self.ev = {"accept_len": np.zeros(logits.shape[0], np.int32), "p_row": None}
        return self.ev

    def device_resample(self, p_row, draft_q, n, u_rs, gamma, threads=1):
        logits, tokens, u, T, th = self.args
        r = self.O.dsd_verify({"target_logits": logits, "draft_q": draft_q, "draft_tokens": tokens, "uniforms": u,
                               "uniforms_rs": u_rs}, T, threads=th)
        self.ev["accept_len"][:] = r["accept_len"]
        return {"token": r["token"]}


@pytest.mark.parametrize("name", ["V4_g2", "V3_g3", "V8_g1", "V4_g1_qzero"])
def test_d1_emitted_law_equals_target(oracle_mod, name):
    p_rows, q_rows = CASES[name]
    num, den, K, B = _enumerate(_Fused(oracle_mod), p_rows, q_rows)
    for j in range(len(q_rows) + 1):
        assert den[j] > 0
        for a in range(len(p_rows[0])):
            assert num[j][a] / den[j] == p_rows[j][a], (name, j, a, K, B)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_d2_agrees_with_the_split_round(oracle_mod, dtype):
    w = di.custom(B=200, gamma=4, V=900, dtype=dtype, temperature=0.8, sigma_d=0.6, seed=31)
    d = di.generate(w, threads=4)
    split = oracle_mod.verify_round(d, w.temperature, threads=4)
    fused = oracle_mod.dsd_verify(d, w.temperature, threads=4)
    assert (fused["accept_len"] == split["accept_len"]).all()
    assert (fused["flags"] == split["flags"]).all() and (fused["rs_flags"] == split["rs_flags"]).all()
    np.testing.assert_allclose(fused["margin_acc"], split["margin_acc"], rtol=1e-12)
    # the mass the token is drawn from: the split round forms it from the float32 row (each entry within
    # 2^-24 relative of the float64 one, so the sums differ by at most 2^-24 * sum p = 6e-8)
    np.testing.assert_allclose(fused["Z"], split["Z"], rtol=0, atol=1e-7)
    safe = split["margin_cdf"] > 1e-5
    assert safe.mean() > 0.95 and (fused["token"][safe] == split["token"][safe]).all()
    assert len(set(fused["accept_len"].tolist())) >= 3


def test_d3_gamma_zero_is_a_plain_draw(oracle_mod):
    w = di.custom(B=64, gamma=0, V=333, dtype="f32", temperature=1.3, seed=8)
    d = di.generate(w)
    r = oracle_mod.dsd_verify(d, w.temperature)
    z = d["target_logits"][:, 0, :].astype(np.float64) / np.float64(np.float32(w.temperature))
    p = np.exp(z - z.max(axis=1, keepdims=True))
    p /= p.sum(axis=1, keepdims=True)
    cdf = np.cumsum(p, axis=1)
    want = [int(np.searchsorted(cdf[b], np.float64(d["uniforms_rs"][b]) * cdf[b, -1], side="right")) for b in range(w.B)]
    clear = r["margin_cdf"] > 1e-9
    assert clear.all() and (r["token"] == np.array(want)).all()
    assert (r["accept_len"] == 0).all() and (r["rs_flags"] == oracle_mod.RS_FLAG_BONUS).all()


def test_d4_no_residual_falls_back(oracle_mod):
    w = di.custom(B=8, gamma=2, V=50, dtype="f32", temperature=1.0, seed=4)
    d = di.generate(w)
    z = d["target_logits"].astype(np.float64)
    p = np.exp(z - z.max(axis=2, keepdims=True))
    p /= p.sum(axis=2, keepdims=True)
    d["draft_q"] = (p[:, :2, :] * 1.001).astype(np.float32)   # q >= p everywhere: max(0, p - q) = 0
    d["uniforms"][:] = 0.9995                                  # p/q = 1/1.001 < u: position 0 is rejected
    r = oracle_mod.dsd_verify(d, 1.0)
    assert (r["accept_len"] == 0).all()
    assert (r["rs_flags"] == oracle_mod.RS_FLAG_FALLBACK).all()
    cdf = np.cumsum(p[:, 0, :], axis=1)
    want = [int(np.searchsorted(cdf[b], np.float64(d["uniforms_rs"][b]) * cdf[b, -1], side="right")) for b in range(w.B)]
    assert (r["token"] == np.array(want)).all()
    # a token id outside the vocabulary is flagged and rejected there
    d["draft_tokens"][3, 0] = w.V
    r = oracle_mod.dsd_verify(d, 1.0)
    assert r["flags"][3] == oracle_mod.FLAG_BAD_TOKEN and r["accept_len"][3] == 0
