"""Pins of the vocabulary-sharded oracle (oracle/shard_oracle.py) against facts that do not come from it.

H1  hand-worked rows: partial sums, combined log-sum-exp, emitted slices, masses and the owning
    shard of a draw, from fractions written out by hand.
H2  equality with the dense oracle (itself pinned by enumeration, closed forms and Table 1) for
    G in {1, 2, 3, 8}: ragged V / G, more shards than entries, a shard of -inf only, both dtypes.
H3  the degenerate inputs of the dense round (NaN, +inf, all -inf, bad token ids, q = 0, no
    residual mass, no mass at all) give the dense oracle's lengths, tokens and flags.
H4  exhaustive enumeration through the sharded functions: the emitted-token law is the target
    law exactly (Section 1: the split scheme "maintains inference quality").
H5  every shard reaches the same verdict, and exactly one of them returns the token.
"""
import numpy as np
import pytest

import dssd_inputs as di
from oracle import shard_oracle as S
from test_oracle_pins import CASES, _enumerate


def _dense(O, d, T):
    return O.verify_round(d, T, threads=4)


def _compare_with_dense(O, d, T, G):
    V = d["target_logits"].shape[2]
    ref = _dense(O, d, T)
    out = S.verify_round_sharded(d, T, S.shard_bounds(V, G))
    assert (out["accept_len"] == ref["accept_len"]).all()
    assert (out["flags"] == ref["flags"]).all()
    np.testing.assert_allclose(out["lse"], ref["lse"], rtol=1e-13, atol=1e-13, equal_nan=True)
    np.testing.assert_allclose(out["p_tok"], ref["p_tok"], rtol=1e-12, atol=0, equal_nan=True)
    np.testing.assert_allclose(out["margin_acc"], ref["margin_acc"], rtol=1e-9, atol=1e-15)
    # the float32 row: the two log-sum-exps differ by rounding only, so at most the last bit moves
    np.testing.assert_allclose(out["p_row"], ref["p_row"], rtol=1.2e-7, atol=0, equal_nan=True)
    same_row = np.array([np.array_equal(a, b, equal_nan=True) for a, b in zip(out["p_row"], ref["p_row"])])
    assert (out["rs_flags"] == ref["rs_flags"]).all()
    safe = same_row & (ref["margin_cdf"] > 1e-12)
    assert (out["token"][safe] == ref["token"][safe]).all()
    drawn = same_row & (ref["token"] >= 0)  # a sequence without a token has no mass to compare
    np.testing.assert_allclose(out["Z"][drawn], ref["Z"][drawn], rtol=1e-12, atol=1e-300)
    np.testing.assert_allclose(out["margin_cdf"][safe], ref["margin_cdf"][safe], rtol=1e-6, atol=1e-13)
    return out, ref, safe


def test_h1_hand_worked_rows():
    ln = np.log
    # one sequence, gamma = 1, V = 4, T = 1, two shards of two entries
    # row 0: p = (1, 3, 2, 0) / 6;  row 1: p = (1, 1, 1, 1) / 4
    logits = np.array([[[0.0, ln(3.0), ln(2.0), -np.inf], [0.0, 0.0, 0.0, 0.0]]], np.float32)
    tokens = np.array([[2]], np.int32)
    a = S.edge_partial(logits[:, :, 0:2], tokens, 0, 1.0)
    b = S.edge_partial(logits[:, :, 2:4], tokens, 2, 1.0)
    f = lambda x: float(np.float32(x))  # noqa: E731  (the logits are float32)
    np.testing.assert_allclose(a["m"], [[f(ln(3.0)), 0.0]], rtol=1e-15)
    np.testing.assert_allclose(a["S"], [[1.0 + np.exp(-f(ln(3.0))), 2.0]], rtol=1e-15)
    np.testing.assert_allclose(b["m"], [[f(ln(2.0)), 0.0]], rtol=1e-15)
    np.testing.assert_allclose(b["S"], [[1.0, 2.0]], rtol=1e-15)
    assert np.isnan(a["z_tok"][0, 0]) and b["z_tok"][0, 0] == f(ln(2.0))  # token 2 lives in the second shard
    # q(x) = 1/2 > p(x) = 1/3: accepted iff u < 2/3
    for u, n in ((0.6, 1), (0.7, 0)):
        ev = S.edge_combine([a, b], tokens, np.array([[0.5]], np.float32), np.array([[u]], np.float32), 4)
        np.testing.assert_allclose(ev["lse"], [[ln(6.0), ln(4.0)]], rtol=2e-7)
        np.testing.assert_allclose(ev["p_tok"], [[1.0 / 3.0]], rtol=2e-7)
        assert ev["accept_len"][0] == n and ev["flags"][0] == 0
        np.testing.assert_allclose(ev["margin_acc"], [abs(f(u) - 2.0 / 3.0)], rtol=1e-6)
    # rejected at position 0: row 0 goes down; slices (1/6, 3/6) and (2/6, 0)
    ev = S.edge_combine([a, b], tokens, np.array([[0.5]], np.float32), np.array([[0.7]], np.float32), 4)
    r0 = S.edge_emit_shard(logits[:, :, 0:2], ev["accept_len"], ev["lse"], 1.0)
    r1 = S.edge_emit_shard(logits[:, :, 2:4], ev["accept_len"], ev["lse"], 1.0)
    np.testing.assert_allclose(r0, [[1 / 6, 3 / 6]], rtol=3e-7)
    np.testing.assert_allclose(r1, [[2 / 6, 0.0]], rtol=3e-7)
    # device row q = (1/2, 1/6, 1/6, 1/6): residual = (0, 1/3, 1/6, 0), Z = 1/2
    p0, p1 = np.array([[1 / 6, 3 / 6]], np.float32), np.array([[2 / 6, 0.0]], np.float32)
    q0, q1 = np.array([[[1 / 2, 1 / 6]]], np.float32), np.array([[[1 / 6, 1 / 6]]], np.float32)
    m0 = S.resample_shard_mass(p0, q0, ev["accept_len"], 1)
    m1 = S.resample_shard_mass(p1, q1, ev["accept_len"], 1)
    np.testing.assert_allclose(m0, [[1 / 3, 4 / 6]], rtol=3e-7)
    np.testing.assert_allclose(m1, [[1 / 6, 2 / 6]], rtol=3e-7)
    masses = np.stack([m0, m1])
    # u' Z below 1/3 falls in the first shard (token 1), above it in the second (token 2)
    for u, tok, own in ((0.5, 1, 0), (0.7, 2, 1), (0.0, 1, 0), (0.999, 2, 1)):
        d0 = S.resample_shard_draw(masses, 0, 0, p0, q0, ev["accept_len"], np.array([u], np.float32), 1)
        d1 = S.resample_shard_draw(masses, 1, 2, p1, q1, ev["accept_len"], np.array([u], np.float32), 1)
        assert d0["owner"][0] == own and d1["owner"][0] == own
        assert (d0["token"][0], d1["token"][0]) == ((tok, -1) if own == 0 else (-1, tok))
        assert d0["flags"][0] == 0 and d1["flags"][0] == 0
        np.testing.assert_allclose(d0["Z"], [0.5], rtol=3e-7)
    assert S.shard_bounds(10, 3) == [(0, 4), (4, 7), (7, 10)] and S.shard_bounds(2, 3) == [(0, 1), (1, 2), (2, 2)]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("G", [1, 2, 3, 8])
def test_h2_equals_the_dense_oracle(oracle_mod, dtype, G):
    seen = set()
    for V, gamma, Bn, seed in ((1000, 3, 40, 1), (37, 2, 60, 2), (5, 4, 50, 3), (4099, 0, 12, 4), (2048, 1, 30, 5)):
        w = di.custom(B=Bn, gamma=gamma, V=V, dtype=dtype, temperature=0.8, sigma_d=0.9, zipf=V > 8, seed=seed + 10 * G)
        d = di.generate(w, threads=4)
        out, ref, safe = _compare_with_dense(oracle_mod, d, w.temperature, G)
        assert safe.mean() > 0.9
        seen.update(out["owner"].tolist())
    if G <= 3:
        assert seen >= set(range(G))  # every shard got to own some draw


def test_h2_a_shard_of_minus_infinity_only(oracle_mod):
    w = di.custom(B=30, gamma=3, V=12, dtype="f32", temperature=1.0, sigma_d=0.7, zipf=False, seed=77)
    d = di.generate(w)
    d["target_logits"][:, :, 4:8] = -np.inf  # the middle shard of three has no mass in any row
    out, ref, safe = _compare_with_dense(oracle_mod, d, 1.0, 3)
    assert not (out["owner"] == 1).any() and safe.all()
    assert (out["masses"][1] == 0.0).all()
    assert (out["parts"][1]["m"] == -np.inf).all() and (out["parts"][1]["S"] == 0.0).all()


def test_h3_degenerate_inputs(oracle_mod):
    V, gamma, Bn = 60, 3, 12
    w = di.custom(B=Bn, gamma=gamma, V=V, dtype="f32", seed=9)
    d = di.generate(w)
    tl = d["target_logits"]
    tl[0, 1, 17] = np.nan
    tl[1, 0, 5] = np.inf
    tl[2, 2, :] = -np.inf
    tl[3, 1, ::2] = -np.inf
    d["draft_tokens"][4, 0] = -1
    d["draft_tokens"][5, 2] = V
    d["draft_q_tok"][6, 0] = 0.0
    d["uniforms"][7, :] = 0.0
    # sequence 8: rejected at once, and the device's row equals the target's: no residual mass
    d["uniforms"][8, 0] = 0.99999
    d["draft_q_tok"][8, 0] = 1.0
    ref0 = oracle_mod.edge_verify(tl, d["draft_tokens"], d["draft_q_tok"], d["uniforms"], 1.0)
    d["draft_q"][8, 0] = ref0["p_row"][8]
    # sequence 9: the device's row dominates the target's everywhere
    d["uniforms"][9, 0] = 0.99999
    d["draft_q_tok"][9, 0] = 1.0
    d["draft_q"][9, 0] = 1.0
    for G in (1, 2, 4, 7):
        out, ref, _ = _compare_with_dense(oracle_mod, d, 1.0, G)
        assert (out["token"] == ref["token"]).all()
        assert ref["rs_flags"][8] & S.RS_FLAG_FALLBACK and ref["rs_flags"][9] & S.RS_FLAG_FALLBACK
        assert ref["rs_flags"][0] & S.RS_FLAG_INVALID or ref["accept_len"][0] != 1
    # accepted lengths outside [0, gamma] are refused sequence by sequence
    p = np.full((2, 4), 0.25, np.float32)
    m = np.stack([S.resample_shard_mass(p[:, :2], None, np.array([0, 5]), 0),
                  S.resample_shard_mass(p[:, 2:], None, np.array([0, 5]), 0)])
    dr = S.resample_shard_draw(m, 0, 0, p[:, :2], None, np.array([0, 5]), np.array([0.1, 0.1], np.float32), 0)
    assert dr["token"].tolist() == [0, -1] and dr["flags"].tolist() == [S.RS_FLAG_BONUS, S.RS_FLAG_INVALID]


class _Sharded:
    """The sharded functions behind the two calls that the enumeration makes."""

    def __init__(self, G):
        self.G = G

    def edge_verify(self, logits, tokens, q_tok, u, T, threads=1):
        V = logits.shape[2]
        self.bounds = S.shard_bounds(V, self.G)
        parts = [S.edge_partial(logits[:, :, a:b], tokens, a, T) for a, b in self.bounds]
        ev = S.edge_combine(parts, tokens, q_tok, u, V)
        rows = [S.edge_emit_shard(logits[:, :, a:b], ev["accept_len"], ev["lse"], T) for a, b in self.bounds]
        return {"accept_len": ev["accept_len"], "p_row": np.concatenate(rows, axis=1)}

    def device_resample(self, p_row, draft_q, n, u_rs, gamma, threads=1):
        ps = [p_row[:, a:b] for a, b in self.bounds]
        qs = [draft_q[:, :, a:b] if gamma else None for a, b in self.bounds]
        masses = np.stack([S.resample_shard_mass(ps[g], qs[g], n, gamma) for g in range(self.G)])
        toks = np.stack([S.resample_shard_draw(masses, g, self.bounds[g][0], ps[g], qs[g], n, u_rs, gamma)["token"]
                         for g in range(self.G)])
        assert ((toks >= 0).sum(axis=0) == 1).all()  # exactly one shard answers
        return {"token": toks.max(axis=0)}


@pytest.mark.parametrize("name,G", [("V8_g1", 3), ("V4_g1_qzero", 2), ("V8_g1", 8)])
def test_h4_emitted_law_equals_target(name, G):
    p_rows, q_rows = CASES[name]
    num, den, K, B = _enumerate(_Sharded(G), p_rows, q_rows)
    for j in range(len(q_rows) + 1):
        assert den[j] > 0
        for a in range(len(p_rows[0])):
            assert num[j][a] / den[j] == p_rows[j][a], (name, G, j, a)


def test_h5_every_shard_reaches_the_same_verdict(oracle_mod):
    w = di.custom(B=80, gamma=2, V=300, dtype="f32", temperature=1.1, sigma_d=1.2, seed=404)
    d = di.generate(w)
    out = S.verify_round_sharded(d, w.temperature, S.shard_bounds(w.V, 4))
    assert (out["shard_flags"] == out["shard_flags"][0]).all()
    assert ((out["shard_tokens"] >= 0).sum(axis=0) == 1).all()
    own = out["shard_tokens"].argmax(axis=0)
    assert (own == out["owner"]).all()
    lo = np.array([b[0] for b in S.shard_bounds(w.V, 4)])[own]
    hi = np.array([b[1] for b in S.shard_bounds(w.V, 4)])[own]
    assert ((out["token"] >= lo) & (out["token"] < hi)).all()
