"""Pins of the oracle's bonus-at-the-edge round (Algorithm 2 as printed: x_{gamma+1} ~ P_{gamma+1}
drawn by the edge) against things it does not share code with:
  E1  the C implementation of Algorithm 1, which draws its bonus token from the float64 row too;
  E2  gamma = 0, where the round is softmax + cumsum + searchsorted (torch, float64);
  E3  the split round, wherever the float32 rounding of the row cannot move the draw;
  E4  closed forms of the draw on hand-made rows (zero-mass entries, u at the steps, no mass);
  E5  the law of the bonus token on a rational row, by exhaustive enumeration of u on a grid.
A planted mistake (>= in place of >, the clamp to the last entry instead of the last entry with
mass) fails E4."""
import numpy as np
import torch

import dssd_inputs as di


def test_e1_bonus_token_equals_algorithm_1(oracle_mod):
    O = oracle_mod
    seen = 0
    for seed, sigma in ((1, 0.2), (2, 0.4), (3, 0.1)):
        w = di.custom(B=48, gamma=3, V=777, dtype="bf16", temperature=0.8, sigma_d=sigma, seed=seed)
        d = di.generate(w)
        a = O.verify_round_bonus_at_edge(d, w.temperature)
        f = O.dsd_verify(d, w.temperature)
        assert (a["accept_len"] == f["accept_len"]).all()
        full = a["accept_len"] == w.gamma
        seen += int(full.sum())
        assert (a["bonus_token"][full] == f["token"][full]).all()
        assert (a["bonus_flags"][full] == f["rs_flags"][full]).all()
        assert (a["bonus_token"][~full] == -1).all() and (a["bonus_flags"][~full] == 0).all()
        np.testing.assert_allclose(a["margin_cdf"][full], f["margin_cdf"][full], rtol=1e-9, atol=1e-15)
    assert seen >= 20


def test_e2_gamma_zero_is_softmax_cumsum_searchsorted(oracle_mod):
    O = oracle_mod
    w = di.custom(B=40, gamma=0, V=1500, dtype="f32", temperature=0.7, seed=9)
    d = di.generate(w)
    a = O.verify_round_bonus_at_edge(d, w.temperature)
    z = torch.from_numpy(d["target_logits"][:, 0, :]).double() / float(np.float32(w.temperature))
    C = torch.cumsum(torch.softmax(z, dim=-1), dim=-1)
    t = torch.from_numpy(d["uniforms_rs"]).double() * C[:, -1]
    tok = torch.searchsorted(C, t.unsqueeze(-1), right=True).squeeze(-1).numpy()
    clear = a["margin_cdf"] > 1e-12
    assert clear.sum() >= 38 and (a["bonus_token"][clear] == tok[clear]).all()
    assert (a["accept_len"] == 0).all() and (a["token"] == a["bonus_token"]).all()


def test_e3_agrees_with_the_split_round_away_from_cdf_steps(oracle_mod):
    O = oracle_mod
    w = di.custom(B=64, gamma=2, V=3001, dtype="f32", temperature=1.0, sigma_d=0.3, seed=4)
    d = di.generate(w)
    a = O.verify_round_bonus_at_edge(d, w.temperature)
    s = O.verify_round(d, w.temperature)
    assert (a["accept_len"] == s["accept_len"]).all()
    rej = a["accept_len"] < w.gamma
    assert (a["token"][rej] == s["token"][rej]).all() and (a["rs_flags"][rej] == s["rs_flags"][rej]).all()
    # the float32 row moves every CDF step by at most 2^-24 of the row's sum
    clear = ~rej & (s["margin_cdf"] > 1e-6)
    assert clear.sum() >= 10 and (a["token"][clear] == s["token"][clear]).all()


def test_e4_closed_forms_of_the_draw(oracle_mod):
    draw = oracle_mod.bonus_draw
    p = np.array([0.0, 0.25, 0.0, 0.5, 0.25, 0.0])
    assert draw(p, 0.0)[0] == 1                 # strict >: zero-mass entry 0 is never returned
    assert draw(p, 0.2499)[0] == 1
    assert draw(p, 0.25)[0] == 3                # u * Z on a step: the step's entry is passed
    assert draw(p, 0.75)[0] == 4
    assert draw(p, 1.0 - 2.0 ** -24)[0] == 4
    assert draw(p, 1.0)[0] == 4                 # beyond every step: last entry with mass, not the last entry
    assert draw(2.0 * p, 0.5)[0] == 3           # the row's sum need not be 1
    tok, fl, _ = draw(np.zeros(5), 0.3)
    assert tok == -1 and fl == (oracle_mod.RS_FLAG_BONUS | oracle_mod.RS_FLAG_INVALID)
    tok, fl, _ = draw(np.array([0.5, np.nan, 0.5]), 0.3)
    assert tok == -1 and fl & oracle_mod.RS_FLAG_INVALID
    tok, fl, margin = draw(p, 0.5)
    assert tok == 3 and fl == oracle_mod.RS_FLAG_BONUS and abs(margin - 0.25) < 1e-15


def test_e5_law_of_the_bonus_token(oracle_mod):
    """u on the midpoint grid (k + 1/2) / K with K a multiple of the row's denominator: the number of
    grid points mapped to token v is exactly K * p_v."""
    p = np.array([3, 0, 1, 6, 2, 0, 4, 0]) / 16.0
    K = 64
    counts = np.zeros(p.size, int)
    for k in range(K):
        counts[oracle_mod.bonus_draw(p, (k + 0.5) / K)[0]] += 1
    assert (counts == (K * p).astype(int)).all()
