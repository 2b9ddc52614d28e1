"""Parity of the vocabulary-sharded round with its oracle, through the C ABI.

One GPU plays every shard in turn: shard g's calls get views of columns [v_g, v_{g+1}) of the same
arrays (the row stride arguments exist for exactly that), the two exchanges are torch.stack.  What
is compared: every shard's partial sums, the combined lengths / probabilities / flags, every
emitted slice, every shard's masses, and the tokens (exactly one shard answers per sequence).
"""
import numpy as np
import pytest
import torch

import dssd_inputs as di
from gpu_util import ATOL, NEAR, RTOL, prob_close, to_device
from oracle import shard_oracle as S

pytestmark = pytest.mark.gpu

LN2 = float(np.log(2.0))


@pytest.fixture(scope="module")
def B():
    from paper_2507_12000_b200 import binding

    assert torch.cuda.is_available()
    return binding


def run_sharded(B, g, T, bounds, p_row_in=None, n_in=None, logits_view=None):
    """The seven steps on one GPU.  With p_row_in / n_in the device half runs on those instead of the
    edge half's outputs (the device half in isolation, on the oracle's float32 rows)."""
    tl = g["target_logits"] if logits_view is None else logits_view(g["target_logits"])
    Bn, g1, V = tl.shape
    gamma = g1 - 1
    parts = [B.dssd_edge_partial(tl[:, :, a:b], g["draft_tokens"], a, T) for a, b in bounds]
    ref = torch.stack([p["part_ref"] for p in parts])
    sm = torch.stack([p["part_sum"] for p in parts])
    tz = torch.stack([p["tok_logit"] for p in parts])
    ev = B.dssd_edge_combine(ref, sm, tz, g["draft_tokens"], g["draft_q_tok"], g["uniforms"], T, V)
    p_row = torch.full((Bn, V), -7.0, dtype=torch.float32, device="cuda")
    for a, b in bounds:
        B.dssd_edge_emit_shard(tl[:, :, a:b], ev["accept_len"], ev["row_scale"], T, out=p_row[:, a:b])
    p_use = p_row if p_row_in is None else p_row_in
    n_use = ev["accept_len"] if n_in is None else n_in
    dq = g.get("draft_q")
    work, masses = [], []
    for a, b in bounds:
        m, ws = B.dssd_resample_shard_mass(p_use[:, a:b], dq[:, :, a:b] if gamma else None, n_use, gamma)
        masses.append(m)
        work.append(ws)
    masses = torch.stack(masses)
    draws = [B.dssd_resample_shard_draw(masses, i, a, p_use[:, a:b], dq[:, :, a:b] if gamma else None, n_use,
                                        g["uniforms_rs"], gamma, work[i]) for i, (a, b) in enumerate(bounds)]
    torch.cuda.synchronize()
    return {"parts": parts, "ev": ev, "p_row": p_row, "masses": masses,
            "tokens": torch.stack([d["token"] for d in draws]).cpu().numpy(),
            "flags": torch.stack([d["flags"] for d in draws]).cpu().numpy().astype(np.uint32)}


def compare_sharded(B, d, T, G, logits_view=None):
    V = d["target_logits"].shape[2]
    gamma = d["target_logits"].shape[1] - 1
    bounds = [b for b in S.shard_bounds(V, G) if b[1] > b[0]]
    ref = S.verify_round_sharded(d, T, bounds)
    g = to_device(d)
    out = run_sharded(B, g, T, bounds, logits_view=logits_view)
    # 1. every shard's partial sums, as a log-sum-exp over the slice, and the drafted tokens' logits
    for i, (a, b) in enumerate(bounds):
        pr = out["parts"][i]["part_ref"].cpu().numpy().astype(np.float64)
        ps = out["parts"][i]["part_sum"].cpu().numpy()
        m, s = ref["parts"][i]["m"], ref["parts"][i]["S"]
        assert (pr == np.rint(pr)).all()
        fin = np.isfinite(m)
        with np.errstate(divide="ignore", invalid="ignore"):
            lse_gpu = (pr + np.log2(ps)) * LN2
            lse_ref = m + np.log(s)
        assert (np.abs(lse_gpu - lse_ref)[fin] <= 2e-6 * np.maximum(1.0, np.abs(lse_ref[fin]))).all()
        assert (ps[m == -np.inf] == 0.0).all() and (pr[m == -np.inf] == 0.0).all()
        assert np.isnan(ps[np.isnan(m) | (m == np.inf)]).all()
        if gamma:
            tz = out["parts"][i]["tok_logit"].cpu().numpy().astype(np.float64)
            zt = ref["parts"][i]["z_tok"] * float(np.float32(T))
            assert (np.isnan(tz) == np.isnan(zt)).all() and (np.isinf(tz) == np.isinf(zt)).all()
            own = np.isfinite(zt)
            assert (np.abs(tz[own] - zt[own]) <= 1e-12 * np.maximum(1.0, np.abs(zt[own]))).all()
    # 2. the combined verdict
    ev = out["ev"]
    n_gpu = ev["accept_len"].cpu().numpy()
    assert (ev["flags"].cpu().numpy().astype(np.uint32) == ref["flags"]).all()
    near = ref["margin_acc"] < NEAR
    bad = (n_gpu != ref["accept_len"]) & ~near
    assert not bad.any(), (np.nonzero(bad)[0][:8], n_gpu[bad][:8], ref["accept_len"][bad][:8])
    clean = ref["flags"] == 0
    lse = ev["lse"].cpu().numpy().astype(np.float64)
    assert (np.abs(lse - ref["lse"])[clean] <= 2e-6 * np.maximum(1.0, np.abs(ref["lse"][clean]))).all()
    if gamma:
        assert prob_close(ev["p_tok"].cpu().numpy(), ref["p_tok"]).all()
    # 3. the emitted slices, assembled
    same = n_gpu == ref["accept_len"]
    p_gpu = out["p_row"].cpu().numpy()
    okrow = prob_close(p_gpu[same], ref["p_row"][same])
    assert okrow.all(), np.argwhere(~okrow)[:8]
    # 4. end to end: the device half on the CUDA path's own row
    tok = out["tokens"]
    assert ((tok >= 0).sum(axis=0) <= 1).all()
    assert (out["flags"] == out["flags"][0]).all()
    slack = np.maximum(NEAR, 2 * RTOL / np.maximum(ref["Z"], 1e-30))
    # (a residual without mass on the oracle's side means p == q to the last bit: the CUDA path's own
    # row differs from q by its rounding, so there the draw is compared in isolation only, below)
    excused = (ref["margin_cdf"] < slack) | ((ref["rs_flags"] & S.RS_FLAG_FALLBACK) != 0)
    bad = (tok.max(axis=0) != ref["token"]) & same & ~excused
    assert not bad.any(), (np.nonzero(bad)[0][:8], tok.max(axis=0)[bad][:8], ref["token"][bad][:8])
    # 5. the device half in isolation: the oracle's float32 row and lengths on both sides
    iso = run_sharded(B, g, T, bounds, p_row_in=torch.from_numpy(ref["p_row"]).cuda(),
                      n_in=torch.from_numpy(ref["accept_len"]).cuda(), logits_view=logits_view)
    m_gpu = iso["masses"].cpu().numpy()
    np.testing.assert_allclose(m_gpu, ref["masses"], rtol=1e-12, atol=1e-300, equal_nan=True)
    tok = iso["tokens"]
    assert (iso["flags"] == ref["shard_flags"]).all()
    near_cdf = ref["margin_cdf"] < NEAR
    bad = ((tok != ref["shard_tokens"]).any(axis=0)) & ~near_cdf
    assert not bad.any(), (np.nonzero(bad)[0][:8], tok[:, bad][:, :8], ref["shard_tokens"][:, bad][:, :8])
    return {"near_acc": int(near.sum()), "near_cdf": int(near_cdf.sum()), "excused_e2e": int((excused & same).sum())}


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("G", [1, 2, 3, 8])
def test_small_vocabularies_ragged_shards(B, dtype, G):
    seed = 900 + G
    for V in (1, 3, 7, 33, 1000, 1025, 16389):
        for gamma in (0, 3):
            for Bn in (2, 150):
                seed += 1
                w = di.custom(B=Bn, gamma=gamma, V=V, dtype=dtype, temperature=0.9, sigma_d=1.0, zipf=V > 8, seed=seed)
                compare_sharded(B, di.generate(w, threads=4), w.temperature, G)


@pytest.mark.parametrize("dtype,V,gamma,Bn,G", [
    ("f32", 50272, 2, 6, 4), ("bf16", 40003, 3, 5, 3), ("bf16", 128256, 8, 4, 8), ("f32", 20001, 16, 3, 2),
    ("bf16", 151936, 4, 9, 8), ("f32", 16385, 1, 40, 5), ("bf16", 70000, 33, 2, 2),
])
def test_several_chunks_and_ragged_tails(B, dtype, V, gamma, Bn, G):
    w = di.custom(B=Bn, gamma=gamma, V=V, dtype=dtype, temperature=0.8, sigma_d=0.8, seed=V + gamma)
    compare_sharded(B, di.generate(w, threads=4), w.temperature, G)


def test_strided_and_unaligned_rows(B):
    for dtype, V, off, Bn, G in (("f32", 1000, 1, 3, 3), ("bf16", 4097, 3, 151, 2), ("bf16", 20001, 1, 3, 4)):
        w = di.custom(B=Bn, gamma=2, V=V, dtype=dtype, seed=V)
        d = di.generate(w)
        stride = V + 5

        def view(t, stride=stride, off=off, Bn=Bn, V=V):
            buf = torch.zeros(Bn * 3 * stride + 16, dtype=t.dtype, device="cuda")
            v = buf[off:off + Bn * 3 * stride].view(Bn, 3, stride)[:, :, :V]
            v.copy_(t)
            assert v.data_ptr() % 16 != 0
            return v

        compare_sharded(B, d, w.temperature, G, logits_view=view)


def test_anomalies_are_flagged_not_faulted(B, oracle_mod):
    V, gamma, Bn = 3000, 3, 12
    w = di.custom(B=Bn, gamma=gamma, V=V, dtype="f32", seed=5)
    d = di.generate(w)
    tl = d["target_logits"]
    tl[0, 1, 17] = np.nan
    tl[1, 0, 5] = np.inf
    tl[2, 2, :] = -np.inf
    tl[3, 1, ::2] = -np.inf
    tl[10, :, 1000:2000] = -np.inf  # the middle shard of three holds no mass for this sequence
    d["draft_tokens"][4, 0] = -1
    d["draft_tokens"][5, 2] = V
    d["draft_q_tok"][6, 0] = 0.0
    d["uniforms"][7, :] = 0.0
    # sequence 8: rejected at once, and the device's row equals the target's (no residual mass);
    # sequence 9: the device's row dominates the target's everywhere
    for b in (8, 9):
        d["uniforms"][b, 0] = 0.99999
        d["draft_q_tok"][b, 0] = 1.0
    ref0 = oracle_mod.edge_verify(tl, d["draft_tokens"], d["draft_q_tok"], d["uniforms"], 1.0)
    d["draft_q"][8, 0] = ref0["p_row"][8]
    d["draft_q"][9, 0] = 1.0
    for G in (1, 3, 4):
        compare_sharded(B, d, 1.0, G)
    bounds = S.shard_bounds(V, 3)
    ref = S.verify_round_sharded(d, 1.0, bounds)
    assert ref["rs_flags"][8] & S.RS_FLAG_FALLBACK and ref["rs_flags"][9] & S.RS_FLAG_FALLBACK
    out = run_sharded(B, to_device(d), 1.0, bounds)
    tok = out["tokens"].max(axis=0)
    # (sequence 8's residual has no mass only while the row equals q to the last bit: the CUDA path's
    # own row does not, so that sequence is compared in isolation, inside compare_sharded)
    clean = (ref["flags"] == 0) & (ref["margin_cdf"] > 1e-4) & ((ref["rs_flags"] & S.RS_FLAG_FALLBACK) == 0)
    assert (tok[clean] == ref["token"][clean]).all()
    assert (np.delete(out["flags"][0], 8) == np.delete(ref["rs_flags"], 8)).all()
    assert (out["tokens"][1, 10] == -1)


def test_one_shard_is_the_dense_round(B):
    """G = 1: the sharded calls give what dssd_edge_verify and dssd_device_resample give."""
    w = di.custom(B=300, gamma=4, V=30011, dtype="bf16", temperature=0.7, sigma_d=0.5, seed=12)
    d = di.generate(w, threads=4)
    g = to_device(d)
    out = run_sharded(B, g, w.temperature, [(0, w.V)])
    ev = B.dssd_edge_verify(g["target_logits"], g["draft_tokens"], g["draft_q_tok"], g["uniforms"], w.temperature)
    rs = B.dssd_device_resample(ev["p_row"], g["draft_q"], ev["accept_len"], g["uniforms_rs"], w.gamma)
    torch.cuda.synchronize()
    assert torch.equal(out["ev"]["accept_len"], ev["accept_len"])
    assert torch.equal(out["p_row"], ev["p_row"])  # same sums (streaming kernel), same emission arithmetic
    assert (out["tokens"][0] == rs["token"].cpu().numpy()).all()
    assert (out["flags"][0] == rs["flags"].cpu().numpy().astype(np.uint32)).all()


@pytest.mark.parametrize("name,G", [("c2", 4), ("c3", 8), ("c4", 8)])
def test_named_configs(B, name, G):
    w = di.get_workload(name)
    rep = compare_sharded(B, di.generate(w, threads=8), w.temperature, G)
    print(f"sharded parity on {name}, G={G}: {rep}")


def test_host_side_refusals(B):
    t = torch.zeros(4, 2, 64, dtype=torch.float32, device="cuda")
    tok = torch.zeros(4, 1, dtype=torch.int32, device="cuda")
    ws = torch.empty(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.DssdError) as e:
        B.dssd_edge_partial(t, tok, 0, 1.0, workspace=ws)  # workspace too small
    assert e.value.status == B.DSSD_ERR_WORKSPACE
    with pytest.raises(B.DssdError) as e:
        B.dssd_edge_partial(t, tok, -1, 1.0)
    assert e.value.status == B.DSSD_ERR_INVALID_ARG
    with pytest.raises(B.DssdError) as e:
        B.dssd_edge_partial(t, tok, 0, 0.0)
    assert e.value.status == B.DSSD_ERR_INVALID_ARG
    m = torch.zeros(2, 4, 2, dtype=torch.float64, device="cuda")
    p = torch.zeros(4, 64, dtype=torch.float32, device="cuda")
    q = torch.zeros(4, 1, 64, dtype=torch.float32, device="cuda")
    n = torch.zeros(4, dtype=torch.int32, device="cuda")
    u = torch.zeros(4, dtype=torch.float32, device="cuda")
    _, ws = B.dssd_resample_shard_mass(p, q, n, 1)
    with pytest.raises(B.DssdError) as e:
        B.dssd_resample_shard_draw(m, 2, 0, p, q, n, u, 1, ws)  # shard index outside [0, G)
    assert e.value.status == B.DSSD_ERR_INVALID_ARG
    torch.cuda.synchronize()


def test_the_rank_plumbing_on_a_group_of_one(B, oracle_mod):
    """paper_2507_12000_b200/sharded.py on a process group with a single rank (all that one GPU allows):
    the five calls, the two all-gathers and the final max run through NCCL on CUDA tensors, and the round
    equals the dense oracle's."""
    import os
    import socket

    import torch.distributed as dist

    from paper_2507_12000_b200.sharded import verify_round_vocab_sharded

    w = di.custom(B=40, gamma=3, V=20011, dtype="bf16", temperature=0.8, sigma_d=0.7, seed=77)
    d = di.generate(w, threads=4)
    ref = oracle_mod.verify_round(d, w.temperature, threads=4)
    g = to_device(d)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    try:
        out = verify_round_vocab_sharded(g["target_logits"], g["draft_tokens"], g["draft_q_tok"], g["uniforms"],
                                         g["draft_q"], g["uniforms_rs"], w.temperature, 0, w.V)
        torch.cuda.synchronize()
    finally:
        dist.destroy_process_group()
    n = out["accept_len"].cpu().numpy()
    assert ((n == ref["accept_len"]) | (ref["margin_acc"] < NEAR)).all()
    same = n == ref["accept_len"]
    slack = np.maximum(NEAR, 2 * RTOL / np.maximum(ref["Z"], 1e-30))
    ok = (out["token"].cpu().numpy() == ref["token"]) | ~same | (ref["margin_cdf"] < slack)
    assert ok.all()
    assert prob_close(out["p_row_shard"].cpu().numpy()[same], ref["p_row"][same]).all()
