"""Parity of the bonus-at-the-edge round (dssd_edge_verify_bonus + dssd_device_resample_rejected)
with the oracle's statement of Algorithm 2 as printed, and with the CUDA path's own split round.

Tolerances: accepted lengths exactly, outside the oracle's 1e-6 acceptance margin.  The bonus token
is drawn from float32 probabilities (relative error about 1e-6, gpu_util.RTOL bounds it) summed in
float64, the oracle's from the float64 row: the two may differ only where u' * Z lies within
2 * RTOL of a CDF step (relative to Z).  The split CUDA round must give the same decisions, flags
and - away from CDF steps - tokens."""
import numpy as np
import pytest
import torch

import dssd_inputs as di
from gpu_util import NEAR, RTOL, prob_close, to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2507_12000_b200 import binding

    assert torch.cuda.is_available()
    return binding


def compare_bonus(B, O, d, T, logits_view=None, threads=4):
    gamma = d["target_logits"].shape[1] - 1
    ref = O.verify_round_bonus_at_edge(d, T, threads=threads)
    g = to_device(d)
    tl = g["target_logits"] if logits_view is None else logits_view(g["target_logits"])
    Bn, V = ref["p_row"].shape
    canary = 7.25
    out = {
        "accept_len": torch.empty(Bn, dtype=torch.int32, device="cuda"),
        "p_row": torch.full((Bn, V), canary, dtype=torch.float32, device="cuda"),
        "token": torch.full((Bn,), -9, dtype=torch.int32, device="cuda"),
        "token_flags": torch.full((Bn,), -9, dtype=torch.int32, device="cuda"),
        "flags": torch.empty(Bn, dtype=torch.int32, device="cuda"),
        "p_tok": torch.empty(Bn, gamma, dtype=torch.float32, device="cuda"),
        "lse": torch.empty(Bn, gamma + 1, dtype=torch.float32, device="cuda"),
    }
    ev = B.dssd_edge_verify_bonus(tl, g["draft_tokens"], g["draft_q_tok"], g["uniforms"], g["uniforms_rs"], T, out=out)
    torch.cuda.synchronize()
    n_gpu = ev["accept_len"].cpu().numpy()
    assert (ev["flags"].cpu().numpy().astype(np.uint32) == ref["flags"]).all()
    near = ref["margin_acc"] < NEAR
    assert ((n_gpu == ref["accept_len"]) | near).all()
    same = n_gpu == ref["accept_len"]
    if gamma:
        assert prob_close(ev["p_tok"].cpu().numpy(), ref["p_tok"]).all()
    p_gpu = ev["p_row"].cpu().numpy()
    full_gpu = n_gpu == gamma
    # a row goes down only after a rejection; the rows of fully accepted sequences are untouched
    assert (p_gpu[full_gpu] == canary).all()
    rej = same & ~full_gpu
    assert prob_close(p_gpu[rej], ref["p_row"][rej]).all()
    tok1 = ev["token"].cpu().numpy()
    fl1 = ev["token_flags"].cpu().numpy().astype(np.uint32)
    assert (tok1[~full_gpu] == -1).all() and (fl1[~full_gpu] == 0).all()
    full = same & full_gpu
    slack = np.maximum(NEAR, 2 * RTOL)
    assert ((tok1[full] == ref["bonus_token"][full]) | (ref["margin_cdf"][full] < slack)).all()
    assert (fl1[full] == ref["bonus_flags"][full]).all()
    # the device half: rejected sequences only, into the same arrays
    rs = B.dssd_device_resample_rejected(ev["p_row"], g["draft_q"], ev["accept_len"], g["uniforms_rs"], gamma,
                                         out={"token": ev["token"], "flags": ev["token_flags"]})
    torch.cuda.synchronize()
    tok2 = rs["token"].cpu().numpy()
    fl2 = rs["flags"].cpu().numpy().astype(np.uint32)
    assert (tok2[full_gpu] == tok1[full_gpu]).all() and (fl2[full_gpu] == fl1[full_gpu]).all()
    slack_rs = np.maximum(NEAR, 2 * RTOL / np.maximum(ref["Z"], 1e-30))
    assert ((tok2[rej] == ref["token"][rej]) | (ref["margin_cdf"][rej] < slack_rs[rej])).all()
    # the split CUDA round (which may take another kernel for this launch, with the float32 sums in
    # another order): same decisions and flags, same tokens away from CDF steps, rows equal up to
    # the order of summation
    sv = B.dssd_edge_verify(tl, g["draft_tokens"], g["draft_q_tok"], g["uniforms"], T)
    sr = B.dssd_device_resample(sv["p_row"], g["draft_q"], sv["accept_len"], g["uniforms_rs"], gamma)
    torch.cuda.synchronize()
    assert torch.equal(sv["flags"], ev["flags"]) and torch.equal(sr["flags"], rs["flags"])
    assert ((sv["accept_len"].cpu().numpy() == n_gpu) | near).all()
    clear = same & (ref["margin_cdf"] >= np.where(full_gpu, slack, slack_rs))
    assert (sr["token"].cpu().numpy()[clear] == tok2[clear]).all()
    keep = torch.from_numpy(same & ~full_gpu).cuda()
    x, y = sv["p_row"][keep].double(), ev["p_row"][keep].double()
    assert (((x - y).abs() <= 1e-7 + 2e-6 * y.abs()) | (x.isnan() & y.isnan())).all()
    return {"full": int(full_gpu.sum()), "rejected": int((~full_gpu).sum())}


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_small_vocabularies(B, oracle_mod, dtype):
    seed = 700
    for V in (1, 3, 7, 33, 1000, 1025, 16389):
        for gamma in (0, 3):
            for Bn in (2, 150):
                seed += 1
                w = di.custom(B=Bn, gamma=gamma, V=V, dtype=dtype, temperature=0.9, sigma_d=0.3, zipf=V > 8, seed=seed)
                compare_bonus(B, oracle_mod, di.generate(w, threads=4), w.temperature)


@pytest.mark.parametrize("dtype,V,gamma,Bn,sigma", [
    ("f32", 50272, 2, 6, 0.2), ("bf16", 40003, 3, 5, 0.2), ("bf16", 128256, 8, 4, 0.1), ("f32", 20001, 16, 3, 0.05),
    ("bf16", 151936, 4, 9, 0.3), ("f32", 16385, 1, 40, 0.6), ("bf16", 32768, 2, 200, 0.4),
])
def test_several_slices_and_ragged_tails(B, oracle_mod, dtype, V, gamma, Bn, sigma):
    w = di.custom(B=Bn, gamma=gamma, V=V, dtype=dtype, temperature=0.8, sigma_d=sigma, seed=V + gamma)
    rep = compare_bonus(B, oracle_mod, di.generate(w, threads=4), w.temperature)
    print(rep)


def test_all_accepted_and_none_accepted(B, oracle_mod):
    w = di.custom(B=40, gamma=3, V=9000, dtype="bf16", temperature=1.0, sigma_d=0.5, seed=12)
    d = di.generate(w, threads=4)
    d["uniforms"][:] = 0.0
    assert compare_bonus(B, oracle_mod, d, w.temperature) == {"full": 40, "rejected": 0}
    d["uniforms"][:] = 1.0 - 2.0 ** -24
    d["draft_q_tok"][:] = 1.0
    assert compare_bonus(B, oracle_mod, d, w.temperature) == {"full": 0, "rejected": 40}


def test_unaligned_rows(B, oracle_mod):
    for dtype, V, off in (("f32", 1000, 1), ("bf16", 4097, 3), ("bf16", 20000, 1)):
        w = di.custom(B=21, gamma=2, V=V, dtype=dtype, sigma_d=0.2, seed=V)
        d = di.generate(w)
        stride = V + 5

        def view(t):
            buf = torch.zeros(w.B * 3 * stride + 16, dtype=t.dtype, device="cuda")
            v = buf[off:off + w.B * 3 * stride].view(w.B, 3, stride)[:, :, :V]
            v.copy_(t)
            assert v.data_ptr() % 16 != 0
            return v

        compare_bonus(B, oracle_mod, d, w.temperature, logits_view=view)


def test_rows_without_a_distribution(B, oracle_mod):
    """A fully accepted sequence whose bonus row holds NaN, +inf or no mass: token -1, INVALID."""
    V, gamma, Bn = 3000, 2, 6
    w = di.custom(B=Bn, gamma=gamma, V=V, dtype="f32", seed=5)
    d = di.generate(w)
    d["uniforms"][:] = 0.0  # everything accepted
    d["target_logits"][0, gamma, 17] = np.nan
    d["target_logits"][1, gamma, 5] = np.inf
    d["target_logits"][2, gamma, :] = -np.inf
    d["target_logits"][3, gamma, ::2] = -np.inf
    rep = compare_bonus(B, oracle_mod, d, 1.0)
    assert rep["full"] == Bn


@pytest.mark.parametrize("name", ["c3", "c4"])
def test_full_size_configs(B, oracle_mod, name):
    w = di.get_workload(name)
    rep = compare_bonus(B, oracle_mod, di.generate(w, threads=8), w.temperature, threads=8)
    print(name, rep)
    assert rep["full"] > 0 and rep["rejected"] > 0


def test_garbage_workspace_and_cuda_graph(B):
    w = di.custom(B=160, gamma=3, V=12000, dtype="bf16", temperature=0.8, sigma_d=0.3, seed=78)
    g = to_device(di.generate(w, threads=4))
    n1 = B.dssd_edge_verify_bonus_workspace_bytes(w.B, w.gamma, w.V)

    def run(ws, ws2, out=None):
        ev = B.dssd_edge_verify_bonus(g["target_logits"], g["draft_tokens"], g["draft_q_tok"], g["uniforms"],
                                      g["uniforms_rs"], w.temperature, workspace=ws, out=out)
        B.dssd_device_resample_rejected(ev["p_row"], g["draft_q"], ev["accept_len"], g["uniforms_rs"], w.gamma,
                                        out={"token": ev["token"], "flags": ev["token_flags"]}, workspace=ws2)
        return ev

    ref = None
    for fill in (0, 0xFF, None):
        mk = (lambda: torch.randint(0, 256, (n1,), dtype=torch.uint8, device="cuda")) if fill is None else \
             (lambda: torch.full((n1,), fill, dtype=torch.uint8, device="cuda"))
        cur = run(mk(), mk())
        torch.cuda.synchronize()
        cur = {k: v.clone() for k, v in cur.items()}
        if ref is None:
            ref = cur
        for k in ("accept_len", "token", "token_flags", "flags"):
            assert torch.equal(cur[k], ref[k]), k
        assert torch.equal(cur["p_row"].view(torch.int32), ref["p_row"].view(torch.int32))
    ws, ws2 = torch.empty(n1, dtype=torch.uint8, device="cuda"), torch.empty(n1, dtype=torch.uint8, device="cuda")
    out = run(ws, ws2)
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            run(ws, ws2, out=out)
    out["token"].fill_(-5)
    for _ in range(2):
        graph.replay()
    torch.cuda.synchronize()
    for k in ("accept_len", "token", "token_flags", "flags"):
        assert torch.equal(out[k], ref[k]), k


def test_rejected_only_draw_leaves_other_entries_alone(B, oracle_mod):
    """dssd_device_resample_rejected on hand-made accepted lengths: n < gamma is drawn for, n == gamma
    keeps what the arrays held, n outside [0, gamma] gives token -1 and DSSD_RS_FLAG_INVALID."""
    V, gamma = 9000, 3
    rng = np.random.default_rng(3)
    p = rng.random((6, V)).astype(np.float32)
    p /= p.sum(axis=1, keepdims=True)
    q = rng.random((6, gamma, V)).astype(np.float32)
    q /= q.sum(axis=2, keepdims=True)
    n = np.array([0, gamma, -1, gamma + 1, 2, gamma], np.int32)
    u = rng.random(6).astype(np.float32)
    ref = oracle_mod.device_resample(p, q, n, u, gamma)
    tok = torch.full((6,), -77, dtype=torch.int32, device="cuda")
    fl = torch.full((6,), -77, dtype=torch.int32, device="cuda")
    B.dssd_device_resample_rejected(torch.from_numpy(p).cuda(), torch.from_numpy(q).cuda(), torch.from_numpy(n).cuda(),
                                    torch.from_numpy(u).cuda(), gamma, out={"token": tok, "flags": fl})
    torch.cuda.synchronize()
    tok, fl = tok.cpu().numpy(), fl.cpu().numpy()
    for b in (0, 4):
        assert tok[b] == ref["token"][b] and np.uint32(fl[b]) == ref["flags"][b]
    for b in (1, 5):
        assert tok[b] == -77 and fl[b] == -77
    for b in (2, 3):
        assert tok[b] == -1 and np.uint32(fl[b]) == ref["flags"][b] == oracle_mod.RS_FLAG_INVALID
