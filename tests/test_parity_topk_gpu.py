"""Parity of the truncated-support (top-k) CUDA path, through the C ABI, with the CPU oracle.

Both sides evaluate probabilities and the acceptance test in float64, so supports, accepted
lengths and tokens are compared exactly; only a decision whose margin is at rounding level
(different exp implementations) may differ, and float32 payload values may differ in the last bit.
"""
import numpy as np
import pytest
import torch

import dssd_inputs as di
from gpu_util import to_device

pytestmark = pytest.mark.gpu

EDGE = 1e-12   # |u - min(1, p/q)| or CDF-step distance below which a float64 decision may flip
RTOL_VAL = 3e-7  # float32 payload: the float64 value rounded once, +- one more bit


@pytest.fixture(scope="module")
def B():
    from paper_2507_12000_b200 import binding

    assert torch.cuda.is_available()
    return binding


def _val_close(gpu, ref):
    gpu = gpu.astype(np.float64)
    ref = ref.astype(np.float64)
    return (np.isnan(gpu) & np.isnan(ref)) | (np.abs(gpu - ref) <= RTOL_VAL * np.abs(ref))


def compare_topk(B, O, d, T, k, logits_view=None, threads=4):
    gamma = d["target_logits"].shape[1] - 1
    ref = O.verify_round_topk(d, T, k, threads=threads)
    g = to_device(d)
    tl = g["target_logits"] if logits_view is None else logits_view(g["target_logits"])
    ev = B.dssd_edge_verify_topk(tl, g["draft_tokens"], g["draft_q_tok"], g["uniforms"], T, k)
    torch.cuda.synchronize()
    n_gpu = ev["accept_len"].cpu().numpy()
    assert (ev["flags"].cpu().numpy().astype(np.uint32) == ref["flags"]).all()
    edge = ref["margin_acc"] < EDGE
    bad = (n_gpu != ref["accept_len"]) & ~edge
    assert not bad.any(), (np.nonzero(bad)[0][:8], n_gpu[bad][:8], ref["accept_len"][bad][:8])
    same = n_gpu == ref["accept_len"]
    idx_gpu = ev["p_idx"].cpu().numpy()
    assert (idx_gpu[same] == ref["p_idx"][same]).all(), np.argwhere(idx_gpu[same] != ref["p_idx"][same])[:8]
    assert _val_close(ev["p_val"].cpu().numpy()[same], ref["p_val"][same]).all()
    if gamma:
        assert _val_close(ev["p_tok"].cpu().numpy(), ref["p_tok"].astype(np.float32)).all()
    # device half in isolation, on the oracle's pairs: bit-exact
    rs = B.dssd_device_resample_topk(torch.from_numpy(ref["p_idx"]).cuda(), torch.from_numpy(ref["p_val"]).cuda(),
                                     g.get("q_idx"), g.get("q_val"), torch.from_numpy(ref["accept_len"]).cuda(),
                                     g["uniforms_rs"], gamma)
    torch.cuda.synchronize()
    assert (rs["token"].cpu().numpy() == ref["token"]).all()
    assert (rs["flags"].cpu().numpy().astype(np.uint32) == ref["rs_flags"]).all()
    # end to end on the CUDA path's own pairs
    rs2 = B.dssd_device_resample_topk(ev["p_idx"], ev["p_val"], g.get("q_idx"), g.get("q_val"), ev["accept_len"],
                                      g["uniforms_rs"], gamma)
    torch.cuda.synchronize()
    tok = rs2["token"].cpu().numpy()
    slack = np.maximum(1e-6, 4 * RTOL_VAL / np.maximum(ref["Z"], 1e-30))
    bad = (tok != ref["token"]) & same & ~(ref["margin_cdf"] < slack)
    assert not bad.any(), (np.nonzero(bad)[0][:8], tok[bad][:8], ref["token"][bad][:8])
    return {"mismatch_accept": int((n_gpu != ref["accept_len"]).sum()), "mismatch_token": int((tok != ref["token"]).sum()),
            "accept_rate": float(ref["accept_len"].mean() / max(gamma, 1))}


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_small_vocabularies(B, oracle_mod, dtype):
    seed = 300
    for V in (1, 2, 9, 33, 1000, 2049, 4100):
        for gamma in (0, 1, 3):
            for k in (1, 10, 32):
                if k > V:
                    continue
                seed += 1
                w = di.custom(B=3, gamma=gamma, V=V, dtype=dtype, temperature=0.9, sigma_d=0.6, zipf=V > 8, seed=seed)
                compare_topk(B, oracle_mod, di.generate_topk(w, k), w.temperature, k, threads=1)


@pytest.mark.parametrize("name", ["c1", "c2"])
def test_small_configs(B, oracle_mod, name):
    w = di.get_workload(name)
    rep = compare_topk(B, oracle_mod, di.generate_topk(w, 10), w.temperature, 10)
    assert rep["mismatch_accept"] == 0 and rep["mismatch_token"] == 0


@pytest.mark.parametrize("dtype,V,gamma,Bn,k", [
    ("f32", 50272, 2, 6, 10), ("bf16", 40003, 3, 5, 10), ("bf16", 128256, 8, 4, 32), ("f32", 20001, 16, 3, 5),
    ("bf16", 151936, 4, 9, 10), ("f32", 16385, 1, 700, 10), ("bf16", 8192, 33, 2, 1), ("f32", 70000, 40, 2, 17),
    ("bf16", 5000, 2, 1300, 10),
])
def test_several_pieces_and_ragged_tails(B, oracle_mod, dtype, V, gamma, Bn, k):
    w = di.custom(B=Bn, gamma=gamma, V=V, dtype=dtype, temperature=0.8, sigma_d=0.5, seed=V + gamma)
    compare_topk(B, oracle_mod, di.generate_topk(w, k, threads=4), w.temperature, k)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_ties_and_adversarial_orders(B, oracle_mod, dtype):
    """Rows full of equal logits, ascending and descending rows (the candidate buffer overflows
    on ascending input), constant rows, signed zeros."""
    rng = np.random.default_rng(5)
    Bn, gamma, V, k = 6, 4, 30011, 10
    w = di.custom(B=Bn, gamma=gamma, V=V, dtype="f32", seed=9)
    d = di.generate_topk(w, k)
    tl = np.empty((Bn, gamma + 1, V), np.float32)
    tl[0] = rng.integers(-2, 3, size=(gamma + 1, V)).astype(np.float32)       # a handful of distinct values
    tl[1] = np.linspace(-8, 8, V, dtype=np.float32)[None]                      # ascending
    tl[2] = np.linspace(8, -8, V, dtype=np.float32)[None]                      # descending
    tl[3] = 1.5                                                                 # constant
    tl[4] = rng.choice(np.array([0.0, -0.0], np.float32), size=(gamma + 1, V))  # signed zeros only
    tl[5] = np.round(rng.standard_normal((gamma + 1, V)) * 2, 1)               # many ties at the top
    # drafted tokens inside the target support now and then, so that some drafts are accepted
    for b in range(Bn):
        for i in range(gamma):
            order = np.lexsort((np.arange(V), -tl[b, i].astype(np.float64)))
            d["draft_tokens"][b, i] = order[(b + i) % k]
    d["target_logits"] = di.f32_to_bf16_bits(tl) if dtype == "bf16" else tl
    rep = compare_topk(B, oracle_mod, d, 1.0, k)
    assert rep["mismatch_accept"] == 0


def test_strided_and_unaligned_rows(B, oracle_mod):
    for dtype, V, off, Bn in (("f32", 1000, 1, 3), ("bf16", 4097, 3, 3), ("bf16", 20000, 1, 200), ("f32", 9001, 2, 151)):
        w = di.custom(B=Bn, gamma=2, V=V, dtype=dtype, seed=V)
        d = di.generate_topk(w, 10)
        stride = V + 5

        def view(t, stride=stride, off=off, Bn=Bn, V=V):
            buf = torch.zeros(Bn * 3 * stride + 16, dtype=t.dtype, device="cuda")
            v = buf[off:off + Bn * 3 * stride].view(Bn, 3, stride)[:, :, :V]
            v.copy_(t)
            assert v.data_ptr() % 16 != 0
            return v

        compare_topk(B, oracle_mod, d, w.temperature, 10, logits_view=view)


def test_anomalies_are_flagged_not_faulted(B, oracle_mod):
    V, gamma, Bn, k = 3000, 3, 9, 10
    w = di.custom(B=Bn, gamma=gamma, V=V, dtype="f32", seed=5)
    d = di.generate_topk(w, k)
    tl = d["target_logits"]
    tl[0, 1, 17] = np.nan
    tl[1, 0, 5] = np.inf
    tl[2, 2, :] = -np.inf
    tl[3, 1, 12:] = -np.inf           # fewer finite entries than k: the support holds zero-mass entries
    d["draft_tokens"][4, 0] = -1
    d["draft_tokens"][5, 2] = V
    d["draft_q_tok"][6, 0] = 0.0
    d["uniforms"][7, :] = 0.0
    tl[8, gamma, 100] = np.nan        # the bonus row itself is bad
    d["uniforms"][8, :] = 0.0
    ref = oracle_mod.edge_verify_topk(tl, d["draft_tokens"], d["draft_q_tok"], d["uniforms"], 1.0, k)
    assert list(ref["flags"][:6]) == [2, 2, 2, 0, 1, 1] and ref["flags"][8] == 2
    compare_topk(B, oracle_mod, d, 1.0, k)


def test_first_rejection_beyond_32_positions(B, oracle_mod):
    """The sequence fold looks at 32 verdicts at a time: runs of accepted positions that cross that
    boundary, a first rejection exactly at 31, 32, 33 and at the last position, and no rejection at all."""
    V, gamma, k = 9000, 45, 10
    rejects = [31, 32, 33, 44, None, 0]
    w = di.custom(B=len(rejects), gamma=gamma, V=V, dtype="bf16", temperature=0.9, sigma_d=0.4, seed=41)
    d = di.generate_topk(w, k)
    d["uniforms"][:] = 0.0          # u = 0 accepts every token with p > 0 ...
    top = np.argmax(di.bf16_bits_to_f32(d["target_logits"][:, :gamma]), axis=-1)
    d["draft_tokens"][:] = top.astype(np.int32)   # ... and the row's best token is in its support
    for b, j in enumerate(rejects):
        if j is not None:
            d["uniforms"][b, j] = 0.99999         # ... except here: q = 1 and p < 1 reject
            d["draft_q_tok"][b, j] = 1.0
    ref = oracle_mod.edge_verify_topk(d["target_logits"], d["draft_tokens"], d["draft_q_tok"], d["uniforms"], w.temperature, k)
    assert list(ref["accept_len"]) == [gamma if j is None else j for j in rejects]
    compare_topk(B, oracle_mod, d, w.temperature, k)


@pytest.mark.parametrize("name,k", [("c2", 10), ("c1", 1)])
def test_round_on_host_buffers(B, oracle_mod, name, k):
    """dssd_round_host_topk on pinned host tensors and a garbage-filled arena, against the oracle's round;
    a second call on the same arena (captured-style reuse) gives the same results."""
    w = di.get_workload(name)
    d = di.generate_topk(w, k)
    ref = oracle_mod.verify_round_topk(d, w.temperature, k, threads=4)
    host = {}
    for key, v in d.items():
        t = torch.from_numpy(v.view(np.int16)).view(torch.bfloat16) if v.dtype == np.uint16 else torch.from_numpy(v)
        host[key] = t.pin_memory()
    code = B.DSSD_BF16 if w.dtype == "bf16" else B.DSSD_F32
    arena = torch.randint(0, 256, (B.dssd_round_host_topk_arena_bytes(w.B, w.gamma, w.V, k, code),), dtype=torch.uint8,
                          device="cuda")
    for _ in range(2):
        out = B.dssd_round_host_topk(host, w.temperature, k, arena, want_pairs=True)
        torch.cuda.synchronize()
        edge = ref["margin_acc"] < EDGE
        n = out["accept_len"].numpy()
        assert ((n == ref["accept_len"]) | edge).all()
        same = n == ref["accept_len"]
        assert (out["edge_flags"].numpy().astype(np.uint32) == ref["flags"]).all()
        assert (out["p_idx"].numpy()[same] == ref["p_idx"][same]).all()
        assert _val_close(out["p_val"].numpy()[same], ref["p_val"][same]).all()
        slack = np.maximum(1e-6, 4 * RTOL_VAL / np.maximum(ref["Z"], 1e-30))
        bad = (out["token"].numpy() != ref["token"]) & same & ~(ref["margin_cdf"] < slack)
        assert not bad.any()
    # the call waits for nothing on the host, so it can be recorded in a CUDA graph and replayed
    want_n, want_tok = out["accept_len"].clone(), out["token"].clone()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            B.dssd_round_host_topk(host, w.temperature, k, arena, out=out)
    out["accept_len"].fill_(-7)
    out["token"].fill_(-7)
    graph.replay()
    torch.cuda.synchronize()
    assert (out["accept_len"] == want_n).all() and (out["token"] == want_tok).all()
    # host-side refusals: nothing is enqueued
    with pytest.raises(B.DssdError):
        B.dssd_round_host_topk(host, w.temperature, k, arena[: arena.numel() // 2])
    with pytest.raises(B.DssdError):
        B.dssd_round_host_topk(host, w.temperature, 33, arena)
    assert B.dssd_round_host_topk_arena_bytes(w.B, w.gamma, w.V, 0, code) == 0


def test_run_to_run_determinism(B):
    w = di.custom(B=300, gamma=4, V=50000, dtype="bf16", seed=77)
    g = to_device(di.generate_topk(w, 10, threads=4))
    outs = []
    for _ in range(3):
        ev = B.dssd_edge_verify_topk(g["target_logits"], g["draft_tokens"], g["draft_q_tok"], g["uniforms"], 0.8, 10)
        rs = B.dssd_device_resample_topk(ev["p_idx"], ev["p_val"], g["q_idx"], g["q_val"], ev["accept_len"],
                                         g["uniforms_rs"], w.gamma)
        torch.cuda.synchronize()
        outs.append({k: v.clone() for k, v in {**ev, "token": rs["token"]}.items()})
    for o in outs[1:]:
        for k in ("accept_len", "token", "flags", "p_idx"):
            assert torch.equal(o[k], outs[0][k])
        for k in ("p_val", "p_tok"):
            assert torch.equal(o[k].view(torch.int32), outs[0][k].view(torch.int32)), k


def test_outputs_stay_inside_their_buffers(B):
    w = di.custom(B=5, gamma=3, V=12345, dtype="bf16", seed=3)
    k = 10
    g = to_device(di.generate_topk(w, k))
    Bn, gamma = w.B, w.gamma
    pad = 64

    def guarded(n, dtype):
        t = torch.full((n + 2 * pad,), -7, dtype=dtype, device="cuda")
        return t, t[pad:pad + n]

    full, out = {}, {}
    for name, n, dt in (("accept_len", Bn, torch.int32), ("p_idx", Bn * k, torch.int32), ("p_val", Bn * k, torch.float32),
                        ("p_tok", Bn * gamma, torch.float32), ("flags", Bn, torch.int32)):
        full[name], out[name] = guarded(n, dt)
    out["p_idx"] = out["p_idx"].view(Bn, k)
    out["p_val"] = out["p_val"].view(Bn, k)
    B.dssd_edge_verify_topk(g["target_logits"], g["draft_tokens"], g["draft_q_tok"], g["uniforms"], 1.0, k, out=out)
    rf, rt = guarded(Bn, torch.int32)
    ff, ft = guarded(Bn, torch.int32)
    B.dssd_device_resample_topk(out["p_idx"], out["p_val"], g["q_idx"], g["q_val"], out["accept_len"],
                                g["uniforms_rs"], gamma, out={"token": rt, "flags": ft})
    torch.cuda.synchronize()
    for t in list(full.values()) + [rf, ff]:
        assert (t[:pad] == -7).all() and (t[-pad:] == -7).all()
    assert (rt >= 0).all() and (rt < w.V).all()


@pytest.mark.parametrize("name", ["c3", "c4"])
def test_full_size_configs(B, oracle_mod, name):
    """The named configurations at full size with k = 10 (the experiments' sampler)."""
    w = di.get_workload(name)
    rep = compare_topk(B, oracle_mod, di.generate_topk(w, 10, threads=8), w.temperature, 10, threads=8)
    print(name, rep)
    assert rep["mismatch_accept"] == 0
