"""Parity of the CUDA path (through the C ABI) with the CPU oracle on seeded inputs."""
import numpy as np
import pytest
import torch

import dssd_inputs as di
from gpu_util import compare_round, prob_close, to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2507_12000_b200 import binding

    assert torch.cuda.is_available()
    return binding


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_tiny_grid(B, oracle_mod, dtype):
    """Small vocabularies around vector and warp boundaries, gamma 0..3, B 1..3."""
    seed = 100
    for V in (1, 2, 3, 5, 7, 8, 31, 33, 1000, 1025):
        for gamma in (0, 1, 2, 3):
            for Bn in (1, 2, 3):
                seed += 1
                w = di.custom(B=Bn, gamma=gamma, V=V, dtype=dtype, temperature=0.9, sigma_d=1.0,
                              zipf=V > 8, seed=seed)
                compare_round(B, oracle_mod, di.generate(w), w.temperature, threads=1)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_tiny_vocabularies_through_the_streaming_kernel(B, oracle_mod, dtype):
    """More sequences than SMs, so that the persistent streaming kernel (not the one-CTA-per-
    sequence kernel of small launches) sees vocabularies around vector and stage boundaries."""
    seed = 900
    for V in (1, 7, 33, 1025, 16389):
        for gamma in (0, 3):
            seed += 1
            w = di.custom(B=150, gamma=gamma, V=V, dtype=dtype, temperature=0.9, sigma_d=1.0, zipf=V > 8, seed=seed)
            compare_round(B, oracle_mod, di.generate(w, threads=4), w.temperature, threads=4)


@pytest.mark.parametrize("name", ["c1", "c2"])
def test_small_configs(B, oracle_mod, name):
    w = di.get_workload(name)
    rep = compare_round(B, oracle_mod, di.generate(w), w.temperature)
    assert rep["mismatch_accept"] == 0 and rep["mismatch_token_iso"] == 0


@pytest.mark.parametrize("dtype,V,gamma,Bn", [
    ("f32", 50272, 2, 6), ("bf16", 40003, 3, 5), ("bf16", 128256, 8, 4), ("f32", 20001, 16, 3),
    ("bf16", 151936, 4, 9), ("f32", 16385, 1, 40), ("bf16", 8192, 33, 2), ("f32", 70000, 40, 2),
])
def test_several_slices_and_ragged_tails(B, oracle_mod, dtype, V, gamma, Bn):
    w = di.custom(B=Bn, gamma=gamma, V=V, dtype=dtype, temperature=0.8, sigma_d=0.8, seed=V + gamma)
    compare_round(B, oracle_mod, di.generate(w, threads=4), w.temperature)


@pytest.mark.parametrize("name", ["c3", "c4"])
def test_full_size_configs(B, oracle_mod, name):
    """The full named configurations, in the launch configuration the benchmark times."""
    w = di.get_workload(name)
    rep = compare_round(B, oracle_mod, di.generate(w, threads=8), w.temperature)
    print(name, rep)
    assert rep["mismatch_accept"] <= rep["near_acc"]
    assert rep["mismatch_token_iso"] <= rep["near_cdf"]


def test_largest_sweep_point_sampled(B, oracle_mod):
    """B=1024, gamma=16, V=50272 float32 (3.5 GB of logits) in the benchmark's launch configuration;
    the oracle checks a sample of the sequences one by one."""
    w = di.sweep_max()
    d = di.generate(w, threads=16)
    g = to_device(d)
    ev = B.dssd_edge_verify(g["target_logits"], g["draft_tokens"], g["draft_q_tok"], g["uniforms"], w.temperature)
    rs = B.dssd_device_resample(ev["p_row"], g["draft_q"], ev["accept_len"], g["uniforms_rs"], w.gamma)
    torch.cuda.synchronize()
    n_gpu = ev["accept_len"].cpu().numpy()
    tok_gpu = rs["token"].cpu().numpy()
    assert (ev["flags"].cpu().numpy() == 0).all()
    assert ((n_gpu >= 0) & (n_gpu <= w.gamma)).all() and ((tok_gpu >= 0) & (tok_gpu < w.V)).all()
    sample = np.r_[0:24, 500:524, w.B - 24:w.B]
    sub = {k: np.ascontiguousarray(v[sample]) for k, v in d.items()}
    ref = oracle_mod.verify_round(sub, w.temperature, threads=8)
    near = (ref["margin_acc"] < 1e-6)
    assert ((n_gpu[sample] == ref["accept_len"]) | near).all()
    same = n_gpu[sample] == ref["accept_len"]
    p_gpu = ev["p_row"][torch.from_numpy(sample).cuda()].cpu().numpy()
    assert prob_close(p_gpu[same], ref["p_row"][same]).all()
    slack = np.maximum(1e-6, 2e-5 / np.maximum(ref["Z"], 1e-30))
    assert ((tok_gpu[sample] == ref["token"]) | ~same | (ref["margin_cdf"] < slack)).all()


def test_sweep_points_sampled(B, oracle_mod):
    """A spread of the V=50272 sweep (largest batch sizes run on a slice of their sequences)."""
    for w in di.sweep_points():
        if (w.B, w.gamma) in ((1, 1), (16, 4), (128, 2), (1, 16), (16, 16)):
            compare_round(B, oracle_mod, di.generate(w, threads=8), w.temperature)


@pytest.mark.parametrize("Bn", [3, 151])  # one CTA per sequence / the streaming kernel
def test_strided_and_unaligned_rows(B, oracle_mod, Bn):
    for dtype, V, off in (("f32", 1000, 1), ("bf16", 4097, 3), ("bf16", 20000, 1), ("f32", 9001, 2)):
        w = di.custom(B=Bn, gamma=2, V=V, dtype=dtype, seed=V)
        d = di.generate(w)
        ref = oracle_mod.verify_round(d, w.temperature)
        g = to_device(d)
        stride = V + 5
        buf = torch.zeros(Bn * 3 * stride + 16, dtype=g["target_logits"].dtype, device="cuda")
        view = buf[off:off + Bn * 3 * stride].view(Bn, 3, stride)[:, :, :V]
        view.copy_(g["target_logits"])
        assert view.data_ptr() % 16 != 0
        ev = B.dssd_edge_verify(view, g["draft_tokens"], g["draft_q_tok"], g["uniforms"], w.temperature)
        torch.cuda.synchronize()
        assert (ev["accept_len"].cpu().numpy() == ref["accept_len"]).all()
        assert prob_close(ev["p_row"].cpu().numpy(), ref["p_row"]).all()
        assert prob_close(ev["p_tok"].cpu().numpy(), ref["p_tok"]).all()


def test_run_to_run_determinism(B):
    w = di.custom(B=24, gamma=4, V=50000, dtype="bf16", seed=77)
    g = to_device(di.generate(w, threads=4))
    outs = []
    for _ in range(3):
        ev = B.dssd_edge_verify(g["target_logits"], g["draft_tokens"], g["draft_q_tok"], g["uniforms"], 0.8)
        rs = B.dssd_device_resample(ev["p_row"], g["draft_q"], ev["accept_len"], g["uniforms_rs"], w.gamma)
        torch.cuda.synchronize()
        outs.append({k: v.clone() for k, v in {**ev, "token": rs["token"]}.items()})
    for o in outs[1:]:
        for k in ("accept_len", "token", "flags"):
            assert torch.equal(o[k], outs[0][k])
        for k in ("p_row", "p_tok", "lse"):
            assert torch.equal(o[k].view(torch.int32), outs[0][k].view(torch.int32)), k


def test_anomalies_are_flagged_not_faulted(B, oracle_mod):
    V, gamma, Bn = 3000, 3, 8
    w = di.custom(B=Bn, gamma=gamma, V=V, dtype="f32", seed=5)
    d = di.generate(w)
    tl = d["target_logits"]
    tl[0, 1, 17] = np.nan
    tl[1, 0, 5] = np.inf
    tl[2, 2, :] = -np.inf
    tl[3, 1, ::2] = -np.inf          # legitimate zero-mass entries
    d["draft_tokens"][4, 0] = -1
    d["draft_tokens"][5, 2] = V
    d["draft_q_tok"][6, 0] = 0.0     # q = 0, p > 0: accepted
    d["uniforms"][6, 0] = 0.99
    d["uniforms"][7, :] = 0.0        # u = 0 accepts whenever p > 0
    ref = oracle_mod.edge_verify(tl, d["draft_tokens"], d["draft_q_tok"], d["uniforms"], 1.0)
    g = to_device(d)
    ev = B.dssd_edge_verify(g["target_logits"], g["draft_tokens"], g["draft_q_tok"], g["uniforms"], 1.0)
    torch.cuda.synchronize()
    assert (ev["flags"].cpu().numpy().astype(np.uint32) == ref["flags"]).all()
    assert list(ref["flags"][:6]) == [2, 2, 2, 0, 1, 1]
    assert (ev["accept_len"].cpu().numpy() == ref["accept_len"]).all()
    clean = ref["flags"] == 0
    assert prob_close(ev["p_row"].cpu().numpy()[clean], ref["p_row"][clean]).all()
    assert prob_close(ev["p_tok"].cpu().numpy(), ref["p_tok"]).all()
    # device half: p == q (no residual mass), bad accept_len, all-zero row
    p = torch.full((4, V), 1.0 / V, device="cuda")
    q = torch.full((4, gamma, V), 1.0 / V, device="cuda")
    p[3] = 0.0
    n = torch.tensor([1, gamma + 1, -1, gamma], dtype=torch.int32, device="cuda")
    u = torch.tensor([0.5, 0.5, 0.5, 0.5], device="cuda")
    rs = B.dssd_device_resample(p, q, n, u, gamma)
    torch.cuda.synchronize()
    rr = oracle_mod.device_resample(p.cpu().numpy(), q.cpu().numpy(), n.cpu().numpy(), u.cpu().numpy(), gamma)
    assert (rs["token"].cpu().numpy() == rr["token"]).all()
    assert (rs["flags"].cpu().numpy().astype(np.uint32) == rr["flags"]).all()
    assert list(rr["flags"]) == [2, 4, 4, 5] and list(rr["token"]) == [V // 2, -1, -1, -1]


@pytest.mark.parametrize("Bn,V", [(6, 9000), (200, 4500)])
def test_first_rejection_beyond_32_positions(B, oracle_mod, Bn, V):
    """Long runs of accepted positions: first rejection exactly at 31, 32, 33, at the last position, at 0,
    and no rejection at all (u = 0 accepts whatever has p > 0; u close to 1 with q = 1 rejects), through
    the small-launch kernel (few sequences) and the streaming kernel (many)."""
    gamma = 45
    rejects = [31, 32, 33, 44, None, 0]
    w = di.custom(B=Bn, gamma=gamma, V=V, dtype="bf16", temperature=0.9, sigma_d=0.4, seed=43)
    d = di.generate(w, threads=4)
    d["uniforms"][:] = 0.0
    for b in range(Bn):
        j = rejects[b % len(rejects)]
        if j is not None:
            d["uniforms"][b, j] = 0.99999
            d["draft_q_tok"][b, j] = 1.0
    ref = oracle_mod.edge_verify(d["target_logits"], d["draft_tokens"], d["draft_q_tok"], d["uniforms"], w.temperature)
    want = [gamma if rejects[b % len(rejects)] is None else rejects[b % len(rejects)] for b in range(Bn)]
    assert list(ref["accept_len"]) == want
    compare_round(B, oracle_mod, d, w.temperature)


def test_outputs_stay_inside_their_buffers(B):
    """Canary words either side of every output survive the call."""
    w = di.custom(B=5, gamma=3, V=12345, dtype="bf16", seed=3)
    g = to_device(di.generate(w))
    Bn, gamma, V = w.B, w.gamma, w.V
    pad = 64

    def guarded(n, dtype):
        t = torch.full((n + 2 * pad,), -7, dtype=dtype, device="cuda")
        return t, t[pad:pad + n]

    full = {}
    out = {}
    for k, n, dt in (("accept_len", Bn, torch.int32), ("p_row", Bn * V, torch.float32),
                     ("p_tok", Bn * gamma, torch.float32), ("lse", Bn * (gamma + 1), torch.float32),
                     ("flags", Bn, torch.int32)):
        full[k], out[k] = guarded(n, dt)
    out["p_row"] = out["p_row"].view(Bn, V)
    B.dssd_edge_verify(g["target_logits"], g["draft_tokens"], g["draft_q_tok"], g["uniforms"], 1.0, out=out)
    rf, rt = guarded(Bn, torch.int32)
    ff, ft = guarded(Bn, torch.int32)
    B.dssd_device_resample(out["p_row"], g["draft_q"], out["accept_len"], g["uniforms_rs"], gamma,
                           out={"token": rt, "flags": ft})
    torch.cuda.synchronize()
    for t in list(full.values()) + [rf, ff]:
        assert (t[:pad] == -7).all() and (t[-pad:] == -7).all()
    assert (rt >= 0).all() and (rt < V).all()


def test_round_on_host_buffers(B, oracle_mod):
    w = di.get_workload("c2")
    d = di.generate(w)
    ref = oracle_mod.verify_round(d, w.temperature)
    host = {}
    for k, v in d.items():
        t = torch.from_numpy(v.view(np.int16)).view(torch.bfloat16) if v.dtype == np.uint16 else torch.from_numpy(v)
        host[k] = t.pin_memory()
    arena = torch.empty(B.dssd_round_host_arena_bytes(w.B, w.gamma, w.V, B.DSSD_BF16), dtype=torch.uint8, device="cuda")
    out = B.dssd_round_host(host, w.temperature, arena, want_p_row=True)
    torch.cuda.synchronize()
    assert (out["accept_len"].numpy() == ref["accept_len"]).all()
    assert (out["token"].numpy() == ref["token"]).all()
    assert (out["rs_flags"].numpy().astype(np.uint32) == ref["rs_flags"]).all()
    assert prob_close(out["p_row"].numpy(), ref["p_row"]).all()


@pytest.mark.parametrize("gamma", [0, 3])
def test_round_on_host_buffers_uploads_only_the_rows_it_reads(B, oracle_mod, gamma):
    """Every row of draft_q except Q_n of the sequences with a rejection is poisoned on the host:
    the results must not change (those rows neither cross the bus nor are read)."""
    w = di.custom(B=24, gamma=gamma, V=20000, dtype="f32", temperature=0.9, sigma_d=0.5, seed=41 + gamma)
    d = di.generate(w)
    ref = oracle_mod.verify_round(d, w.temperature)
    assert gamma == 0 or (0 < (ref["accept_len"] == gamma).sum() < w.B)
    if gamma:
        keep = np.zeros((w.B, gamma), bool)
        rej = ref["accept_len"] < gamma
        keep[np.nonzero(rej)[0], ref["accept_len"][rej]] = True
        d["draft_q"][~keep] = np.nan
    host = {k: torch.from_numpy(v).pin_memory() for k, v in d.items()}
    arena = torch.full((B.dssd_round_host_arena_bytes(w.B, w.gamma, w.V, B.DSSD_F32),), 0xFF, dtype=torch.uint8, device="cuda")
    out = B.dssd_round_host(host, w.temperature, arena)
    torch.cuda.synchronize()
    assert (out["accept_len"].numpy() == ref["accept_len"]).all()
    assert (out["token"].numpy() == ref["token"]).all()
    assert (out["rs_flags"].numpy().astype(np.uint32) == ref["rs_flags"]).all()
