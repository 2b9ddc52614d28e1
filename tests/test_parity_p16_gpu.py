"""Parity of the 16-bit payload path (dssd_edge_verify_p16, dssd_device_resample_p16) with the oracle.

Tolerance of the row: the oracle rounds the float64 probability once to binary16; the kernel
computes it in float32 (relative error about 1e-6, see gpu_util.RTOL) and rounds that.  The two
agree except where the value sits within that error of a binary16 rounding boundary, where they
differ by one unit in the last place: bit patterns may differ by at most 1, and by 0 for at least
99 % of the entries.  The draw is compared exactly on identical 16-bit rows.
"""
import numpy as np
import pytest
import torch

import dssd_inputs as di
from gpu_util import NEAR, prob_close, to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2507_12000_b200 import binding

    assert torch.cuda.is_available()
    return binding


def compare_p16(B, O, d, T, logits_view=None, threads=4):
    gamma = d["target_logits"].shape[1] - 1
    ref = O.verify_round(d, T, threads=threads, payload="f16")
    g = to_device(d)
    tl = g["target_logits"] if logits_view is None else logits_view(g["target_logits"])
    ev = B.dssd_edge_verify(tl, g["draft_tokens"], g["draft_q_tok"], g["uniforms"], T, payload="f16")
    torch.cuda.synchronize()
    assert ev["p_row"].dtype == torch.float16
    n_gpu = ev["accept_len"].cpu().numpy()
    assert (ev["flags"].cpu().numpy().astype(np.uint32) == ref["flags"]).all()
    near = ref["margin_acc"] < NEAR
    assert ((n_gpu == ref["accept_len"]) | near).all()
    if gamma:
        assert prob_close(ev["p_tok"].cpu().numpy(), ref["p_tok"]).all()
    same = n_gpu == ref["accept_len"]
    clean = same & (ref["flags"] == 0)
    bits_gpu = ev["p_row"].cpu().numpy().view(np.uint16).astype(np.int32)[clean]
    bits_ref = ref["p_row16"].view(np.uint16).astype(np.int32)[clean]
    diff = np.abs(bits_gpu - bits_ref)
    assert diff.max(initial=0) <= 1, int(diff.max())
    if diff.size:
        assert (diff == 0).mean() >= 0.99, float((diff == 0).mean())
    # device half in isolation: the oracle's 16-bit row on both sides, exact up to CDF-step margins
    p_ref = torch.from_numpy(ref["p_row16"]).cuda()
    n_ref = torch.from_numpy(ref["accept_len"]).cuda()
    rs = B.dssd_device_resample(p_ref, g["draft_q"], n_ref, g["uniforms_rs"], gamma)
    torch.cuda.synchronize()
    tok = rs["token"].cpu().numpy()
    assert ((tok == ref["token"]) | (ref["margin_cdf"] < NEAR)).all()
    assert (rs["flags"].cpu().numpy().astype(np.uint32) == ref["rs_flags"]).all()
    # end to end on the CUDA path's own 16-bit row: one unit in the last place moves a CDF step by
    # up to 2^-11 of that entry
    rs2 = B.dssd_device_resample(ev["p_row"], g["draft_q"], ev["accept_len"], g["uniforms_rs"], gamma)
    torch.cuda.synchronize()
    tok2 = rs2["token"].cpu().numpy()
    slack = np.maximum(NEAR, 2.0 ** -10 / np.maximum(ref["Z"], 1e-30))
    assert ((tok2 == ref["token"]) | ~same | (ref["margin_cdf"] < slack)).all()
    return {"exact": float((diff == 0).mean()) if diff.size else 1.0, "token_mismatch": int((tok2 != ref["token"]).sum())}


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_small_vocabularies_both_kernels(B, oracle_mod, dtype):
    """Bn = 2 goes through the one-cluster-per-sequence kernel, Bn = 150 through the streaming kernel."""
    seed = 500
    for V in (1, 3, 7, 33, 1000, 1025, 16389):
        for gamma in (0, 3):
            for Bn in (2, 150):
                seed += 1
                w = di.custom(B=Bn, gamma=gamma, V=V, dtype=dtype, temperature=0.9, sigma_d=1.0, zipf=V > 8, seed=seed)
                compare_p16(B, oracle_mod, di.generate(w, threads=4), w.temperature)


@pytest.mark.parametrize("dtype,V,gamma,Bn", [
    ("f32", 50272, 2, 6), ("bf16", 40003, 3, 5), ("bf16", 128256, 8, 4), ("f32", 20001, 16, 3),
    ("bf16", 151936, 4, 9), ("f32", 16385, 1, 40),
])
def test_several_slices_and_ragged_tails(B, oracle_mod, dtype, V, gamma, Bn):
    w = di.custom(B=Bn, gamma=gamma, V=V, dtype=dtype, temperature=0.8, sigma_d=0.8, seed=V + gamma)
    compare_p16(B, oracle_mod, di.generate(w, threads=4), w.temperature)


@pytest.mark.parametrize("Bn", [3, 151])
def test_strided_and_unaligned_rows(B, oracle_mod, Bn):
    for dtype, V, off in (("f32", 1000, 1), ("bf16", 4097, 3), ("bf16", 20001, 1), ("f32", 9001, 2)):
        w = di.custom(B=Bn, gamma=2, V=V, dtype=dtype, seed=V)
        d = di.generate(w)
        stride = V + 5

        def view(t, stride=stride, off=off, Bn=Bn, V=V):
            buf = torch.zeros(Bn * 3 * stride + 16, dtype=t.dtype, device="cuda")
            v = buf[off:off + Bn * 3 * stride].view(Bn, 3, stride)[:, :, :V]
            v.copy_(t)
            assert v.data_ptr() % 16 != 0
            return v

        compare_p16(B, oracle_mod, d, w.temperature, logits_view=view)


def test_outputs_stay_inside_their_buffers(B):
    w = di.custom(B=5, gamma=3, V=12345, dtype="bf16", seed=3)
    g = to_device(di.generate(w))
    pad = 64
    full = torch.full((w.B * w.V + 2 * pad,), 7.0, dtype=torch.float16, device="cuda")
    out = {"accept_len": torch.empty(w.B, dtype=torch.int32, device="cuda"),
           "p_row": full[pad:pad + w.B * w.V].view(w.B, w.V),
           "flags": torch.empty(w.B, dtype=torch.int32, device="cuda"), "p_tok": None, "lse": None}
    B.dssd_edge_verify(g["target_logits"], g["draft_tokens"], g["draft_q_tok"], g["uniforms"], 1.0, out=out,
                       payload="f16")
    torch.cuda.synchronize()
    assert (full[:pad] == 7.0).all() and (full[-pad:] == 7.0).all()
    assert (out["p_row"].float().sum(dim=1) - 1.0).abs().max() < 2e-3


@pytest.mark.parametrize("name", ["c2", "c3", "c4"])
def test_named_configs(B, oracle_mod, name):
    w = di.get_workload(name)
    rep = compare_p16(B, oracle_mod, di.generate(w, threads=8), w.temperature, threads=8)
    print(name, rep)
