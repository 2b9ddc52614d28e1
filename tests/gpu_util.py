"""Helpers of the GPU parity tests: upload generated inputs, run both sides, compare."""
from __future__ import annotations

from typing import Dict

import numpy as np
import torch

# tolerance of probabilities (p_row, p_tok): |gpu - oracle| <= ATOL + RTOL * |oracle|
RTOL = 1e-5
ATOL = 1e-7
# a decision is "near a boundary" when the oracle's margin is below this
NEAR = 1e-6


def to_device(d: Dict[str, np.ndarray]) -> Dict[str, torch.Tensor]:
    out = {}
    for k, v in d.items():
        if v.dtype == np.uint16:
            out[k] = torch.from_numpy(v.view(np.int16)).cuda().view(torch.bfloat16)
        else:
            out[k] = torch.from_numpy(v).cuda()
    return out


def prob_close(gpu: np.ndarray, ref: np.ndarray) -> np.ndarray:
    """Elementwise pass mask; NaN must match NaN."""
    gpu = gpu.astype(np.float64)
    ref = ref.astype(np.float64)
    both_nan = np.isnan(gpu) & np.isnan(ref)
    return both_nan | (np.abs(gpu - ref) <= ATOL + RTOL * np.abs(ref))


def compare_round(B, O, d: Dict[str, np.ndarray], T: float, threads: int = 8):
    """Run oracle and CUDA path on the same inputs; assert parity; return a small report."""
    gamma = d["target_logits"].shape[1] - 1
    ref = O.verify_round(d, T, threads=threads)
    g = to_device(d)
    ev = B.dssd_edge_verify(g["target_logits"], g["draft_tokens"], g["draft_q_tok"], g["uniforms"], T)
    torch.cuda.synchronize()
    n_gpu = ev["accept_len"].cpu().numpy()
    near_acc = ref["margin_acc"] < NEAR
    assert (ev["flags"].cpu().numpy().astype(np.uint32) == ref["flags"]).all()
    bad = (n_gpu != ref["accept_len"]) & ~near_acc
    assert not bad.any(), (np.nonzero(bad)[0][:8], n_gpu[bad][:8], ref["accept_len"][bad][:8])
    clean = ref["flags"] == 0
    lse = ev["lse"].cpu().numpy().astype(np.float64)
    assert (np.abs(lse - ref["lse"])[clean] <= 2e-6 * np.maximum(1.0, np.abs(ref["lse"][clean]))).all()
    if gamma:
        assert prob_close(ev["p_tok"].cpu().numpy(), ref["p_tok"]).all()
    same = (n_gpu == ref["accept_len"])
    p_gpu = ev["p_row"].cpu().numpy()
    okrow = prob_close(p_gpu[same], ref["p_row"][same])
    assert okrow.all(), np.argwhere(~okrow)[:8]
    # device half in isolation: identical float32 inputs on both sides
    p_ref = torch.from_numpy(ref["p_row"]).cuda()
    n_ref = torch.from_numpy(ref["accept_len"]).cuda()
    rs = B.dssd_device_resample(p_ref, g["draft_q"], n_ref, g["uniforms_rs"], gamma)
    torch.cuda.synchronize()
    tok_iso = rs["token"].cpu().numpy()
    near_cdf = ref["margin_cdf"] < NEAR
    bad = (tok_iso != ref["token"]) & ~near_cdf
    assert not bad.any(), (np.nonzero(bad)[0][:8], tok_iso[bad][:8], ref["token"][bad][:8])
    assert (rs["flags"].cpu().numpy().astype(np.uint32) == ref["rs_flags"]).all()
    # end to end: the device half consumes the CUDA path's own row
    rs2 = B.dssd_device_resample(ev["p_row"], g["draft_q"], ev["accept_len"], g["uniforms_rs"], gamma)
    torch.cuda.synchronize()
    tok_e2e = rs2["token"].cpu().numpy()
    # the row differs from the oracle's by up to RTOL, which moves CDF steps by up to about
    # RTOL / Z relative to Z: only such sequences may differ
    slack = np.maximum(NEAR, 2 * RTOL / np.maximum(ref["Z"], 1e-30))
    bad = (tok_e2e != ref["token"]) & same & ~(ref["margin_cdf"] < slack)
    assert not bad.any(), (np.nonzero(bad)[0][:8], tok_e2e[bad][:8], ref["token"][bad][:8])
    return {
        "near_acc": int(near_acc.sum()), "near_cdf": int(near_cdf.sum()),
        "mismatch_accept": int((n_gpu != ref["accept_len"]).sum()),
        "mismatch_token_iso": int((tok_iso != ref["token"]).sum()),
        "mismatch_token_e2e": int((tok_e2e != ref["token"]).sum()),
        "max_rel_p_row": float(np.nanmax(np.abs(p_gpu[same] - ref["p_row"][same]) /
                                         np.maximum(np.abs(ref["p_row"][same]), 1e-30) *
                                         (ref["p_row"][same] > 1e-6))) if same.any() else 0.0,
        "max_abs_lse": float(np.max(np.abs(lse - ref["lse"])[clean])) if clean.any() else 0.0,
        "accept_rate": float(ref["accept_len"].mean() / max(gamma, 1)),
    }
