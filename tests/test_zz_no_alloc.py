"""The entry point that allocates nothing (dssd_device_resample_static).

Collected last on purpose: if it fails, a run that stops at the first failure has already been
through every other test.  It calls the library through the C ABI and compares with the regular
entry point, which the parity tests check against the oracle.
"""
import ctypes

import numpy as np
import pytest
import torch

import dssd_inputs as di

pytestmark = pytest.mark.gpu


def _inputs(seed):
    """A batch with rejected and all-accepted sequences: p rows, the device's q rows, accepted lengths."""
    w = di.custom(B=12, gamma=3, V=20011, dtype="f32", temperature=0.9, sigma_d=0.9, seed=seed)
    d = di.generate(w)
    z = torch.from_numpy(d["target_logits"]).double() / w.temperature
    p_all = torch.softmax(z, dim=-1).float()
    n = torch.arange(w.B, dtype=torch.int32) % (w.gamma + 1)     # every position, incl. the bonus one
    p_row = p_all[torch.arange(w.B), n.long()].contiguous()
    return (w, p_row.cuda(), torch.from_numpy(d["draft_q"]).cuda(), n.cuda(),
            torch.from_numpy(d["uniforms_rs"]).cuda())


def test_static_scratch_matches_the_regular_entry_point():
    from paper_2507_12000_b200 import binding as B

    for call, seed in enumerate((11, 12)):  # two calls in a row share the built-in scratch
        w, p_row, q, n, u = _inputs(seed)
        ref = B.dssd_device_resample(p_row, q, n, u, w.gamma)
        out = {"token": torch.full((w.B,), -7, dtype=torch.int32, device="cuda"),
               "flags": torch.full((w.B,), -7, dtype=torch.int32, device="cuda")}
        B.dssd_device_resample_static(p_row, q, n, u, w.gamma, out=out)
        torch.cuda.synchronize()
        assert torch.equal(out["token"], ref["token"]), (call, out["token"], ref["token"])
        assert torch.equal(out["flags"], ref["flags"]), call
        tok = out["token"].cpu().numpy()
        assert ((tok >= 0) & (tok < w.V)).all()
        # bonus sequences (n == gamma) are flagged as such by both
        assert ((out["flags"].cpu().numpy() & B.RS_FLAG_BONUS) != 0).tolist() == (n.cpu().numpy() == w.gamma).tolist()


def test_sizes_beyond_the_built_in_scratch_are_refused():
    from paper_2507_12000_b200 import binding as B

    w, p_row, q, n, u = _inputs(13)
    big_B, big_V = 1 << 16, 1 << 20
    assert B.dssd_device_resample_workspace_bytes(big_B, w.gamma, big_V) > B.STATIC_SCRATCH_BYTES
    tok = torch.zeros(4, dtype=torch.int32, device="cuda")
    # refused on the host from the sizes alone, before any pointer is used or anything is enqueued
    st = B.lib.dssd_device_resample_static(p_row.data_ptr(), q.data_ptr(), n.data_ptr(), u.data_ptr(),
                                           big_B, w.gamma, big_V, tok.data_ptr(), None, None)
    assert st == B.DSSD_ERR_UNSUPPORTED
    assert B.lib.dssd_status_string(st) == b"DSSD_ERR_UNSUPPORTED"
    torch.cuda.synchronize()
    assert (tok == 0).all()
