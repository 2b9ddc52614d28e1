"""The entry point that allocates nothing (dssd_device_resample_static).

Collected last on purpose: if it fails, a run that stops at the first failure has already been
through every other test.  It calls the library through the C ABI and compares with the regular
entry point and with the CPU oracle, on two calls in a row (they share the built-in scratch), at a
small size and at a size that fills the built-in scratch to within one percent, and checks that
the call itself takes no device memory.
"""
import numpy as np
import pytest
import torch

import dssd_inputs as di

pytestmark = pytest.mark.gpu

NEAR = 1e-6  # a draw closer than this to a CDF step may fall on either side


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


def _check_against_oracle(O, p_row, q, n, u, gamma, tok, flags, threads=8):
    """Tokens and flags of the CUDA path against the oracle's float64 draw on the same float32 arrays."""
    ref = O.device_resample(p_row.cpu().numpy(), q.cpu().numpy() if gamma else None, n.cpu().numpy(),
                            u.cpu().numpy(), gamma, threads=threads)
    near = ref["margin_cdf"] < NEAR
    bad = (tok != ref["token"]) & ~near
    assert not bad.any(), (np.nonzero(bad)[0][:8], tok[bad][:8], ref["token"][bad][:8])
    assert (flags.astype(np.uint32) == ref["flags"]).all()
    return int(near.sum())


def test_static_scratch_matches_the_regular_entry_point_and_the_oracle(oracle_mod):
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
        _check_against_oracle(oracle_mod, p_row, q, n, u, w.gamma, tok, out["flags"].cpu().numpy())


def test_a_batch_that_fills_the_built_in_scratch(oracle_mod):
    """B * ceil(V / 4096) chunk sums of 8 bytes each, plus 256 bytes of counters, must fit 1 MiB:
    65 000 sequences of 4097 entries need 99 % of it.  Two calls in a row, the second on other
    uniforms, each checked against the regular entry point and the oracle; the second call is
    made straight through the C ABI and must leave the device's free memory as it found it."""
    from paper_2507_12000_b200 import binding as B

    Bn, V, gamma = 65000, 4097, 1
    need = B.dssd_device_resample_workspace_bytes(Bn, gamma, V)
    assert 0.9 * B.STATIC_SCRATCH_BYTES <= need <= B.STATIC_SCRATCH_BYTES
    assert B.dssd_device_resample_workspace_bytes(Bn + 600, gamma, V) > B.STATIC_SCRATCH_BYTES
    g = torch.Generator(device="cuda").manual_seed(4097)
    p_row = torch.softmax(3.0 * torch.randn(Bn, V, generator=g, device="cuda", dtype=torch.float64), dim=-1).float()
    q = torch.softmax(3.0 * torch.randn(Bn, V, generator=g, device="cuda", dtype=torch.float64), dim=-1).float()
    q = q.view(Bn, gamma, V)
    n = (torch.arange(Bn, device="cuda", dtype=torch.int32) % 3 == 2).to(torch.int32)  # a third of the draws are bonus draws
    out = {"token": torch.full((Bn,), -7, dtype=torch.int32, device="cuda"),
           "flags": torch.full((Bn,), -7, dtype=torch.int32, device="cuda")}
    for call in range(2):
        u = torch.rand(Bn, generator=g, device="cuda", dtype=torch.float32).clamp_(max=1.0 - 2.0 ** -24)
        ref = B.dssd_device_resample(p_row, q, n, u, gamma)
        torch.cuda.synchronize()
        if call == 0:
            B.dssd_device_resample_static(p_row, q, n, u, gamma, out=out)
        else:
            free0, reserved0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_reserved()
            st = B.lib.dssd_device_resample_static(p_row.data_ptr(), q.data_ptr(), n.data_ptr(), u.data_ptr(),
                                                   Bn, gamma, V, out["token"].data_ptr(), out["flags"].data_ptr(), None)
            assert st == B.DSSD_OK
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info()[0] == free0 and torch.cuda.memory_reserved() == reserved0
        torch.cuda.synchronize()
        assert torch.equal(out["token"], ref["token"]), call
        assert torch.equal(out["flags"], ref["flags"]), call
        near = _check_against_oracle(oracle_mod, p_row, q, n, u, gamma, out["token"].cpu().numpy(),
                                     out["flags"].cpu().numpy())
        assert near < Bn // 100


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
