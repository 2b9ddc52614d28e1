"""The bounded waits inside the kernels, made to run out on purpose (failure detection without a
fault): one store that a wait depends on is withheld through the library's test hooks
(include/dssd_test_hooks.h), the wait gives up after a small number of polls, the kernel ends
normally, the affected sequence - and only that one - reports the timeout, and the next ordinary
call on the same workspace is correct again."""
import ctypes

import numpy as np
import pytest
import torch

import dssd_inputs as di
from gpu_util import to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2507_12000_b200 import binding

    assert torch.cuda.is_available()
    L = binding.lib
    c = ctypes
    L.dssd_test_edge_verify_wait_runs_out.restype = c.c_int
    L.dssd_test_edge_verify_wait_runs_out.argtypes = [
        c.c_void_p, c.c_int, c.c_int64, c.c_void_p, c.c_void_p, c.c_void_p, c.c_float, c.c_int, c.c_int, c.c_int,
        c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_size_t, c.c_longlong, c.c_uint, c.c_void_p]
    L.dssd_test_device_resample_wait_runs_out.restype = c.c_int
    L.dssd_test_device_resample_wait_runs_out.argtypes = [
        c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_int, c.c_int, c.c_int, c.c_void_p, c.c_void_p,
        c.c_void_p, c.c_size_t, c.c_int, c.c_uint, c.c_void_p]
    return binding


@pytest.mark.parametrize("dtype,Bn,gamma,V,drop_row", [("bf16", 200, 3, 9001, 417), ("f32", 40, 8, 70001, 0),
                                                        ("bf16", 7, 2, 300000, 20)])
def test_a_partial_sum_that_never_arrives(B, dtype, Bn, gamma, V, drop_row):
    w = di.custom(B=Bn, gamma=gamma, V=V, dtype=dtype, temperature=0.9, sigma_d=0.8, seed=V)
    g = to_device(di.generate(w, threads=4))
    tl = g["target_logits"]
    ws = torch.empty(B.dssd_edge_verify_workspace_bytes(Bn, gamma, V), dtype=torch.uint8, device="cuda")
    good = B.dssd_edge_verify(tl, g["draft_tokens"], g["draft_q_tok"], g["uniforms"], w.temperature, workspace=ws)
    torch.cuda.synchronize()
    n = torch.full((Bn,), -7, dtype=torch.int32, device="cuda")
    p_row = torch.full((Bn, V), -7.0, dtype=torch.float32, device="cuda")
    flags = torch.full((Bn,), -7, dtype=torch.int32, device="cuda")
    st = B.lib.dssd_test_edge_verify_wait_runs_out(
        tl.data_ptr(), B._dtype_code(tl), V, g["draft_tokens"].data_ptr(), g["draft_q_tok"].data_ptr(),
        g["uniforms"].data_ptr(), ctypes.c_float(w.temperature), Bn, gamma, V, n.data_ptr(), p_row.data_ptr(),
        flags.data_ptr(), ws.data_ptr(), ws.numel(), drop_row, 64, None)
    assert st == B.DSSD_OK
    torch.cuda.synchronize()  # the kernel ended by itself
    b = drop_row // (gamma + 1)
    others = torch.arange(Bn, device="cuda") != b
    assert int(n[b]) == -1 and (int(flags[b]) & B.EDGE_FLAG_TIMEOUT)
    assert (p_row[b] == -7.0).all()  # nothing was written for the sequence without a verdict
    assert torch.equal(n[others], good["accept_len"][others])
    assert torch.equal(flags[others], good["flags"][others])
    assert torch.equal(p_row[others], good["p_row"][others])
    # the context is intact and the next ordinary call on the same workspace is correct
    again = B.dssd_edge_verify(tl, g["draft_tokens"], g["draft_q_tok"], g["uniforms"], w.temperature, workspace=ws)
    torch.cuda.synchronize()
    for k in ("accept_len", "flags", "p_row", "p_tok", "lse"):
        assert torch.equal(again[k], good[k]), k


@pytest.mark.parametrize("Bn,gamma,V,drop_seq", [(300, 3, 20011, 123), (5, 2, 300001, 4), (2000, 1, 4097, 0)])
def test_a_chunk_sum_that_never_arrives(B, Bn, gamma, V, drop_seq):
    gen = torch.Generator(device="cuda").manual_seed(V)
    p = torch.softmax(3.0 * torch.randn(Bn, V, generator=gen, device="cuda"), dim=-1)
    q = torch.softmax(3.0 * torch.randn(Bn, gamma, V, generator=gen, device="cuda"), dim=-1)
    n = (torch.arange(Bn, device="cuda", dtype=torch.int32) % (gamma + 1)).to(torch.int32)
    u = torch.rand(Bn, generator=gen, device="cuda")
    ws = torch.empty(B.dssd_device_resample_workspace_bytes(Bn, gamma, V), dtype=torch.uint8, device="cuda")
    good = B.dssd_device_resample(p, q, n, u, gamma, workspace=ws)
    torch.cuda.synchronize()
    tok = torch.full((Bn,), -7, dtype=torch.int32, device="cuda")
    fl = torch.full((Bn,), -7, dtype=torch.int32, device="cuda")
    st = B.lib.dssd_test_device_resample_wait_runs_out(p.data_ptr(), q.data_ptr(), n.data_ptr(), u.data_ptr(), Bn, gamma, V,
                                                       tok.data_ptr(), fl.data_ptr(), ws.data_ptr(), ws.numel(),
                                                       drop_seq, 64, None)
    assert st == B.DSSD_OK
    torch.cuda.synchronize()
    others = torch.arange(Bn, device="cuda") != drop_seq
    assert int(tok[drop_seq]) == -1
    assert (int(fl[drop_seq]) & (B.RS_FLAG_TIMEOUT | B.RS_FLAG_INVALID)) == (B.RS_FLAG_TIMEOUT | B.RS_FLAG_INVALID)
    assert torch.equal(tok[others], good["token"][others]) and torch.equal(fl[others], good["flags"][others])
    again = B.dssd_device_resample(p, q, n, u, gamma, workspace=ws)
    torch.cuda.synchronize()
    assert torch.equal(again["token"], good["token"]) and torch.equal(again["flags"], good["flags"])


def test_the_hooks_refuse_bad_arguments(B):
    p = torch.zeros(4, 64, dtype=torch.float32, device="cuda")
    n = torch.zeros(4, dtype=torch.int32, device="cuda")
    u = torch.zeros(4, dtype=torch.float32, device="cuda")
    tok = torch.zeros(4, dtype=torch.int32, device="cuda")
    ws = torch.empty(B.dssd_device_resample_workspace_bytes(4, 0, 64), dtype=torch.uint8, device="cuda")
    st = B.lib.dssd_test_device_resample_wait_runs_out(p.data_ptr(), None, n.data_ptr(), u.data_ptr(), 4, 0, 64,
                                                       tok.data_ptr(), None, ws.data_ptr(), ws.numel(), 9, 64, None)
    assert st == B.DSSD_ERR_INVALID_ARG  # no such sequence
