"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, sizes its workspaces, and rejects bad arguments before touching CUDA."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2507_12000_b200 import build

    build.build()
    from paper_2507_12000_b200 import binding

    return binding


def _declared():
    """Every function that a header under include/ declares."""
    import glob

    names = set()
    for path in sorted(glob.glob(os.path.join(ROOT, "include", "*.h"))):
        src = re.sub(r"/\*.*?\*/", "", open(path).read(), flags=re.S)
        names.update(re.findall(r"\b(dssd_[a-z_0-9]+)\s*\(", src))
    return sorted(names)


def test_every_declared_symbol_is_exported(B):
    names = _declared()
    assert "dssd_edge_verify" in names and "dssd_device_resample" in names and "dssd_round_host" in names
    for n in names:
        assert hasattr(B.lib, n), n


def test_version_and_status_strings(B):
    assert B.lib.dssd_version() >= 100
    assert B.lib.dssd_status_string(0) == b"DSSD_OK"
    assert B.lib.dssd_status_string(3) == b"DSSD_ERR_WORKSPACE"
    assert B.lib.dssd_status_string(99) == b"DSSD_ERR_UNKNOWN"


def test_workspace_sizes(B):
    assert B.dssd_edge_verify_workspace_bytes(0, 4, 100) == 0
    assert B.dssd_edge_verify_workspace_bytes(1, -1, 100) == 0
    assert B.dssd_edge_verify_workspace_bytes(1, 4, 0) == 0
    a = B.dssd_edge_verify_workspace_bytes(1, 4, 1024)
    b = B.dssd_edge_verify_workspace_bytes(256, 4, 151936)
    c = B.dssd_edge_verify_workspace_bytes(1024, 16, 50272)
    assert 0 < a < b < c < 64 << 20 and a % 256 == 0
    r = B.dssd_device_resample_workspace_bytes(256, 4, 151936)
    assert 0 < r < 4 << 20
    assert B.dssd_edge_verify_topk_workspace_bytes(256, 4, 151936, 0) == 0
    assert B.dssd_edge_verify_topk_workspace_bytes(256, 4, 151936, 33) == 0
    assert B.dssd_edge_verify_topk_workspace_bytes(1, 0, 8, 9) == 0
    fused = B.dssd_dsd_verify_workspace_bytes(256, 4, 151936)
    assert fused >= b + r and fused % 256 == 0 and B.dssd_dsd_verify_workspace_bytes(0, 4, 100) == 0
    eb = B.dssd_edge_verify_bonus_workspace_bytes(256, 4, 151936)
    assert eb >= b + r and eb % 256 == 0 and B.dssd_edge_verify_bonus_workspace_bytes(1, 4, 0) == 0
    t = B.dssd_edge_verify_topk_workspace_bytes(256, 4, 151936, 10)
    assert 0 < t < 4 << 20 and t % 256 == 0
    assert B.dssd_round_host_arena_bytes(8, 4, 32000, B.DSSD_BF16) > 8 * 5 * 32000 * 2 + 8 * 4 * 32000 * 4
    assert B.dssd_round_host_arena_bytes(8, 4, 32000, 7) == 0


def test_bad_arguments_are_rejected_before_any_launch(B):
    L = B.lib
    buf = (ctypes.c_char * 4096)()
    p = ctypes.addressof(buf)
    p = (p + 255) & ~255  # any non-NULL, aligned address: it is never dereferenced on these paths
    f = ctypes.c_float
    ok_ws = 1 << 30

    def ev(logits=p, dtype=0, stride=16, tok=p, qt=p, u=p, T=1.0, Bn=1, g=2, V=16, n=p, prow=p, ws=p, wsb=ok_ws):
        return L.dssd_edge_verify(logits, dtype, stride, tok, qt, u, f(T), Bn, g, V, n, prow, None, None, None,
                                  ws, wsb, None)

    assert ev(logits=None) == B.DSSD_ERR_INVALID_ARG
    assert ev(n=None) == B.DSSD_ERR_INVALID_ARG
    assert ev(prow=None) == B.DSSD_ERR_INVALID_ARG
    assert ev(tok=None) == B.DSSD_ERR_INVALID_ARG
    assert ev(Bn=0) == B.DSSD_ERR_INVALID_ARG
    assert ev(g=-1) == B.DSSD_ERR_INVALID_ARG
    assert ev(V=0) == B.DSSD_ERR_INVALID_ARG
    assert ev(T=0.0) == B.DSSD_ERR_INVALID_ARG
    assert ev(T=-1.0) == B.DSSD_ERR_INVALID_ARG
    assert ev(T=float("inf")) == B.DSSD_ERR_INVALID_ARG
    assert ev(T=float("nan")) == B.DSSD_ERR_INVALID_ARG
    assert ev(stride=15) == B.DSSD_ERR_INVALID_ARG
    assert ev(dtype=5) == B.DSSD_ERR_UNSUPPORTED
    assert ev(V=(1 << 30) + 1, stride=(1 << 30) + 1) == B.DSSD_ERR_UNSUPPORTED
    assert ev(Bn=1 << 30, g=3) == B.DSSD_ERR_UNSUPPORTED
    assert ev(ws=None) == B.DSSD_ERR_WORKSPACE
    assert ev(ws=p + 8) == B.DSSD_ERR_WORKSPACE
    assert ev(wsb=16) == B.DSSD_ERR_WORKSPACE

    def rs(prow=p, q=p, n=p, u=p, Bn=1, g=2, V=16, tok=p, ws=p, wsb=ok_ws):
        return L.dssd_device_resample(prow, q, n, u, Bn, g, V, tok, None, ws, wsb, None)

    assert rs(prow=None) == B.DSSD_ERR_INVALID_ARG
    assert rs(q=None) == B.DSSD_ERR_INVALID_ARG
    assert rs(tok=None) == B.DSSD_ERR_INVALID_ARG
    assert rs(Bn=-3) == B.DSSD_ERR_INVALID_ARG
    assert rs(wsb=8) == B.DSSD_ERR_WORKSPACE
    assert rs(ws=None) == B.DSSD_ERR_WORKSPACE

    def evk(logits=p, dtype=0, stride=64, tok=p, qt=p, u=p, T=1.0, Bn=1, g=2, V=64, k=10, n=p, pi=p, pv=p, ws=p,
            wsb=ok_ws):
        return L.dssd_edge_verify_topk(logits, dtype, stride, tok, qt, u, f(T), Bn, g, V, k, n, pi, pv, None, None,
                                       ws, wsb, None)

    assert evk(logits=None) == B.DSSD_ERR_INVALID_ARG
    assert evk(pi=None) == B.DSSD_ERR_INVALID_ARG
    assert evk(pv=None) == B.DSSD_ERR_INVALID_ARG
    assert evk(u=None) == B.DSSD_ERR_INVALID_ARG
    assert evk(k=0) == B.DSSD_ERR_INVALID_ARG
    assert evk(k=20, V=16, stride=16) == B.DSSD_ERR_INVALID_ARG
    assert evk(k=33) == B.DSSD_ERR_UNSUPPORTED
    assert evk(T=0.0) == B.DSSD_ERR_INVALID_ARG
    assert evk(stride=63) == B.DSSD_ERR_INVALID_ARG
    assert evk(dtype=2) == B.DSSD_ERR_UNSUPPORTED
    assert evk(ws=None) == B.DSSD_ERR_WORKSPACE
    assert evk(wsb=8) == B.DSSD_ERR_WORKSPACE

    def rsk(pi=p, pv=p, qi=p, qv=p, n=p, u=p, Bn=1, g=2, k=10, tok=p):
        return L.dssd_device_resample_topk(pi, pv, qi, qv, n, u, Bn, g, k, tok, None, None)

    assert rsk(pi=None) == B.DSSD_ERR_INVALID_ARG
    assert rsk(qv=None) == B.DSSD_ERR_INVALID_ARG
    assert rsk(tok=None) == B.DSSD_ERR_INVALID_ARG
    assert rsk(Bn=0) == B.DSSD_ERR_INVALID_ARG
    assert rsk(k=0) == B.DSSD_ERR_INVALID_ARG
    assert rsk(k=33) == B.DSSD_ERR_UNSUPPORTED

    def p16(prow=p, **kw):
        return L.dssd_edge_verify_p16(p, 0, 16, p, p, p, f(1.0), 1, 2, 16, p, prow, None, None, None, p, kw.get("wsb", ok_ws),
                                      None)

    assert p16(prow=None) == B.DSSD_ERR_INVALID_ARG
    assert p16(prow=p + 1) == B.DSSD_ERR_INVALID_ARG
    assert p16(wsb=16) == B.DSSD_ERR_WORKSPACE
    assert L.dssd_device_resample_p16(None, p, p, p, 1, 2, 16, p, None, p, ok_ws, None) == B.DSSD_ERR_INVALID_ARG
    assert L.dssd_device_resample_p16(p + 1, p, p, p, 1, 2, 16, p, None, p, ok_ws, None) == B.DSSD_ERR_INVALID_ARG

    def dsd(logits=p, dtype=0, stride=16, q=p, tok=p, u=p, urs=p, T=1.0, Bn=1, g=2, V=16, n=p, token=p, ws=p,
            wsb=ok_ws):
        return L.dssd_dsd_verify(logits, dtype, stride, q, tok, u, urs, f(T), Bn, g, V, n, token, None, None, ws, wsb, None)

    assert dsd(logits=None) == B.DSSD_ERR_INVALID_ARG
    assert dsd(q=None) == B.DSSD_ERR_INVALID_ARG
    assert dsd(urs=None) == B.DSSD_ERR_INVALID_ARG
    assert dsd(token=None) == B.DSSD_ERR_INVALID_ARG
    assert dsd(T=0.0) == B.DSSD_ERR_INVALID_ARG
    assert dsd(stride=15) == B.DSSD_ERR_INVALID_ARG
    assert dsd(dtype=3) == B.DSSD_ERR_UNSUPPORTED
    assert dsd(ws=None) == B.DSSD_ERR_WORKSPACE
    assert dsd(wsb=64) == B.DSSD_ERR_WORKSPACE

    def evb(logits=p, dtype=0, stride=16, tok=p, qt=p, u=p, ub=p, T=1.0, Bn=1, g=2, V=16, n=p, prow=p, token=p, ws=p,
            wsb=ok_ws):
        return L.dssd_edge_verify_bonus(logits, dtype, stride, tok, qt, u, ub, f(T), Bn, g, V, n, prow, token, None, None,
                                        None, None, ws, wsb, None)

    assert evb(logits=None) == B.DSSD_ERR_INVALID_ARG
    assert evb(ub=None) == B.DSSD_ERR_INVALID_ARG
    assert evb(token=None) == B.DSSD_ERR_INVALID_ARG
    assert evb(prow=None) == B.DSSD_ERR_INVALID_ARG
    assert evb(qt=None) == B.DSSD_ERR_INVALID_ARG
    assert evb(T=0.0) == B.DSSD_ERR_INVALID_ARG
    assert evb(stride=15) == B.DSSD_ERR_INVALID_ARG
    assert evb(dtype=3) == B.DSSD_ERR_UNSUPPORTED
    assert evb(ws=None) == B.DSSD_ERR_WORKSPACE
    assert evb(wsb=B.dssd_edge_verify_workspace_bytes(1, 2, 16)) == B.DSSD_ERR_WORKSPACE  # the draw's scratch is missing
    assert L.dssd_device_resample_rejected(None, p, p, p, 1, 2, 16, p, None, p, ok_ws, None) == B.DSSD_ERR_INVALID_ARG
    assert L.dssd_device_resample_rejected(p, p, p, p, 1, 2, 16, None, None, p, ok_ws, None) == B.DSSD_ERR_INVALID_ARG
    assert L.dssd_device_resample_rejected(p, p, p, p, 1, 2, 16, p, None, p, 8, None) == B.DSSD_ERR_WORKSPACE

    assert L.dssd_round_host(None, 0, p, p, p, p, p, f(1.0), 1, 2, 16, p, p, None, None, None, p, ok_ws, None) \
        == B.DSSD_ERR_INVALID_ARG
    assert L.dssd_round_host(p, 0, p, p, p, p, p, f(1.0), 1, 2, 16, p, p, None, None, None, p, 64, None) \
        == B.DSSD_ERR_WORKSPACE
    assert L.dssd_last_cuda_error() == 0


def test_missing_library_fails_loudly(B, monkeypatch, tmp_path):
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(ImportError, match="no CPU fallback"):
        B._load()
