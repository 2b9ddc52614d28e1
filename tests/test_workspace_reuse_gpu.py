"""The workspaces need no initialisation: every entry point must give the same results on a
workspace full of garbage, on one left behind by a larger problem, and when replayed from a CUDA graph."""
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
    return binding


def _round_dense(B, g, w, ws_e, ws_r, payload="f32"):
    ev = B.dssd_edge_verify(g["target_logits"], g["draft_tokens"], g["draft_q_tok"], g["uniforms"], w.temperature,
                            workspace=ws_e, payload=payload)
    rs = B.dssd_device_resample(ev["p_row"], g["draft_q"], ev["accept_len"], g["uniforms_rs"], w.gamma, workspace=ws_r)
    return {"n": ev["accept_len"], "p": ev["p_row"], "tok": rs["token"], "fl": ev["flags"], "rfl": rs["flags"]}


def _round_topk(B, g, w, ws, k=10):
    ev = B.dssd_edge_verify_topk(g["target_logits"], g["draft_tokens"], g["draft_q_tok"], g["uniforms"], w.temperature, k,
                                 workspace=ws)
    rs = B.dssd_device_resample_topk(ev["p_idx"], ev["p_val"], g["q_idx"], g["q_val"], ev["accept_len"], g["uniforms_rs"],
                                     w.gamma)
    return {"n": ev["accept_len"], "idx": ev["p_idx"], "val": ev["p_val"], "tok": rs["token"], "fl": ev["flags"]}


def _round_fused(B, g, w, ws):
    out = B.dssd_dsd_verify(g["target_logits"], g["draft_q"], g["draft_tokens"], g["uniforms"], g["uniforms_rs"],
                            w.temperature, workspace=ws)
    return {"n": out["accept_len"], "tok": out["token"], "fl": out["edge_flags"], "rfl": out["rs_flags"]}


def _round_sharded(B, g, w, ws_e, ws_r, G=3):
    """All G shards in turn on this GPU, every call on the caller's (garbage-filled) workspaces."""
    tl, dq = g["target_logits"], g["draft_q"]
    base, extra = divmod(w.V, G)
    bounds, v = [], 0
    for i in range(G):
        bounds.append((v, v + base + (1 if i < extra else 0)))
        v = bounds[-1][1]
    parts = [B.dssd_edge_partial(tl[:, :, a:b], g["draft_tokens"], a, w.temperature, workspace=ws_e) for a, b in bounds]
    ev = B.dssd_edge_combine(torch.stack([p["part_ref"] for p in parts]), torch.stack([p["part_sum"] for p in parts]),
                             torch.stack([p["tok_logit"] for p in parts]), g["draft_tokens"], g["draft_q_tok"],
                             g["uniforms"], w.temperature, w.V)
    p_row = torch.empty(w.B, w.V, dtype=torch.float32, device="cuda")
    for a, b in bounds:
        B.dssd_edge_emit_shard(tl[:, :, a:b], ev["accept_len"], ev["row_scale"], w.temperature, out=p_row[:, a:b])
    need = B.dssd_resample_shard_workspace_bytes(w.B, w.gamma, bounds[0][1] - bounds[0][0])
    chunks = [ws_r[i * ((need + 255) // 256 * 256):][:need] for i in range(G)]  # one piece of the scratch per shard
    masses = torch.stack([B.dssd_resample_shard_mass(p_row[:, a:b], dq[:, :, a:b], ev["accept_len"], w.gamma,
                                                     workspace=chunks[i])[0] for i, (a, b) in enumerate(bounds)])
    toks = torch.stack([B.dssd_resample_shard_draw(masses, i, a, p_row[:, a:b], dq[:, :, a:b], ev["accept_len"],
                                                   g["uniforms_rs"], w.gamma, chunks[i])["token"]
                        for i, (a, b) in enumerate(bounds)])
    return {"n": ev["accept_len"], "p": p_row, "tok": toks.max(dim=0).values, "fl": ev["flags"]}


def _same(a, b):
    for k in a:
        x, y = a[k], b[k]
        if x.is_floating_point():
            x, y = x.view(torch.int16 if x.element_size() == 2 else torch.int32), y.view(torch.int16 if y.element_size() == 2 else torch.int32)
        assert torch.equal(x, y), k


@pytest.mark.parametrize("shape", [(3, 2, 5000), (200, 3, 9001)])  # cluster kernel / streaming kernel
def test_garbage_and_stale_workspaces(B, shape):
    Bn, gamma, V = shape
    w = di.custom(B=Bn, gamma=gamma, V=V, dtype="bf16", temperature=0.9, sigma_d=0.6, seed=Bn)
    big = di.custom(B=Bn + 57, gamma=gamma + 2, V=V + 4099, dtype="bf16", temperature=0.9, sigma_d=0.6, seed=Bn + 1)
    g, gb = to_device(di.generate(w, threads=4)), to_device(di.generate(big, threads=4))
    gk, gbk = to_device(di.generate_topk(w, 10, threads=4)), to_device(di.generate_topk(big, 10, threads=4))

    def spaces(fill):
        n = max(B.dssd_dsd_verify_workspace_bytes(big.B, big.gamma, big.V),
                B.dssd_edge_verify_topk_workspace_bytes(big.B, big.gamma, big.V, 10))
        mk = (lambda: torch.randint(0, 256, (n,), dtype=torch.uint8, device="cuda")) if fill is None else \
             (lambda: torch.full((n,), fill, dtype=torch.uint8, device="cuda"))
        return mk(), mk()

    ref = None
    for fill in (0, 0xFF, 0x5A, None):
        ws1, ws2 = spaces(fill)
        cur = {"dense": _round_dense(B, g, w, ws1, ws2), "p16": _round_dense(B, g, w, ws1, ws2, payload="f16"),
               "topk": _round_topk(B, gk, w, ws1), "fused": _round_fused(B, g, w, ws1),
               "sharded": _round_sharded(B, g, w, ws1, ws2)}
        torch.cuda.synchronize()
        if ref is None:
            ref = cur
        else:
            for name in cur:
                _same(cur[name], ref[name])
    # the same workspaces after a larger problem went through them
    ws1, ws2 = spaces(0)
    _round_dense(B, gb, big, ws1, ws2)
    _round_topk(B, gbk, big, ws1)
    _round_fused(B, gb, big, ws1)
    cur = {"dense": _round_dense(B, g, w, ws1, ws2), "topk": _round_topk(B, gk, w, ws1), "fused": _round_fused(B, g, w, ws1)}
    torch.cuda.synchronize()
    for name in cur:
        _same(cur[name], ref[name])


def test_replay_from_a_cuda_graph(B):
    w = di.custom(B=160, gamma=3, V=12000, dtype="bf16", temperature=0.8, sigma_d=0.6, seed=77)
    g = to_device(di.generate(w, threads=4))
    gk = to_device(di.generate_topk(w, 10, threads=4))
    n = max(B.dssd_dsd_verify_workspace_bytes(w.B, w.gamma, w.V), B.dssd_edge_verify_topk_workspace_bytes(w.B, w.gamma, w.V, 10))
    ws1 = torch.empty(n, dtype=torch.uint8, device="cuda")
    ws2 = torch.empty_like(ws1)
    # first calls outside the capture: they look up device attributes once
    eager = {"dense": _round_dense(B, g, w, ws1, ws2), "topk": _round_topk(B, gk, w, ws1), "fused": _round_fused(B, g, w, ws1)}
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            captured = {"dense": _round_dense(B, g, w, ws1, ws2), "topk": _round_topk(B, gk, w, ws1),
                        "fused": _round_fused(B, g, w, ws1)}
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    for name in captured:
        _same(captured[name], eager[name])
