#!/usr/bin/env python
"""Benchmark of the split speculative verification round on B200.

One step = one pass of the whole verification round (dssd_edge_verify, then
dssd_device_resample) over one batch of synthetic inputs that are already resident in HBM.
The metric is verified rows per second, rows = B * (gamma + 1).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c4] [--impl ours|reference]

With N > 1 (launched through torch.distributed.run) every rank verifies its own batch of the
same shape (sequences are independent: no data-path collective); time is the maximum over ranks.
`--impl reference` times the CPU oracle on a bounded sample of the same workload instead.
`--sampler topk [--k 10]` runs the same round on distributions truncated to their k most likely
tokens (dssd_edge_verify_topk, dssd_device_resample_topk), the sampler of the paper's experiments.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import dssd_inputs as di  # noqa: E402

METRIC = "verified_rows_per_s"
UNIT = "rows/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0

# DRAM traffic of the dominant kernel from ncu (dram__bytes_read.sum + dram__bytes_write.sum,
# bytes per launch), valid only for the kernel source whose hash is recorded with it.
NCU_TRAFFIC = {
    # profiles/edge_verify_kernel_c4.md: 428.4 MB read (389.0 MB of logits + 51 % of the second read of row n)
    # and 96.6 MB written inside the kernel; the other 59.0 MB of p_row were still in L2 when the kernel ended
    # and reach DRAM after it.  "bytes" counts all of p_row.
    "c4": {"bytes": 428413440 + 155582464, "kernel_hash": "174f9e8708fc9d97",
           "note": "dram__bytes_read.sum 428.4 MB + all 155.6 MB of p_row (96.6 MB of it written inside the "
                   "kernel, the rest still in L2 at its end); reads are 1.10x the logits: the second read of "
                   "row n misses L2 for 51 % of its bytes",
           "counted_inside_kernel": 428413440 + 96619264},
}


# the same for topk_verify_kernel (k = 10)
NCU_TRAFFIC_TOPK = {
    # profiles/topk_verify_kernel_c4.md: 389.1 MB read + 3.4 MB written
    "c4": {"bytes": 389107968 + 3403264, "kernel_hash": "191879487eaaf336"},
}


def _kernel_hash_topk() -> str:
    h = hashlib.sha256()
    for f in ("topk_verify.cu", "topk_verify.h", "dssd_device.cuh"):
        with open(os.path.join(ROOT, "paper_2507_12000_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def _kernel_hash() -> str:
    h = hashlib.sha256()
    for f in ("edge_verify.cu", "edge_verify.h", "edge_judge.cuh", "dssd_device.cuh"):
        with open(os.path.join(ROOT, "paper_2507_12000_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return FALLBACK_HBM_GBS, "fallback"


def edge_algorithmic_bytes(w: di.Workload, payload_bytes: int = 4) -> int:
    """Bytes dssd_edge_verify must move: every logit once, plus the row it emits (4 or 2 bytes per value)."""
    return w.B * w.V * ((w.gamma + 1) * w.logit_bytes + payload_bytes)


def resample_algorithmic_bytes(w: di.Workload, n_bonus: int, payload_bytes: int = 4) -> int:
    """p row for every sequence, q row for the rejected ones, one token each."""
    return w.V * (payload_bytes * w.B + 4 * (w.B - n_bonus)) + 4 * w.B


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the benchmark runs."""

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.samples = []  # (t, sm_mhz, reasons bitmask, power_w)
        self.stop_flag = False
        self.max_mhz = None
        self.ok = False
        try:
            import pynvml

            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:  # NVML missing: report no clocks rather than fail the run
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        while not self.stop_flag:
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                reasons = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h) if hasattr(
                    nv, "nvmlDeviceGetCurrentClocksEventReasons") else nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                power = nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0
                self.samples.append((time.perf_counter(), mhz, int(reasons), power))
            except Exception:
                pass
            time.sleep(0.002)

    def summary(self, t0: float, t1: float):
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        scope = "timed region"
        if not inside:
            inside, scope = self.samples, "warm-up and timed region (timed region shorter than one sample)"
        names = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
                 0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown"}
        mask = 0
        for s in inside:
            mask |= s[2]
        return {"sm_mhz": statistics.median(s[1] for s in inside), "sm_max_mhz": self.max_mhz,
                "reasons": [n for b, n in names.items() if mask & b], "samples": len(inside),
                "power_w_max": max(s[3] for s in inside), "scope": scope}


def _torch_inputs(d, device=None, pin=False):
    import torch

    out = {}
    for k, v in d.items():
        t = torch.from_numpy(v.view(np.int16)).view(torch.bfloat16) if v.dtype == np.uint16 else torch.from_numpy(v)
        if device is not None:
            t = t.to(device)
        elif pin:
            t = t.pin_memory()
        out[k] = t
    return out


def oracle_rate(w: di.Workload, d, n_seq: int, threads: int, min_seconds: float = 1.5, payload: str = "f32",
                bonus: str = "device"):
    """rows/s of the CPU oracle (both halves) on the first n_seq sequences: whole passes are
    repeated until about `min_seconds` of wall time (some 10-30 s of CPU work on all cores) have gone."""
    from oracle import oracle as O

    sub = {k: v[:n_seq] for k, v in d.items()}
    passes = 0
    t0 = time.perf_counter()
    while True:
        if bonus == "edge":
            O.verify_round_bonus_at_edge(sub, w.temperature, threads=threads)
        else:
            O.verify_round(sub, w.temperature, threads=threads, payload=payload)
        passes += 1
        dt = time.perf_counter() - t0
        if dt >= min_seconds or passes >= 64:
            break
    return passes * n_seq * (w.gamma + 1) / dt, dt, passes


def run_reference(args, w: di.Workload):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return  # the oracle runs on rank 0's host cores alone; the other ranks leave at once
    from oracle import oracle as O

    O.build()
    cores = os.cpu_count() or 1
    n_seq = min(w.B, args.ref_sequences)
    d = di.generate(w, 0, n_seq, threads=cores)
    for _ in range(args.warmup):
        O.verify_round(d, w.temperature, threads=cores)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        O.verify_round(d, w.temperature, threads=cores)
    dt = time.perf_counter() - t0
    value = args.steps * n_seq * (w.gamma + 1) / dt
    sample = f"first {n_seq} of {w.B} sequences of {w.name} per step, both halves, float64"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": _config(w, args),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def _config(w: di.Workload, args):
    return {"workload": f"{w.name}: B={w.B} gamma={w.gamma} V={w.V} {w.dtype} T={w.temperature} "
                        f"sigma_d={w.sigma_d} (per GPU)",
            "B": w.B, "gamma": w.gamma, "V": w.V, "logits_dtype": w.dtype, "temperature": w.temperature,
            "l2": "inputs larger than L2, no flush" if w.rows * w.V * w.logit_bytes > 200e6 else
                  "inputs rotate through copies larger than L2",
            "parallelism": f"batch-sharded x{args.gpus}, no collective",
            "payload": getattr(args, "payload", "f32")}


MIN_TIMED_MS = 300.0  # device time the timed loops add up to at least


def timed_loops(one_loop, min_ms: float = None, max_loops: int = 400):
    """one_loop() times exactly K steps on the device and returns a dict with "total_ms" (already the
    maximum over ranks).  It is repeated until the loops add up to min_ms of device time, so that the
    clock samples and the average rest on more than a few milliseconds; the reported loop is the
    median one.  Returns (median loop, all loops)."""
    if min_ms is None:
        min_ms = MIN_TIMED_MS
    first = one_loop()
    n = int(min(max_loops, max(1, math.ceil(min_ms / max(first["total_ms"], 1e-3)))))
    loops = [first] + [one_loop() for _ in range(n - 1)]
    order = sorted(range(len(loops)), key=lambda i: loops[i]["total_ms"])
    return loops[order[len(order) // 2]], loops


def rank_workload(w: di.Workload, rank: int) -> di.Workload:
    """Weak scaling: every rank verifies its own batch of the same shape, drawn from its own seed."""
    return di.Workload(**{**w.__dict__, "seed": w.seed + 7919 * rank})


def max_over_ranks(value_ms: float, dist, device) -> float:
    """The job's time is the slowest rank's (device-timed) time."""
    import torch

    t = torch.tensor([value_ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def run_ours(args, w: di.Workload, light: bool = False):
    """The split round on workload w.  Returns the JSON line's dict on rank 0 (None elsewhere).
    light: a sub-record of another run: no end-to-end leg, a smaller CPU sample."""
    import torch
    import torch.distributed as dist

    from oracle import oracle as O

    O.build()  # before the first CUDA call
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    cores = os.cpu_count() or 1
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    from paper_2507_12000_b200 import binding as B

    wr = rank_workload(w, rank)
    d = di.generate(wr, threads=max(1, cores // max(1, min(world, 8))))
    logit_bytes = d["target_logits"].nbytes
    # inputs smaller than L2 rotate through enough copies to exceed it
    copies = 1 if logit_bytes > 200e6 else int(min(64, 300e6 // max(logit_bytes, 1) + 1))
    sets = [_torch_inputs(d, dev) for _ in range(copies)]
    gamma, Bn, V = w.gamma, w.B, w.V
    ws_e = torch.empty(B.dssd_edge_verify_workspace_bytes(Bn, gamma, V), dtype=torch.uint8, device=dev)
    ws_r = torch.empty(B.dssd_device_resample_workspace_bytes(Bn, gamma, V), dtype=torch.uint8, device=dev)
    ev_out = None
    rs_out = None
    bonus_edge = args.bonus == "edge"  # Algorithm 2 as printed: the edge draws the bonus token, rows go down after rejections only
    if bonus_edge:
        assert args.payload == "f32", "--bonus edge carries the float32 row"
        ws_e = torch.empty(B.dssd_edge_verify_bonus_workspace_bytes(Bn, gamma, V), dtype=torch.uint8, device=dev)

    def edge_call(g):
        nonlocal ev_out
        if bonus_edge:
            ev_out = B.dssd_edge_verify_bonus(g["target_logits"], g["draft_tokens"], g["draft_q_tok"], g["uniforms"],
                                              g["uniforms_rs"], w.temperature, out=ev_out, workspace=ws_e)
        else:
            ev_out = B.dssd_edge_verify(g["target_logits"], g["draft_tokens"], g["draft_q_tok"], g["uniforms"],
                                        w.temperature, out=ev_out, workspace=ws_e, payload=args.payload)

    def device_call(g):
        nonlocal rs_out
        if bonus_edge:
            rs_out = B.dssd_device_resample_rejected(ev_out["p_row"], g["draft_q"], ev_out["accept_len"], g["uniforms_rs"],
                                                     gamma, out={"token": ev_out["token"], "flags": ev_out["token_flags"]},
                                                     workspace=ws_r)
        else:
            rs_out = B.dssd_device_resample(ev_out["p_row"], g["draft_q"], ev_out["accept_len"], g["uniforms_rs"],
                                            gamma, out=rs_out, workspace=ws_r)

    def step(i):
        step_on(sets[i % copies])

    def step_on(g):
        edge_call(g)
        device_call(g)

    sampler = ClockSampler(local)
    sampler.start()
    for i in range(max(args.warmup, 3)):
        step(i)
    torch.cuda.synchronize()
    K = args.steps

    def one_loop():
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(K)]
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        for i in range(K):
            g = sets[i % copies]
            ev[i][0].record()
            edge_call(g)
            ev[i][1].record()
            device_call(g)
            ev[i][2].record()
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        total = ev[0][0].elapsed_time(ev[K - 1][2])
        if world > 1:
            total = max_over_ranks(total, dist, dev)
        return {"total_ms": total, "edge_ms": [e[0].elapsed_time(e[1]) for e in ev],
                "rs_ms": [e[1].elapsed_time(e[2]) for e in ev]}

    t_host0 = time.perf_counter()
    loop, loops = timed_loops(one_loop)
    t_host1 = time.perf_counter()
    total_ms, edge_ms, rs_ms = loop["total_ms"], loop["edge_ms"], loop["rs_ms"]
    sampler.stop_flag = True
    sampler.join(timeout=1.0)
    clocks = sampler.summary(t_host0, t_host1)
    n_gpu = ev_out["accept_len"].cpu().numpy()
    n_bonus = int((n_gpu == gamma).sum())

    # ---- the same K steps replayed from a CUDA graph (the calls allocate nothing and ask the host nothing,
    # so they capture as they are): what is left of a step once the host's launch work is off the path ----
    graph_rec = None
    if world == 1:
        side = torch.cuda.Stream()
        cg = torch.cuda.CUDAGraph()
        KG = min(K, 64)  # steps per graph (the rotation of input copies has at most 64 of them)
        with torch.cuda.stream(side):
            with torch.cuda.graph(cg, stream=side):
                for i in range(KG):
                    step(i)
        torch.cuda.synchronize()
        cg.replay()
        torch.cuda.synchronize()
        replays = max(3, int(math.ceil(MIN_TIMED_MS / 4 / max(total_ms * KG / K, 1e-3))))
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record()
        for _ in range(replays):
            cg.replay()
        g1.record()
        torch.cuda.synchronize()
        g_ms = g0.elapsed_time(g1) / (replays * KG)
        graph_rec = {"ms_per_step": g_ms, "value": w.rows / (g_ms * 1e-3), "unit": UNIT, "steps_per_graph": KG,
                     "replays": replays}
        assert (ev_out["accept_len"].cpu().numpy() == n_gpu).all()

    # ---- end to end through the host-buffer entry point: copies inside the timed region ----
    e2e = None
    if not light:
        host = _torch_inputs(d, pin=True)
        e2e_steps = max(3, min(K, args.e2e_steps))
        if args.payload == "f32" and not bonus_edge:
            arena = torch.empty(B.dssd_round_host_arena_bytes(Bn, gamma, V, B.DSSD_BF16 if w.dtype == "bf16" else B.DSSD_F32),
                                dtype=torch.uint8, device=dev)
            h_out = None

            def e2e_step():
                nonlocal h_out
                h_out = B.dssd_round_host(host, w.temperature, arena, out=h_out)
        else:
            # the host-buffer entry point carries the float32 row only: copy, call, copy back by hand
            names = ("target_logits", "draft_tokens", "draft_q_tok", "uniforms", "draft_q", "uniforms_rs")
            stage = {n: torch.empty_like(sets[0][n]) for n in names}
            h_out = {"accept_len": torch.empty(Bn, dtype=torch.int32).pin_memory(),
                     "token": torch.empty(Bn, dtype=torch.int32).pin_memory()}

            def e2e_step():
                for n in names:
                    stage[n].copy_(host[n], non_blocking=True)
                step_on(stage)
                h_out["accept_len"].copy_(ev_out["accept_len"], non_blocking=True)
                h_out["token"].copy_(rs_out["token"], non_blocking=True)

        for _ in range(2):
            e2e_step()
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(e2e_steps):
            e2e_step()
        e1.record()
        torch.cuda.synchronize()
        e2e_ms = e0.elapsed_time(e1)
        if world > 1:
            e2e_ms = max_over_ranks(e2e_ms, dist, dev)
        h2d = sum(host[k].numel() * host[k].element_size() for k in
                  ("target_logits", "draft_tokens", "draft_q_tok", "uniforms", "draft_q", "uniforms_rs"))
        if args.payload == "f32" and not bonus_edge:
            # dssd_round_host uploads of draft_q only the rows Q_n of the sequences with a rejection
            h2d -= host["draft_q"].numel() * 4
            h2d += int((n_gpu < gamma).sum()) * V * 4
        d2h = (4 if args.payload == "f32" and not bonus_edge else 2) * Bn * 4
        assert (h_out["accept_len"].numpy() == n_gpu).all()
        e2e = {"value": world * w.rows / (e2e_ms / e2e_steps * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    rows = w.rows
    ms_per_step = total_ms / K
    value = world * rows / (ms_per_step * 1e-3)
    peak, peak_kind = _peaks()
    edge_avg_ms = sum(edge_ms) / K
    pbytes = 4 if args.payload == "f32" else 2
    edge_bytes = edge_algorithmic_bytes(w, pbytes)
    if bonus_edge:  # every logit once, a row written per rejected sequence; row gamma's second read is not counted
        edge_bytes = w.rows * V * w.logit_bytes + (Bn - n_bonus) * V * 4
    achieved = edge_bytes / (edge_avg_ms * 1e-3) / 1e9
    traffic = NCU_TRAFFIC.get(w.name) if args.payload == "f32" and not bonus_edge else None
    if traffic is not None and traffic.get("kernel_hash") != _kernel_hash():
        traffic = None
    rs_avg_ms = sum(rs_ms) / K
    rs_bytes = resample_algorithmic_bytes(w, n_bonus, pbytes)
    if bonus_edge:  # p and q rows of the rejected sequences only
        rs_bytes = (Bn - n_bonus) * (8 * V + 4)

    # ---- CPU baseline: the oracle as it stands, on this machine's host cores, rank 0, N = 1 ----
    cpu = None
    alpha_hat = None
    if world == 1 and not args.no_cpu_baseline:
        from oracle import closed_forms as cf

        n_seq = min(Bn, args.ref_sequences if not light else min(args.ref_sequences, 64))
        rate, secs, passes = oracle_rate(w, d, n_seq, cores, min_seconds=0.5 if light else 1.5, payload=args.payload,
                                         bonus=args.bonus)
        n_one = max(1, min(n_seq, 8))
        rate1, secs1, passes1 = oracle_rate(w, d, n_one, 1, min_seconds=0.5 if light else 1.0, payload=args.payload,
                                            bonus=args.bonus)
        cpu = {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"first {n_seq} of {Bn} sequences of {w.name}, both halves, {passes} passes in {secs:.2f} s "
                         f"wall on {cores} threads",
               "one_core": {"value": rate1, "unit": UNIT, "cores": 1,
                            "sample": f"first {n_one} sequences, {passes1} passes in {secs1:.2f} s wall on 1 thread"}}
        sub = {k: v[:n_seq] for k, v in d.items()}
        ref = (O.verify_round_bonus_at_edge(sub, w.temperature, threads=cores) if bonus_edge else
               O.verify_round(sub, w.temperature, threads=cores, payload=args.payload))
        near = ref["margin_acc"] < 1e-6
        same = n_gpu[:n_seq] == ref["accept_len"]
        # the CUDA path's row is within 1e-5 relative of the oracle's, which moves a CDF step by up to about
        # 2e-5 / Z relative to Z: draws closer than that to a step may fall on either side
        slack = np.maximum(1e-6, 2e-5 / np.maximum(ref["Z"], 1e-30))
        near_cdf = ref["margin_cdf"] < slack
        tok_gpu = rs_out["token"].cpu().numpy()[:n_seq]
        alpha_hat = cf.batch_acceptance_rate(d["target_logits"], d["draft_q"], w.temperature, min(n_seq, 32))
        parity = {"sequences_checked": n_seq,
                  "accept_len_mismatch": int(((n_gpu[:n_seq] != ref["accept_len"]) & ~near).sum()),
                  "near_boundary_accept": int(near.sum()),
                  "token_mismatch": int(((tok_gpu != ref["token"]) & same & ~near_cdf).sum()),
                  "near_boundary_cdf": int((near_cdf & same).sum()),
                  "token_differs_near_boundary": int(((tok_gpu != ref["token"]) & same & near_cdf).sum()),
                  "mean_accept_len_over_gamma": float(ref["accept_len"].mean() / max(gamma, 1)),
                  "alpha_hat": alpha_hat}
    else:
        parity = None

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic", "config": _config(w, args),
        "roofline": {"bound": "hbm", "kernel": "edge_verify_kernel", "achieved": achieved, "peak": peak,
                     "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                     "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                     "algorithmic_bytes_per_launch": edge_bytes, "avg_launch_ms": edge_avg_ms,
                     "min_launch_ms": min(edge_ms),
                     "traffic": None if traffic is None else traffic["bytes"],
                     "traffic_note": None if traffic is None else traffic.get("note"),
                     "traffic_counted_inside_kernel": None if traffic is None else traffic.get("counted_inside_kernel")},
        "resample": {"avg_launch_ms": rs_avg_ms, "algorithmic_bytes_per_launch": rs_bytes,
                     "achieved_gbs": rs_bytes / (rs_avg_ms * 1e-3) / 1e9,
                     "frac": rs_bytes / (rs_avg_ms * 1e-3) / 1e9 / peak,
                     "note": "algorithmic bytes / time; part of p_row is still in L2 from the edge call, so this "
                             "is not a pure HBM fraction"},
        "edge_rows_per_s": world * rows / (edge_avg_ms * 1e-3),
        "timed": {"loops": len(loops), "device_ms": sum(lp["total_ms"] for lp in loops),
                  "loop_ms_min": min(lp["total_ms"] for lp in loops), "loop_ms_max": max(lp["total_ms"] for lp in loops),
                  "reported": "median loop"},
        "graph": graph_rec,
        "cpu_baseline": cpu,
        "parity": parity,
        "e2e": e2e,
        "gpu_launches": (3 if bonus_edge else 2) * K * len(loops),
        "clocks": clocks,
    }
    if bonus_edge:
        line["config"]["workload"] = line["config"]["workload"].replace(
            f"{w.name}:", f"{w.name}, bonus token drawn at the edge (Algorithm 2 as printed):")
        line["config"]["fully_accepted_sequences"] = n_bonus
        line["roofline"]["kernel"] = "edge_verify_kernel + resample_kernel<RowLogits> (dssd_edge_verify_bonus)"
    if world > 1:
        dist.destroy_process_group()
    return line


def topk_algorithmic_bytes(w: di.Workload) -> int:
    """Bytes dssd_edge_verify_topk must move: every logit once (its outputs are k pairs per sequence)."""
    return w.rows * w.V * w.logit_bytes


def _config_topk(w: di.Workload, args):
    c = _config(w, args)
    c["workload"] = c["workload"].replace(f"{w.name}:", f"{w.name} with top-k sampling, k={args.k}:")
    c["k"] = args.k
    return c


def run_reference_topk(args, w: di.Workload):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from oracle import oracle as O

    O.build()
    cores = os.cpu_count() or 1
    n_seq = min(w.B, args.ref_sequences)
    d = di.generate_topk(w, args.k, 0, n_seq, threads=cores)
    for _ in range(args.warmup):
        O.verify_round_topk(d, w.temperature, args.k, threads=cores)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        O.verify_round_topk(d, w.temperature, args.k, threads=cores)
    dt = time.perf_counter() - t0
    value = args.steps * n_seq * (w.gamma + 1) / dt
    sample = f"first {n_seq} of {w.B} sequences of {w.name} per step, k={args.k}, both halves, float64"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": _config_topk(w, args),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def run_ours_topk(args, w: di.Workload):
    import torch
    import torch.distributed as dist

    from oracle import oracle as O

    O.build()  # before the first CUDA call
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    cores = os.cpu_count() or 1
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    from paper_2507_12000_b200 import binding as B

    k = args.k
    wr = rank_workload(w, rank)
    d = di.generate_topk(wr, k, threads=max(1, cores // max(1, min(world, 8))))
    logit_bytes = d["target_logits"].nbytes
    copies = 1 if logit_bytes > 200e6 else int(min(64, 300e6 // max(logit_bytes, 1) + 1))
    sets = [_torch_inputs(d, dev) for _ in range(copies)]
    gamma, Bn, V = w.gamma, w.B, w.V
    ws = torch.empty(B.dssd_edge_verify_topk_workspace_bytes(Bn, gamma, V, k), dtype=torch.uint8, device=dev)
    ev_out = None
    rs_out = None

    def step(g):
        nonlocal ev_out, rs_out
        ev_out = B.dssd_edge_verify_topk(g["target_logits"], g["draft_tokens"], g["draft_q_tok"], g["uniforms"],
                                         w.temperature, k, out=ev_out, workspace=ws)
        rs_out = B.dssd_device_resample_topk(ev_out["p_idx"], ev_out["p_val"], g["q_idx"], g["q_val"],
                                             ev_out["accept_len"], g["uniforms_rs"], gamma, out=rs_out)

    sampler = ClockSampler(local)
    sampler.start()
    for i in range(max(args.warmup, 3)):
        step(sets[i % copies])
    torch.cuda.synchronize()
    K = args.steps

    def one_loop():
        nonlocal ev_out, rs_out
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(K)]
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        for i in range(K):
            g = sets[i % copies]
            ev[i][0].record()
            ev_out = B.dssd_edge_verify_topk(g["target_logits"], g["draft_tokens"], g["draft_q_tok"], g["uniforms"],
                                             w.temperature, k, out=ev_out, workspace=ws)
            ev[i][1].record()
            rs_out = B.dssd_device_resample_topk(ev_out["p_idx"], ev_out["p_val"], g["q_idx"], g["q_val"],
                                                 ev_out["accept_len"], g["uniforms_rs"], gamma, out=rs_out)
            ev[i][2].record()
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        total = ev[0][0].elapsed_time(ev[K - 1][2])
        if world > 1:
            total = max_over_ranks(total, dist, dev)
        return {"total_ms": total, "edge_ms": [e[0].elapsed_time(e[1]) for e in ev],
                "rs_ms": [e[1].elapsed_time(e[2]) for e in ev]}

    t_host0 = time.perf_counter()
    loop, loops = timed_loops(one_loop)
    t_host1 = time.perf_counter()
    total_ms, edge_ms, rs_ms = loop["total_ms"], loop["edge_ms"], loop["rs_ms"]
    sampler.stop_flag = True
    sampler.join(timeout=1.0)
    clocks = sampler.summary(t_host0, t_host1)
    n_gpu = ev_out["accept_len"].cpu().numpy()
    tok_gpu = rs_out["token"].cpu().numpy()

    # ---- end to end through the host-buffer entry point: inputs start in pinned host memory, the
    # results end there; the copies are inside the call and inside the timed region ----
    host = _torch_inputs(d, pin=True)
    names = ("target_logits", "draft_tokens", "draft_q_tok", "uniforms", "q_idx", "q_val", "uniforms_rs")
    arena = torch.empty(B.dssd_round_host_topk_arena_bytes(Bn, gamma, V, k, B.DSSD_BF16 if w.dtype == "bf16" else B.DSSD_F32),
                        dtype=torch.uint8, device=dev)
    h_out = None

    def e2e_step():
        nonlocal h_out
        h_out = B.dssd_round_host_topk(host, w.temperature, k, arena, out=h_out)

    e2e_steps = max(3, min(K, args.e2e_steps))
    for _ in range(2):
        e2e_step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        e2e_step()
    e1.record()
    torch.cuda.synchronize()
    e2e_ms = e0.elapsed_time(e1)
    if world > 1:
        e2e_ms = max_over_ranks(e2e_ms, dist, dev)
    h2d = sum(host[n].numel() * host[n].element_size() for n in names)
    d2h = 4 * Bn * 4
    assert (h_out["accept_len"].numpy() == n_gpu).all() and (h_out["token"].numpy() == tok_gpu).all()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    rows = w.rows
    ms_per_step = total_ms / K
    peak, peak_kind = _peaks()
    edge_avg_ms = sum(edge_ms) / K
    edge_bytes = topk_algorithmic_bytes(w)
    achieved = edge_bytes / (edge_avg_ms * 1e-3) / 1e9
    cpu = None
    parity = None
    if world == 1 and not args.no_cpu_baseline:
        n_seq = min(Bn, args.ref_sequences)
        sub = {kk: v[:n_seq] for kk, v in d.items()}
        passes, t0 = 0, time.perf_counter()
        while True:
            ref = O.verify_round_topk(sub, w.temperature, k, threads=cores)
            passes += 1
            dt = time.perf_counter() - t0
            if dt >= 1.5 or passes >= 64:
                break
        cpu = {"value": passes * n_seq * (gamma + 1) / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"first {n_seq} of {Bn} sequences of {w.name}, k={k}, both halves, {passes} passes in "
                         f"{dt:.2f} s wall on {cores} threads"}
        edge = ref["margin_acc"] < 1e-12
        parity = {"sequences_checked": n_seq,
                  "accept_len_mismatch": int(((n_gpu[:n_seq] != ref["accept_len"]) & ~edge).sum()),
                  "support_mismatch": int((ev_out["p_idx"].cpu().numpy()[:n_seq] != ref["p_idx"]).any(axis=1).sum()),
                  "token_mismatch": int((tok_gpu[:n_seq] != ref["token"]).sum()),
                  "accept_rate": float(ref["accept_len"].mean() / max(gamma, 1))}
    line = {
        "metric": METRIC, "value": world * rows / (ms_per_step * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": _config_topk(w, args),
        "roofline": {"bound": "hbm", "kernel": "topk_verify_kernel", "achieved": achieved, "peak": peak,
                     "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                     "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                     "algorithmic_bytes_per_launch": edge_bytes, "avg_launch_ms": edge_avg_ms,
                     "min_launch_ms": min(edge_ms), "traffic": NCU_TRAFFIC_TOPK.get(w.name, {}).get("bytes")
                     if NCU_TRAFFIC_TOPK.get(w.name, {}).get("kernel_hash") == _kernel_hash_topk() else None},
        "resample": {"avg_launch_ms": sum(rs_ms) / K},
        "edge_rows_per_s": world * rows / (edge_avg_ms * 1e-3),
        "cpu_baseline": cpu,
        "parity": parity,
        "e2e": {"value": world * rows / (e2e_ms / e2e_steps * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps},
        "timed": {"loops": len(loops), "device_ms": sum(lp["total_ms"] for lp in loops), "reported": "median loop"},
        "gpu_launches": 2 * K * len(loops),
        "clocks": clocks,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_ours_fused(args, w: di.Workload):
    """One step = one dssd_dsd_verify call (Algorithm 1: acceptance tests and the draw at the edge,
    no row P_n in memory)."""
    import torch
    import torch.distributed as dist

    from oracle import oracle as O

    O.build()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    cores = os.cpu_count() or 1
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    from paper_2507_12000_b200 import binding as B

    wr = rank_workload(w, rank)
    d = di.generate(wr, threads=max(1, cores // max(1, min(world, 8))))
    logit_bytes = d["target_logits"].nbytes
    copies = 1 if logit_bytes > 200e6 else int(min(64, 300e6 // max(logit_bytes, 1) + 1))
    sets = [_torch_inputs(d, dev) for _ in range(copies)]
    gamma, Bn, V = w.gamma, w.B, w.V
    ws = torch.empty(B.dssd_dsd_verify_workspace_bytes(Bn, gamma, V), dtype=torch.uint8, device=dev)
    out = None

    def step(g):
        nonlocal out
        out = B.dssd_dsd_verify(g["target_logits"], g["draft_q"], g["draft_tokens"], g["uniforms"], g["uniforms_rs"],
                                w.temperature, out=out, workspace=ws)

    sampler = ClockSampler(local)
    sampler.start()
    for i in range(max(args.warmup, 3)):
        step(sets[i % copies])
    torch.cuda.synchronize()
    K = args.steps

    def one_loop():
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(K + 1)]
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        ev[0].record()
        for i in range(K):
            step(sets[i % copies])
            ev[i + 1].record()
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        total = ev[0].elapsed_time(ev[K])
        if world > 1:
            total = max_over_ranks(total, dist, dev)
        return {"total_ms": total, "call_ms": [ev[i].elapsed_time(ev[i + 1]) for i in range(K)]}

    t_host0 = time.perf_counter()
    loop, loops = timed_loops(one_loop)
    t_host1 = time.perf_counter()
    total_ms, call_ms = loop["total_ms"], loop["call_ms"]
    sampler.stop_flag = True
    sampler.join(timeout=1.0)
    clocks = sampler.summary(t_host0, t_host1)
    n_gpu = out["accept_len"].cpu().numpy()
    tok_gpu = out["token"].cpu().numpy()
    n_bonus = int((n_gpu == gamma).sum())

    host = _torch_inputs(d, pin=True)
    names = ("target_logits", "draft_tokens", "uniforms", "draft_q", "uniforms_rs")
    stage = {n: torch.empty_like(sets[0][n]) for n in names}
    h_n = torch.empty(Bn, dtype=torch.int32).pin_memory()
    h_tok = torch.empty(Bn, dtype=torch.int32).pin_memory()

    def e2e_step():
        for n in names:
            stage[n].copy_(host[n], non_blocking=True)
        step(stage)
        h_n.copy_(out["accept_len"], non_blocking=True)
        h_tok.copy_(out["token"], non_blocking=True)

    e2e_steps = max(3, min(K, args.e2e_steps))
    for _ in range(2):
        e2e_step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        e2e_step()
    e1.record()
    torch.cuda.synchronize()
    e2e_ms = e0.elapsed_time(e1)
    if world > 1:
        e2e_ms = max_over_ranks(e2e_ms, dist, dev)
    h2d = sum(host[n].numel() * host[n].element_size() for n in names)
    assert (h_n.numpy() == n_gpu).all() and (h_tok.numpy() == tok_gpu).all()
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    rows = w.rows
    ms_per_step = total_ms / K
    peak, peak_kind = _peaks()
    # every logit once and the draft row of every rejected sequence (the second read of row n for the draw
    # is the implementation's, not the method's, and is not counted)
    call_bytes = rows * V * w.logit_bytes + 4 * V * (Bn - n_bonus)
    avg_ms = sum(call_ms) / K
    achieved = call_bytes / (avg_ms * 1e-3) / 1e9
    cpu = None
    parity = None
    if world == 1 and not args.no_cpu_baseline:
        n_seq = min(Bn, args.ref_sequences)
        sub = {kk: v[:n_seq] for kk, v in d.items()}
        passes, t0 = 0, time.perf_counter()
        while True:
            ref = O.dsd_verify(sub, w.temperature, threads=cores)
            passes += 1
            dt = time.perf_counter() - t0
            if dt >= 1.5 or passes >= 64:
                break
        cpu = {"value": passes * n_seq * (gamma + 1) / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"first {n_seq} of {Bn} sequences of {w.name}, Algorithm 1, {passes} passes in {dt:.2f} s wall "
                         f"on {cores} threads"}
        near = ref["margin_acc"] < 1e-6
        same = n_gpu[:n_seq] == ref["accept_len"]
        near_cdf = ref["margin_cdf"] < np.maximum(1e-6, 2e-5 / np.maximum(ref["Z"], 1e-30))
        parity = {"sequences_checked": n_seq,
                  "accept_len_mismatch": int(((n_gpu[:n_seq] != ref["accept_len"]) & ~near).sum()),
                  "near_boundary_accept": int(near.sum()),
                  "token_mismatch": int(((tok_gpu[:n_seq] != ref["token"]) & same & ~near_cdf).sum()),
                  "near_boundary_cdf": int((near_cdf & same).sum()),
                  "token_differs_near_boundary": int(((tok_gpu[:n_seq] != ref["token"]) & same & near_cdf).sum()),
                  "mean_accept_len_over_gamma": float(ref["accept_len"].mean() / max(gamma, 1))}
    cfg = _config(w, args)
    cfg["workload"] = cfg["workload"].replace(f"{w.name}:", f"{w.name}, fused verification of Algorithm 1:")
    print(json.dumps({
        "metric": METRIC, "value": world * rows / (ms_per_step * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": cfg,
        "roofline": {"bound": "hbm", "kernel": "edge_verify_kernel + resample_kernel (one call)", "achieved": achieved,
                     "peak": peak, "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                     "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS, "algorithmic_bytes_per_launch": call_bytes,
                     "avg_launch_ms": avg_ms, "min_launch_ms": min(call_ms), "traffic": None},
        "cpu_baseline": cpu, "parity": parity,
        "e2e": {"value": world * rows / (e2e_ms / e2e_steps * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": 2 * Bn * 4, "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps},
        "timed": {"loops": len(loops), "device_ms": sum(lp["total_ms"] for lp in loops), "reported": "median loop"},
        "gpu_launches": 2 * K * len(loops), "clocks": clocks,
    }))
    if world > 1:
        dist.destroy_process_group()


def shard_bounds(V: int, G: int):
    """G contiguous slices of [0, V), lengths differing by at most one (the slices of a tensor-parallel LM head)."""
    base, extra = divmod(V, G)
    out, v = [], 0
    for g in range(G):
        n = base + (1 if g < extra else 0)
        out.append((v, v + n))
        v += n
    return out


def run_ours_sharded(args, w: di.Workload):
    """The vocabulary-sharded round as ONE of G shards sees it: one step = that shard's five calls
    (partial sums, combine, its slice of row P_n, its masses, the draw) on its slice of the logits.  The
    other shards' partial sums and masses, which a real job receives through two all-gathers of a few
    bytes per row, are computed beforehand on the same GPU; the exchanges themselves are not timed."""
    import torch

    from oracle import oracle as O

    O.build()
    cores = os.cpu_count() or 1
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    from paper_2507_12000_b200 import binding as B

    G = args.shards
    d = di.generate(w, threads=cores)
    g = _torch_inputs(d, dev)
    gamma, Bn, V = w.gamma, w.B, w.V
    bounds = shard_bounds(V, G)
    tl, dq = g["target_logits"], g["draft_q"]
    T = w.temperature
    # every shard once, to have what the exchanges would deliver and the whole round's result
    parts = [B.dssd_edge_partial(tl[:, :, a:b], g["draft_tokens"], a, T) for a, b in bounds]
    ref_all = torch.stack([p["part_ref"] for p in parts])
    sum_all = torch.stack([p["part_sum"] for p in parts])
    tok_all = torch.stack([p["tok_logit"] for p in parts])
    ev = B.dssd_edge_combine(ref_all, sum_all, tok_all, g["draft_tokens"], g["draft_q_tok"], g["uniforms"], T, V)
    rows_out = [B.dssd_edge_emit_shard(tl[:, :, a:b], ev["accept_len"], ev["row_scale"], T) for a, b in bounds]
    mw = [B.dssd_resample_shard_mass(rows_out[i], dq[:, :, a:b], ev["accept_len"], gamma) for i, (a, b) in enumerate(bounds)]
    masses = torch.stack([m for m, _ in mw])
    draws = [B.dssd_resample_shard_draw(masses, i, a, rows_out[i], dq[:, :, a:b], ev["accept_len"], g["uniforms_rs"],
                                        gamma, mw[i][1]) for i, (a, b) in enumerate(bounds)]
    torch.cuda.synchronize()
    n_gpu = ev["accept_len"].cpu().numpy()
    tok_gpu = torch.stack([dr["token"] for dr in draws]).max(dim=0).values.cpu().numpy()
    n_bonus = int((n_gpu == gamma).sum())

    # the timed shard: the first one (the longest when V is not a multiple of G)
    a0, b0 = bounds[0]
    Vs = b0 - a0
    tl0, dq0 = tl[:, :, a0:b0], dq[:, :, a0:b0]
    ws_e = torch.empty(B.dssd_edge_partial_workspace_bytes(Bn, gamma, Vs), dtype=torch.uint8, device=dev)
    ws_r = torch.empty(B.dssd_resample_shard_workspace_bytes(Bn, gamma, Vs), dtype=torch.uint8, device=dev)
    st = {"part": None, "ev": None, "row": None, "mass": None, "draw": None}
    names = ("partial", "combine", "emit", "mass", "draw")

    def calls():
        st["part"] = B.dssd_edge_partial(tl0, g["draft_tokens"], a0, T, out=st["part"], workspace=ws_e)
        yield
        st["ev"] = B.dssd_edge_combine(ref_all, sum_all, tok_all, g["draft_tokens"], g["draft_q_tok"], g["uniforms"], T, V,
                                       out=st["ev"])
        yield
        st["row"] = B.dssd_edge_emit_shard(tl0, st["ev"]["accept_len"], st["ev"]["row_scale"], T, out=st["row"])
        yield
        st["mass"], _ = B.dssd_resample_shard_mass(st["row"], dq0, st["ev"]["accept_len"], gamma, out=st["mass"], workspace=ws_r)
        yield
        st["draw"] = B.dssd_resample_shard_draw(masses, 0, a0, st["row"], dq0, st["ev"]["accept_len"], g["uniforms_rs"],
                                                gamma, ws_r, out=st["draw"])
        yield

    # a slice smaller than L2 would be served from it on every repetition: write a buffer larger than L2 between steps
    slice_bytes = w.rows * Vs * w.logit_bytes
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if slice_bytes < 200e6 else None
    sampler = ClockSampler(0)
    sampler.start()
    for _ in range(max(args.warmup, 3)):
        for _ in calls():
            pass
    torch.cuda.synchronize()
    K = args.steps

    def one_loop():
        ev_ = [[torch.cuda.Event(enable_timing=True) for _ in range(6)] for _ in range(K)]
        torch.cuda.synchronize()
        for i in range(K):
            if flush is not None:
                flush.fill_(i & 1)
            ev_[i][0].record()
            for j, _ in enumerate(calls()):
                ev_[i][j + 1].record()
        torch.cuda.synchronize()
        per = [[e[j].elapsed_time(e[j + 1]) for e in ev_] for j in range(5)]
        return {"total_ms": sum(e[0].elapsed_time(e[5]) for e in ev_), "per_call_ms": [sum(x) / K for x in per]}

    t_host0 = time.perf_counter()
    loop, loops = timed_loops(one_loop)
    t_host1 = time.perf_counter()
    sampler.stop_flag = True
    sampler.join(timeout=1.0)
    clocks = sampler.summary(t_host0, t_host1)
    ms_per_step = loop["total_ms"] / K
    per_call = dict(zip(names, loop["per_call_ms"]))
    # the same steps (flush included) replayed from a CUDA graph: the four small calls are launch- and
    # latency-bound, so this is what a rank pays once the host's launch work is off the path
    KG = min(K, 32)
    side = torch.cuda.Stream()
    cg = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(cg, stream=side):
            for i in range(KG):
                if flush is not None:
                    flush.fill_(i & 1)
                for _ in calls():
                    pass
    torch.cuda.synchronize()
    cg.replay()
    torch.cuda.synchronize()
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    g0.record()
    for _ in range(5):
        cg.replay()
    g1.record()
    torch.cuda.synchronize()
    graph_ms = g0.elapsed_time(g1) / (5 * KG)
    flush_ms = 0.0
    if flush is not None:
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record()
        for i in range(20):
            flush.fill_(i & 1)
        f1.record()
        torch.cuda.synchronize()
        flush_ms = f0.elapsed_time(f1) / 20
    graph_rec = {"ms_per_step_with_flush": graph_ms, "flush_ms": flush_ms, "ms_per_step": graph_ms - flush_ms,
                 "steps_per_graph": KG, "replays": 5}
    peak, peak_kind = _peaks()
    part_bytes = w.rows * Vs * w.logit_bytes  # every logit of the slice once
    achieved = part_bytes / (per_call["partial"] * 1e-3) / 1e9
    step_bytes = part_bytes + Bn * Vs * 4 + Bn * Vs * 4 + (Bn - n_bonus) * Vs * 4  # + the slice written, read back, and Q_n's slice
    cpu, parity = None, None
    if not args.no_cpu_baseline:
        n_seq = min(Bn, args.ref_sequences)
        sub = {k: v[:n_seq] for k, v in d.items()}
        t0 = time.perf_counter()
        ref = O.verify_round(sub, T, threads=cores)
        dt = time.perf_counter() - t0
        cpu = {"value": n_seq * (gamma + 1) / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"first {n_seq} of {Bn} sequences of {w.name}, whole rows (the dense oracle, to which the "
                         f"sharded oracle is pinned), one pass in {dt:.2f} s wall on {cores} threads"}
        near = ref["margin_acc"] < 1e-6
        same = n_gpu[:n_seq] == ref["accept_len"]
        near_cdf = ref["margin_cdf"] < np.maximum(1e-6, 2e-5 / np.maximum(ref["Z"], 1e-30))
        parity = {"sequences_checked": n_seq, "shards_run": G,
                  "accept_len_mismatch": int(((n_gpu[:n_seq] != ref["accept_len"]) & ~near).sum()),
                  "near_boundary_accept": int(near.sum()),
                  "token_mismatch": int(((tok_gpu[:n_seq] != ref["token"]) & same & ~near_cdf).sum()),
                  "near_boundary_cdf": int((near_cdf & same).sum())}
    cfg = _config(w, args)
    cfg["workload"] = cfg["workload"].replace(f"{w.name}:", f"{w.name}, vocabulary sharded over {G} (one shard of {Vs} entries timed):")
    cfg["shards"] = G
    cfg["parallelism"] = f"vocabulary-sharded x{G}: one shard's calls on one GPU; the two all-gathers are not timed"
    cfg["l2"] = "inputs larger than L2, no flush" if flush is None else "256 MB written between steps"
    print(json.dumps({
        "metric": METRIC, "value": w.rows / (ms_per_step * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": K,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "strong",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": cfg,
        "roofline": {"bound": "hbm", "kernel": "edge_verify_kernel (partial sums of one shard)", "achieved": achieved,
                     "peak": peak, "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                     "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS, "algorithmic_bytes_per_launch": part_bytes,
                     "avg_launch_ms": per_call["partial"], "traffic": None},
        "per_call_ms": per_call, "step_algorithmic_bytes": step_bytes,
        "step_gbs": step_bytes / (ms_per_step * 1e-3) / 1e9,
        "timed": {"loops": len(loops), "device_ms": sum(lp["total_ms"] for lp in loops), "reported": "median loop"},
        "graph": graph_rec,
        "cpu_baseline": cpu, "parity": parity, "e2e": None, "gpu_launches": 7 * K * len(loops), "clocks": clocks,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c4")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--ref-sequences", type=int, default=256)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sampler", default="full", choices=["full", "topk"])
    ap.add_argument("--fused", action="store_true", help="Algorithm 1 in one call (dssd_dsd_verify) instead of the split round")
    ap.add_argument("--bonus", default="device", choices=["device", "edge"],
                    help="who draws the bonus token of a fully accepted sequence: the device from the emitted row "
                         "(dssd_edge_verify), or the edge itself with no row emitted (dssd_edge_verify_bonus)")
    ap.add_argument("--k", type=int, default=10)
    ap.add_argument("--payload", default="f32", choices=["f32", "f16"], help="width of the emitted row P_n (full sampler only)")
    ap.add_argument("--min-timed-ms", type=float, default=MIN_TIMED_MS,
                    help="the timed loop of --steps steps is repeated until this much device time has passed (0: once)")
    ap.add_argument("--sweep", action="store_true", help="the 60 points of the V = 50272 float32 sweep, one record each")
    ap.add_argument("--shards", type=int, default=0,
                    help="time one shard of the vocabulary-sharded round (the vocabulary cut into this many slices)")
    ap.add_argument("--also", default="c5max,c3",
                    help="workloads measured after the default one and reported as sub-records (empty: none)")
    args = ap.parse_args()
    globals()["MIN_TIMED_MS"] = args.min_timed_ms
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started by hand rather than by a launcher: become the launcher, one rank per GPU of this node
        import socket

        with socket.socket() as sock:
            sock.bind(("127.0.0.1", 0))
            port = sock.getsockname()[1]
        os.execv(sys.executable, [sys.executable, "-m", "torch.distributed.run", "--nnodes=1",
                                  f"--nproc-per-node={args.gpus}", "--master-addr", "127.0.0.1",
                                  "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:])
    w = di.get_workload(args.workload)
    if args.steps is None:
        args.steps = 3 if args.impl == "reference" else 2000
    if args.shards > 0 and args.impl == "ours":
        run_ours_sharded(args, w)
    elif args.fused and args.impl == "ours":
        run_ours_fused(args, w)
    elif args.sampler == "topk":
        (run_reference_topk if args.impl == "reference" else run_ours_topk)(args, w)
    elif args.impl == "reference":
        run_reference(args, w)
    elif args.sweep:
        # every point of the V = 50272 float32 sweep, one compact record each, in one JSON line
        recs = []
        for pt in di.sweep_points():
            r = run_ours(args, pt, light=True)
            if r is not None:
                recs.append({"workload": pt.name, "B": pt.B, "gamma": pt.gamma, "sigma_d": pt.sigma_d,
                             "edge_call_us": r["roofline"]["avg_launch_ms"] * 1e3, "frac": r["roofline"]["frac"],
                             "achieved_gbs": r["roofline"]["achieved"], "resample_call_us": r["resample"]["avg_launch_ms"] * 1e3,
                             "step_us": r["ms_per_step"] * 1e3, "rows_per_s": r["value"],
                             "graph_step_us": None if r["graph"] is None else r["graph"]["ms_per_step"] * 1e3,
                             "parity": r["parity"],
                             "sm_mhz": r["clocks"]["sm_mhz"], "reasons": r["clocks"]["reasons"]})
        if recs:
            print(json.dumps({"metric": METRIC, "unit": UNIT, "n_gpus": 1, "steps": args.steps, "sweep": recs}))
    else:
        line = run_ours(args, w)
        if line is not None and args.also and args.workload == "c4" and args.gpus == 1 and args.payload == "f32" \
                and args.bonus == "device":
            # the same measurement on the largest workload by bytes and on the mid-sized one, as sub-records
            line["also"] = {}
            for name in args.also.split(","):
                sub = run_ours(args, di.get_workload(name), light=True)
                line["also"][name] = {k: sub[k] for k in ("value", "ms_per_step", "config", "roofline", "resample",
                                                          "timed", "graph", "cpu_baseline", "parity", "clocks")}
        if line is not None:
            print(json.dumps(line))


if __name__ == "__main__":
    main()
