"""The multi-GPU path shards the batch by sequence with no exchange step.  Two gloo ranks on the
CPU check what that rests on: a rank's slice of a workload, generated and verified on its own,
equals the same slice of the whole batch (sequences are independent and individually seeded), and
the job's time is the maximum over the ranks."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    import dssd_inputs as di
    from oracle import oracle as O

    w = di.custom(B=6, gamma=3, V=4099, dtype="bf16", temperature=0.8, sigma_d=0.8, seed=99)
    per = w.B // world
    d = di.generate(w, rank * per, (rank + 1) * per)      # this rank's sequences only
    ref = O.verify_round(d, w.temperature)
    mine = torch.from_numpy(np.stack([ref["accept_len"], ref["token"]]).astype(np.int64))
    gathered = [torch.zeros_like(mine) for _ in range(world)]
    dist.all_gather(gathered, mine)                          # only to check: the path itself needs no collective
    # the truncated-support round shards the same way
    dk = di.generate_topk(w, 5, rank * per, (rank + 1) * per)
    refk = O.verify_round_topk(dk, w.temperature, 5)
    mine_k = torch.from_numpy(np.stack([refk["accept_len"], refk["token"]]).astype(np.int64))
    gathered_k = [torch.zeros_like(mine_k) for _ in range(world)]
    dist.all_gather(gathered_k, mine_k)
    slowest = bench.max_over_ranks(10.0 + rank, dist, torch.device("cpu"))
    seeds = [bench.rank_workload(w, r).seed for r in range(world)]
    if rank == 0:
        whole = O.verify_round(di.generate(w), w.temperature)
        got = torch.cat(gathered, dim=1).numpy()
        whole_k = O.verify_round_topk(di.generate_topk(w, 5), w.temperature, 5)
        got_k = torch.cat(gathered_k, dim=1).numpy()
        np.save(os.path.join(out_dir, "ok.npy"),
                np.array([int((got[0] == whole["accept_len"]).all() and (got[1] == whole["token"]).all() and
                              (got_k[0] == whole_k["accept_len"]).all() and (got_k[1] == whole_k["token"]).all()),
                          int(slowest == 10.0 + world - 1), int(len(set(seeds)) == world)]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_by_sequence(tmp_path, oracle_mod):
    port = 29500 + (os.getpid() % 2000)
    mp.spawn(_rank_main, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    ok = np.load(tmp_path / "ok.npy")
    assert ok.tolist() == [1, 1, 1]


def _vocab_rank_main(rank, world, port, out_dir):
    """Vocabulary sharding over two gloo ranks: every rank holds its slice of each row, computes the
    oracle's per-shard quantities, and the two exchanges go through the package's own gather helper
    (the one the CUDA ranks use)."""
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import dssd_inputs as di
    from oracle import oracle as O
    from oracle import shard_oracle as S
    from paper_2507_12000_b200.sharded import all_gather_shards

    w = di.custom(B=24, gamma=3, V=1001, dtype="bf16", temperature=0.8, sigma_d=0.9, seed=321)
    d = di.generate(w)  # the per-sequence inputs are replicated; of the rows a rank looks at its slice only
    a, b = S.shard_bounds(w.V, world)[rank]
    tl, dq = d["target_logits"][:, :, a:b], d["draft_q"][:, :, a:b]
    part = S.edge_partial(tl, d["draft_tokens"], a, w.temperature)
    gathered = {k: all_gather_shards(torch.from_numpy(v)).numpy() for k, v in part.items()}
    parts = [{k: gathered[k][g] for k in part} for g in range(world)]
    ev = S.edge_combine(parts, d["draft_tokens"], d["draft_q_tok"], d["uniforms"], w.V)
    row = S.edge_emit_shard(tl, ev["accept_len"], ev["lse"], w.temperature)
    mass = S.resample_shard_mass(row, dq, ev["accept_len"], w.gamma)
    masses = all_gather_shards(torch.from_numpy(mass)).numpy()
    dr = S.resample_shard_draw(masses, rank, a, row, dq, ev["accept_len"], d["uniforms_rs"], w.gamma)
    token = torch.from_numpy(dr["token"].astype(np.int64))
    dist.all_reduce(token, op=dist.ReduceOp.MAX)
    rows = all_gather_shards(torch.from_numpy(np.pad(row, ((0, 0), (0, (w.V + world - 1) // world - row.shape[1]))))).numpy()
    if rank == 0:
        ref = O.verify_round(d, w.temperature)
        whole = np.concatenate([rows[g][:, :hi - lo] for g, (lo, hi) in enumerate(S.shard_bounds(w.V, world))], axis=1)
        safe = ref["margin_cdf"] > 1e-9
        np.save(os.path.join(out_dir, "ok.npy"),
                np.array([int((ev["accept_len"] == ref["accept_len"]).all()),
                          int(np.allclose(whole, ref["p_row"], rtol=1.2e-7, atol=0)),
                          int((token.numpy()[safe] == ref["token"][safe]).all() and safe.mean() > 0.9),
                          int((dr["flags"] == ref["rs_flags"]).all())]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_by_vocabulary(tmp_path, oracle_mod):
    port = 31500 + (os.getpid() % 2000)
    mp.spawn(_vocab_rank_main, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    ok = np.load(tmp_path / "ok.npy")
    assert ok.tolist() == [1, 1, 1, 1]


def test_bench_starts_its_own_ranks(oracle_mod):
    """`bench.py --gpus 2` started by hand (no launcher, no WORLD_SIZE) re-executes itself under
    torch.distributed.run with two ranks; with the reference arm rank 0 alone works and prints the one
    JSON line, the other rank leaves with status 0."""
    import json
    import subprocess

    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference", "--workload",
                          "c1", "--steps", "1", "--warmup", "0"], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE,
                         text=True, timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, res.stdout
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["metric"] == "verified_rows_per_s"
