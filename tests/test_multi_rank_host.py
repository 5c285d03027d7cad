"""The N > 1 protocol of the benchmark on CPU: two gloo ranks, barrier + max-over-ranks timing, unit
sharding, rank-dependent seeds, and the reference arm running on rank 0 only."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), LOCAL_RANK=str(rank),
                      WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    from paper_2102_09631_b200 import multi, workloads as wl
    multi.init("gloo")
    assert multi.env_rank_world() == (rank, rank, world)
    multi.barrier()
    my_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    ms = multi.max_over_ranks(my_ms)
    rate = multi.whole_job_rate(144, world, ms * 1e-3)
    units = multi.shard_units(7, rank, world)
    seeds = [wl.seed_for(5, u, rank) for u in range(3)]
    counts = multi.gather_counts([rank * 100 + u for u in units])
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
        json.dump({"ms": ms, "rate": rate, "units": units, "seeds": seeds, "counts": counts}, f)
    multi.barrier()
    torch.distributed.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_slowest_time(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r0 = json.load(open(tmp_path / "r0.json"))
    r1 = json.load(open(tmp_path / "r1.json"))
    assert r0["ms"] == r1["ms"] == 15.0                       # max over ranks, on every rank
    assert r0["rate"] == r1["rate"] == 144 * 2 / 15e-3         # whole-job units per second
    assert r0["units"] == [0, 1, 2, 3] and r1["units"] == [4, 5, 6]   # every unit exactly once
    assert set(r0["seeds"]).isdisjoint(r1["seeds"])            # ranks draw different batches
    assert r0["counts"] == r1["counts"] == [[0, 1, 2, 3], [104, 105, 106]]


def _gather_worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), LOCAL_RANK=str(rank),
                      WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import numpy as np
    from oracle import dad_oracle
    from paper_2102_09631_b200 import multi, workloads as wl
    multi.init("gloo")
    S, N, h_in, h_out, r, iters = 5, 12, 10, 9, 2, 2         # 5 sites over 2 ranks: 3 + 2
    A, D = wl.gaussian_layer(S, N, h_in, h_out, 321)
    Q0 = wl.start_block(S, r, h_out, 321)
    # the exchange logic the benchmark's --shard-sites mode runs (multi.SiteShardedLayer), here on CPU tensors over
    # gloo with the oracle standing in for the library's compress and reconstruct
    shard = multi.SiteShardedLayer(S, r, h_in, h_out)
    mine = shard.sites
    assert mine == multi.shard_units(S, rank, world)
    stacks = {}

    def compress(sites):
        P, Q, _ = dad_oracle.spi_block(A[sites], D[sites], Q0[sites], iters)   # this rank compresses its own sites
        return torch.from_numpy(P), torch.from_numpy(Q)

    def reconstruct(Pc, Qc):
        stacks["P"], stacks["Q"] = Pc, Qc
        return dad_oracle.reconstruct(Pc.numpy(), Qc.numpy())                # every rank reconstructs the same gradient

    marks = []
    grad = shard.step(compress, reconstruct, on_exchange=marks.append)
    assert marks == [True, False]
    assert shard.sent_bytes == len(mine) * dad_oracle.bytes_rank(r, h_in, h_out)
    Pcat, Qcat = stacks["P"], stacks["Q"]
    ref = dad_oracle.rank_dad_layer(A, D, Q0, iters)                       # all sites in one process
    ok = (np.array_equal(Pcat.numpy(), ref["Pcat"]) and np.array_equal(Qcat.numpy(), ref["Qcat"])
          and np.array_equal(grad, ref["grad"]))
    sent = multi.gather_counts([dad_oracle.bytes_rank(r, h_in, h_out)] * len(mine))
    with open(os.path.join(out_dir, f"g{rank}.json"), "w") as f:
        json.dump({"ok": bool(ok), "sent": sent, "rows": int(Pcat.shape[0])}, f)
    multi.barrier()
    torch.distributed.destroy_process_group()


def test_sites_sharded_over_ranks_gather_to_the_same_stacks(tmp_path):
    """Sites split over two ranks, factors all-gathered: every rank holds exactly the stacks (and hence the
    gradient) a single process computes; per-site byte counts survive the exchange."""
    world, port = 2, _free_port()
    mp.spawn(_gather_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    for rank in range(world):
        g = json.load(open(tmp_path / f"g{rank}.json"))
        assert g["ok"] and g["rows"] == 5 * 2
        assert g["sent"] == [[2 * 19 * 4] * 3, [2 * 19 * 4] * 2]


def test_single_rank_helpers_need_no_process_group():
    sys.path.insert(0, ROOT)
    from paper_2102_09631_b200 import multi
    assert multi.max_over_ranks(3.5) == 3.5
    assert multi.shard_units(5, 0, 1) == [0, 1, 2, 3, 4]
    assert sum(len(multi.shard_units(10, r, 4)) for r in range(4)) == 10
    assert multi.gather_counts([1, 2]) == [[1, 2]]
    multi.barrier()


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(_free_port()))
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "1",
                          "--gpus", "2", "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert res.returncode == 0 and res.stdout.strip() == ""
    env["RANK"] = env["LOCAL_RANK"] = "0"
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "1",
                          "--gpus", "2", "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert res.returncode == 0
    line = json.loads(res.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
