#!/usr/bin/env python
"""Benchmark of the rank-dAD per-layer path (compress -> gather -> reconstruct) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--rank r] [--iters n]
    python bench.py --impl reference ...       # the float64 CPU oracle on a bounded sample

One step = one pass of the whole path over one synthetic batch: every linear layer of the
configured network, all S sites per layer.  Prints ONE JSON line (rank 0).  With N > 1 ranks
(torchrun) every rank processes its own batch of the same shape (sites and layers are
independent: no data-path collective); the time is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# dram__bytes_read.sum + dram__bytes_write.sum divided by the algorithmic bytes of the same launch, from one ncu
# capture of each kernel at this workload's launch shapes with 512 rows per site (268.4 MB per launch).  The
# streamed operand and the Y^T planes grow with the rows, the factor planes do not; scaled to the 4096-row launches
# timed here that gives the ratios below.  Set an entry to None when its kernel changes until the counters are taken
# again.
DRAM_TRAFFIC_OVER_ALGORITHMIC = {"rows_dot_tc": 1.039, "cols_acc_tc": 1.047}

METRIC = "rank-dAD compress+reconstruct layers/s"
UNIT = "layers/s"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=5, help="benchmark configuration 1..5")
    ap.add_argument("--rank", type=int, default=None, help="override the configuration's rank r")
    ap.add_argument("--iters", type=int, default=None, help="override the power-iteration count")
    ap.add_argument("--resident-blocks", type=int, default=4,
                    help="distinct transformer blocks of input data kept in HBM and cycled through")
    ap.add_argument("--blocks", type=int, default=None,
                    help="run only this many of the network's blocks per step (profiling captures); default all")
    ap.add_argument("--rows", type=int, default=None,
                    help="rows per site instead of the configuration's N (reduced-size profiler captures of the same launch "
                         "shapes: the CTA count of the streaming kernels does not depend on it once the rows are not split)")
    ap.add_argument("--group-blocks", type=int, default=4,
                    help="stack the same-shape layers of this many consecutive blocks into one call")
    ap.add_argument("--no-group", action="store_true",
                    help="one call per layer instead of stacking the same-shape layers of a block into one call")
    ap.add_argument("--cuda-graph", action="store_true",
                    help="capture one step in a CUDA graph and time its replays (for launch-bound configurations)")
    ap.add_argument("--streams", type=int, default=None,
                    help="CUDA streams the independent calls of a step are dealt over (default 3: the small kernels and "
                         "launch tails of one call run under the streaming kernels of another)")
    ap.add_argument("--e2e-steps", type=int, default=1)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-profile-pass", action="store_true")
    ap.add_argument("--no-full-grad", action="store_true", help="skip timing the uncompressed dAD gradient")
    ap.add_argument("--reconstruct-terms", type=int, default=None, choices=[1, 3],
                    help="bf16 products per reconstruction: 3 = two-term splits of the fp32 factors (about 16 bits of each), "
                         "1 = their hi terms only (about 8 bits); default: 1 where the contraction S*r is at least 512 and "
                         "the product is tensor-bound, else 3")
    ap.add_argument("--shard-sites", action="store_true",
                    help="strong scaling over the ranks: every layer's S sites are dealt over the GPUs, each rank compresses "
                         "its own, one all-gather of the factors (NCCL) gives every rank the stacks of all sites, and every "
                         "rank reconstructs locally")
    ap.add_argument("--no-sweep", action="store_true",
                    help="skip the other configurations and the rank / iteration sweep of configuration 5 that a default "
                         "run reports beside its headline workload")
    ap.add_argument("--sweep-steps", type=int, default=3, help="timed steps of each sweep entry")
    ap.add_argument("--no-check", action="store_true", help="skip the oracle check of one sampled site per workload")
    ap.add_argument("--reconstruct-per-call", action="store_true",
                    help="reconstruct after every call instead of once per layer shape and step (one batched call over all "
                         "of the step's layers of that shape, which fills the GPU's rounds of output tiles)")
    return ap.parse_args()


def expand_layers(cfg):
    out = []
    for sh in cfg.layers:
        out.extend([sh] * sh.count)
    return out


def workload_name(cfg, r, iters):
    shapes = ", ".join(f"{sh.count}x {sh.h_in}->{sh.h_out}" for sh in cfg.layers)
    return (f"config {cfg.index} ({cfg.name}): {cfg.n_layers()} linear layers = {cfg.blocks} block(s) of [{shapes}], "
            f"S={cfg.S} sites, N={cfg.N} rows/site, {cfg.dtype} A/Delta, r={r}, iters={iters}")


def stream_bytes_per_layer(cfg, sh, iters):
    """Algorithmic bytes the compress passes stream for one layer: every pass reads D_s or A_s once;
    2*iters+1 passes over each of A and D (Algorithm 2 through Eq. "reduced_iter")."""
    e = cfg.elem_bytes
    return {"rows_dot": ((iters + 1) * sh.h_out + iters * sh.h_in) * cfg.S * cfg.N * e,
            "cols_acc": ((iters + 1) * sh.h_in + iters * sh.h_out) * cfg.S * cfg.N * e,
            "rows_dot_launches": 2 * iters + 1, "cols_acc_launches": 2 * iters + 1}


# ------------------------------------------------------------------------------------------------
class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid: str):
        self.proc = None
        self.uuid = uuid

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", self.uuid, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
                power.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(power)}


def read_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------------------------------------
def oracle_sample(cfg, r, iters):
    """The oracle, as it stands, on a bounded sample: one layer of each distinct shape class (all S
    sites), weighted by how many layers of that class a block has.  Returns (layers/s, seconds, text)."""
    import torch
    from oracle import dad_oracle
    from paper_2102_09631_b200 import workloads as wl
    shapes = list(cfg.layers)
    # layers with the same h_in+h_out cost the same: time one per class
    classes = {}
    for sh in shapes:
        classes.setdefault(sh.h_in + sh.h_out, []).append(sh)
    total_t, parts = 0.0, []
    per_block_t = 0.0
    for key, members in classes.items():
        sh = members[0]
        A, D = wl.decaying_layer(cfg.S, cfg.N, sh.h_in, sh.h_out, wl.seed_for(cfg.index, 0), cfg.torch_dtype)
        Q0 = wl.start_block(cfg.S, r, sh.h_out, wl.seed_for(cfg.index, 0))
        A64, D64, Q64 = dad_oracle.widen(A), dad_oracle.widen(D), dad_oracle.widen(Q0)
        t0 = time.perf_counter()
        dad_oracle.rank_dad_layer(A64, D64, Q64, iters)
        dt = time.perf_counter() - t0
        total_t += dt
        count = sum(m.count for m in members)
        per_block_t += dt * count
        parts.append(f"{sh.h_in}->{sh.h_out} {dt:.2f}s (stands for {count}/block)")
    layers_per_block = sum(sh.count for sh in shapes)
    return layers_per_block / per_block_t, total_t, "one layer per shape class, all sites: " + "; ".join(parts)


def run_reference(args):
    from oracle import dad_oracle
    from paper_2102_09631_b200 import workloads as wl
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = wl.CONFIGS[args.config]
    r = args.rank or cfg.r
    iters = cfg.iters if args.iters is None else args.iters
    dad_oracle.build()
    times, sample = [], ""
    for i in range(args.warmup + args.steps):
        lps, secs, sample = oracle_sample(cfg, r, iters)
        if i >= args.warmup:
            times.append(1.0 / lps)
    per_layer = sum(times) / len(times)
    value = 1.0 / per_layer
    cores = min(dad_oracle.max_threads(), cfg.S)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_layer * cfg.n_layers() * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload_name(cfg, r, iters)},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
def sweep_entries(args):
    """(config, r, iters) of the workloads a default run reports beside the headline: configurations 1-4 as they are
    defined, and configuration 5 over r in {4, 16, 64} x iters in {1, 3}."""
    from paper_2102_09631_b200 import workloads as wl
    out = [(c, wl.CONFIGS[c].r, wl.CONFIGS[c].iters) for c in (1, 2, 3, 4)]
    out += [(5, r, it) for r in (4, 16, 64) for it in (1, 3)]
    return out


# one more entry after those: the headline workload with ONE CALL PER LAYER instead of same-shape layers stacked per
# call, so that the run also shows what a caller gets who does not stack
EXTRA_ENTRY = (5, 16, 3)


def run_ours(args):
    import copy
    import torch
    import torch.distributed as dist
    from paper_2102_09631_b200 import binding as B, build as dad_build, multi, workloads as wl

    rank, local, world = multi.env_rank_world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback); use --impl reference for the oracle")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    multi.init("nccl", dev)
    dad_build.build()
    B.lib()
    if args.shard_sites:
        line = measure_sharded(args, rank, world, dev)
        if rank == 0:
            print(json.dumps(line))
        if world > 1:
            dist.destroy_process_group()
        return
    line = measure(args, rank, local, world, dev, headline=True)
    default_workload = (args.config == 5 and args.rank is None and args.iters is None and args.blocks is None
                        and args.rows is None
                        and not args.no_group and not args.cuda_graph and args.streams is None)
    if default_workload and not args.no_sweep and world == 1:
        sweep = []
        entries = [(e, False) for e in sweep_entries(args)] + [(EXTRA_ENTRY, True)]
        for (c, r, it), per_layer in entries:
            a = copy.copy(args)
            a.config, a.rank, a.iters = c, r, it
            a.no_group = per_layer
            a.no_e2e = a.no_cpu_baseline = a.no_full_grad = True
            a.steps = args.sweep_steps if c >= 4 else 20      # the launch-bound configurations take well under a millisecond
            a.warmup = max(3, args.warmup if c >= 4 else 10)
            torch.cuda.empty_cache()
            e = measure(a, rank, local, world, dev, headline=False)
            if e is not None:
                keep = ("ms_per_step", "value", "unit", "steps", "warmup", "gpu_launches", "launches_per_compress", "clocks",
                        "roofline", "reconstruct", "stream_gbs", "check", "compress_path")
                sweep.append({"config": c, "r": r, "iters": it, "workload": e["config"]["workload"],
                              "calls": e["config"]["calls"],
                              **{k: e.get(k) for k in keep}})
        if line is not None:
            line["sweep"] = sweep
    if rank == 0 and line is not None:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def measure_sharded(args, rank, world, dev):
    """Sites sharded over the ranks (Algorithm 1 with one exchange): per layer, dad_rank_compress on this rank's
    sites, an all-gather of the factors into this rank's own memory, dad_reconstruct on the stacks of all sites.
    Total work is fixed as ranks are added (strong scaling).  Inputs: every site's (A, Delta) from its own seed,
    whichever rank holds it."""
    import torch
    from paper_2102_09631_b200 import binding as B, multi, workloads as wl
    cfg = wl.CONFIGS[args.config]
    if args.blocks is not None:
        import dataclasses
        cfg = dataclasses.replace(cfg, blocks=max(1, min(cfg.blocks, args.blocks)))
    r = args.rank or cfg.r
    iters = cfg.iters if args.iters is None else args.iters
    stream = torch.cuda.current_stream()
    units = []
    for li, sh in enumerate(cfg.layers):
        shard = multi.SiteShardedLayer(cfg.S, r, sh.h_in, sh.h_out)
        mine = shard.sites
        if not mine:
            raise SystemExit(f"more ranks ({world}) than sites ({cfg.S}): nothing to do for rank {rank}")
        As, Ds, Qs = [], [], []
        for site in mine:                       # a site's data depends on the site, not on the rank that holds it
            seed = wl.seed_for(cfg.index, li * 1000 + site)
            gen = wl.gaussian_layer if cfg.index == 1 else wl.decaying_layer
            a, d = gen(1, cfg.N, sh.h_in, sh.h_out, seed, cfg.torch_dtype, dev)
            As.append(a)
            Ds.append(d)
            Qs.append(wl.start_block(1, r, sh.h_out, seed, dev))
        A, D, Q0 = torch.cat(As), torch.cat(Ds), torch.cat(Qs)
        plan = B.LayerPlan(A, D, r, iters, zero_copy_gather=True)
        K = cfg.S * r
        math = plan.math
        grad = torch.empty(sh.h_in, sh.h_out, device=dev, dtype=torch.float32)
        ws_rec = B.new_workspace(B.dad_reconstruct_workspace_bytes(sh.h_in, sh.h_out, K, math), dev)
        units.append((sh, shard, plan, A, D, Q0, grad, ws_rec, math, K))
    ex_events = []

    def step(record):
        for sh, shard, plan, A, D, Q0, grad, ws_rec, math, K in units:
            for _ in range(sh.count * cfg.blocks):
                def compress(sites):
                    B.dad_rank_compress(plan.layer, A, D, r, iters, Q0, plan.P, plan.Q, plan.sigma, plan.ws, stream)
                    return plan.P, plan.Q

                def reconstruct(Pcat, Qcat):
                    B.dad_reconstruct(sh.h_in, sh.h_out, K, Pcat.contiguous(), Qcat.contiguous(), grad, math, ws_rec, stream)
                    return grad

                def on_exchange(begin):
                    if record:
                        ev = torch.cuda.Event(enable_timing=True)
                        ev.record(stream)
                        ex_events.append(ev)

                shard.step(compress, reconstruct, on_exchange)

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            multi.barrier()
            torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        step(False)
    for u in units:
        B.dad_check(u[2].ws)
    sync_all()
    launches0 = B.dad_launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for _ in range(args.steps):
        step(True)
    ev1.record(stream)
    sync_all()
    ms = multi.max_over_ranks(ev0.elapsed_time(ev1), dev) / args.steps
    ex_ms = sum(ex_events[i].elapsed_time(ex_events[i + 1]) for i in range(0, len(ex_events), 2)) / args.steps
    n_layers = cfg.n_layers()
    sent = sum(shard.sent_bytes * sh.count for sh, shard, *_ in units) * cfg.blocks
    expect = sum(B.dad_bytes_rank(plan.layer, r) * len(shard.sites) * sh.count for sh, shard, plan, *_ in units) * cfg.blocks
    all_sent = multi.gather_counts([sent])
    return {"metric": METRIC, "value": n_layers / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms, "higher_is_better": True, "scaling": "strong",
            "vs_baseline": None, "dtype": "f32" if cfg.dtype == "f32" else "bf16", "data": "synthetic",
            "config": {"workload": workload_name(cfg, r, iters),
                       "parallelism": f"sites sharded over {world} rank(s): {cfg.S} sites -> "
                                      f"{[len(multi.shard_units(cfg.S, k, world)) for k in range(world)]} per rank; one "
                                      "all-gather of the factors per layer, every rank reconstructs"},
            "gpu_launches": B.dad_launch_count() - launches0,
            "exchange": {"collective": "all_gather (nccl)" if world > 1 else "none (one rank)",
                         "sent_bytes_per_step_by_rank": [c[0] for c in all_sent],
                         "equals_sum_of_dad_bytes_rank": sent == expect,
                         "ms_per_step_this_rank": ex_ms, "share_of_step": ex_ms / ms if ms > 0 else None}}


def oracle_check(cfg, r, iters, plan, A, D, Q0, site=0):
    """Relative Frobenius error of the projected gradient P_s^T Q_s of one site, as the library left it in the
    plan's buffers, against the float64 oracle on the same inputs (the oracle as checker, outside every timed region)."""
    import numpy as np
    from oracle import dad_oracle
    dad_oracle.build()
    a, d, q0 = A[site:site + 1].cpu(), D[site:site + 1].cpu(), Q0[site:site + 1].cpu()
    Po, Qo, _ = dad_oracle.spi_block(a, d, q0, iters)
    ref = Po[0].T @ Qo[0]
    got = plan.P[site].double().cpu().numpy().T @ plan.Q[site].double().cpu().numpy()
    err = float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300))
    return {"site": site, "quantity": "P_s^T Q_s", "rel_frobenius_error": err,
            "bar": 1e-5 if cfg.dtype == "f32" else 2e-2, "against": "float64 oracle, same inputs"}


def measure(args, rank, local, world, dev, headline):
    import torch
    from paper_2102_09631_b200 import binding as B, multi, workloads as wl

    cfg = wl.CONFIGS[args.config]
    if args.blocks is not None or args.rows is not None:
        import dataclasses
        if args.blocks is not None:
            cfg = dataclasses.replace(cfg, blocks=max(1, min(cfg.blocks, args.blocks)))
        if args.rows is not None:
            cfg = dataclasses.replace(cfg, N=max(1, args.rows))
    r = args.rank or cfg.r
    iters = cfg.iters if args.iters is None else args.iters
    layers = expand_layers(cfg)
    # call units: after a backward pass every layer's (A, Delta) is at hand, and sites and layers are independent
    # in the power iterations, so the layers of one shape from G consecutive blocks (e.g. 4 x 4 attention
    # projections) are stacked as extra slices of one call -- unless --no-group (one call per layer)
    G = 1
    if not args.no_group:
        G = max(g for g in range(1, max(1, args.group_blocks) + 1) if cfg.blocks % g == 0)
    n_super = cfg.blocks // G                      # calls of each unit per step
    RB = max(1, min(n_super, args.resident_blocks // G))   # distinct input sets resident in HBM, cycled
    units = [(sh, 1) for sh in layers] if args.no_group else [(sh, sh.count * G) for sh in cfg.layers]
    data = []
    encoder = None
    if cfg.index == 3:
        # config 3 is one real encoder layer: forward/backward with hooks on its six projections (CPU, seeded)
        proj = wl.encoder_layers(S=cfg.S, seed=wl.seed_for(3, 0, rank))
        by_shape = {}
        for name, A, D in proj:
            by_shape.setdefault((A.shape[2], D.shape[2]), []).append((A, D))
        encoder = by_shape
    for b in range(RB):
        blk = []
        for ui, (sh, groups) in enumerate(units):
            seed = wl.seed_for(cfg.index, b * len(units) + ui, rank)
            if encoder is not None:
                members = encoder[(sh.h_in, sh.h_out)]
                pick = [members[(ui + g) % len(members)] for g in range(groups)] if args.no_group else \
                       [members[g % len(members)] for g in range(groups)]
                A = torch.cat([m[0] for m in pick]).to(dev)
                D = torch.cat([m[1] for m in pick]).to(dev)
            elif cfg.index == 1:
                A, D = wl.gaussian_layer(cfg.S * groups, cfg.N, sh.h_in, sh.h_out, seed, cfg.torch_dtype, dev)
            else:
                A, D = wl.decaying_layer(cfg.S * groups, cfg.N, sh.h_in, sh.h_out, seed, cfg.torch_dtype, dev)
            blk.append((A, D, wl.start_block(cfg.S * groups, r, sh.h_out, seed, dev)))
        data.append(blk)
    # calls of one plan per step: their layers are reconstructed together at the end of the step (one batched call)
    defer = n_super > 1 and not args.reconstruct_per_call and not args.no_group
    n_calls = n_super if defer else 1
    plans = {}
    for ui, (sh, groups) in enumerate(units):
        key = (sh.h_in, sh.h_out, groups)
        if key not in plans:
            A, D, _ = data[0][ui]
            rmath = None
            if cfg.dtype != "f32":
                terms = args.reconstruct_terms or (1 if cfg.S * r >= 512 else 3)
                rmath = B.DAD_BF16_1TERM if terms == 1 else B.DAD_BF16
            plans[key] = B.LayerPlan(A, D, r, iters, groups=groups, reconstruct_math=rmath, calls=n_calls)
    input_bytes = sum(A.numel() * A.element_size() + D.numel() * D.element_size() for blk in data for A, D, _ in blk)
    stream = torch.cuda.current_stream()
    # Calls on different plans are independent (own inputs, workspace and outputs).  Where one call cannot fill the GPU
    # the plans are dealt over several streams, each plan always on the same one; every step forks from and joins the
    # timed stream, so the events around the timed region see all of the work.
    n_streams = args.streams if args.streams is not None else 3
    n_streams = max(1, min(n_streams, len(plans)))
    side_streams = [torch.cuda.Stream(device=dev) for _ in range(n_streams - 1)]
    lane_of = {key: i % n_streams for i, key in enumerate(plans)}

    def step(serial=False):
        lanes = [stream] * n_streams if serial else [stream] + side_streams
        for sd in side_streams:
            sd.wait_stream(stream)
        for b in range(n_super):
            blk = data[b % RB]
            for ui, (sh, groups) in enumerate(units):
                A, D, Q0 = blk[ui]
                key = (sh.h_in, sh.h_out, groups)
                plans[key].step(A, D, Q0, lanes[lane_of[key]], call=b if defer else None)
        if defer:
            for key, plan in plans.items():
                plan.finish(lanes[lane_of[key]])
        for sd in side_streams:
            stream.wait_stream(sd)

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            multi.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    for p in plans.values():
        B.dad_check(p.ws)
    run_step, per_replay = step, None
    if args.cuda_graph:
        # launch-bound configurations: capture one whole step once, replay it for every timed step
        side = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        torch.cuda.synchronize()
        c0 = B.dad_launch_count()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                stream = side
                step()
        stream = torch.cuda.current_stream()
        per_replay = B.dad_launch_count() - c0
        run_step = graph.replay
        run_step()
    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(dev).uuid).replace("GPU-", ""))
    sync_all()
    if rank == 0:
        sampler.start()
        time.sleep(0.15)
    launches0 = B.dad_launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for _ in range(args.steps):
        run_step()
    ev1.record(stream)
    sync_all()
    launches = B.dad_launch_count() - launches0 if per_replay is None else per_replay * args.steps
    clocks = sampler.stop() if rank == 0 else None
    ms = multi.max_over_ranks(ev0.elapsed_time(ev1), dev)
    ms_per_step = ms / args.steps
    n_layers = cfg.n_layers()
    value = multi.whole_job_rate(n_layers, world, ms_per_step * 1e-3)

    # ---- per-kernel times: a second pass of the same steps with events around every launch ----
    peaks = read_peaks()
    roofline, kernels = None, {}
    if not args.no_profile_pass:
        psteps = min(args.steps, 2)
        B.dad_timing_reset()
        B.dad_timing_enable(True)
        for _ in range(psteps):
            step(serial=True)      # one stream: every kernel timed on its own, as the roofline figure wants it
        torch.cuda.synchronize()
        B.dad_timing_enable(False)
        fam = B.dad_timing_collect()
        tot = sum(v[0] for v in fam.values()) or 1.0
        for name, (tms, n) in sorted(fam.items(), key=lambda kv: -kv[1][0]):
            if n:
                kernels[name] = {"ms_per_step": tms / psteps, "launches_per_step": n / psteps, "share": tms / tot}
        top = max(fam.items(), key=lambda kv: kv[1][0])
        name, (tms, n) = top
        alg = None
        base = "rows_dot" if name.startswith("rows_dot") else "cols_acc" if name.startswith("cols_acc") else None
        if base:
            alg = sum(stream_bytes_per_layer(cfg, sh, iters)[base] for sh in layers) * cfg.blocks * psteps
        elif name.startswith("fused_site"):
            # the one-launch compress makes every pass over A and Delta itself: all of the streamed bytes
            alg = sum(stream_bytes_per_layer(cfg, sh, iters)[b] for sh in layers for b in ("rows_dot", "cols_acc")) \
                  * cfg.blocks * psteps
        if alg and n:
            achieved = alg / (tms * 1e-3) / 1e9
            roofline = {"bound": "hbm", "kernel": name, "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                        "frac": achieved / peaks["hbm_gbs"],
                        "traffic": (DRAM_TRAFFIC_OVER_ALGORITHMIC[name] * alg / n
                                    if DRAM_TRAFFIC_OVER_ALGORITHMIC.get(name) else None),
                        "peak_source": peaks["source"],
                        "avg_launch_us": tms / n * 1e3, "algorithmic_bytes_per_launch": alg / n,
                        "timing": f"CUDA events around every launch, second pass of {psteps} step(s)" +
                                  ("" if n_streams == 1 else f" on one stream (the timed steps use {n_streams})")}
        else:
            roofline = {"bound": "hbm", "kernel": name, "achieved": None, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                        "frac": None, "traffic": None, "peak_source": peaks["source"]}

    # ---- the reconstruction products (P^T Q over the S r stacked rows) of the step, from the same event pass ----
    reconstruct = None
    rec = kernels.get("gemm_tn_tc") or kernels.get("gemm_tn_simt")
    if rec:
        K = cfg.S * r
        bf16 = "gemm_tn_tc" in kernels
        # bf16 math multiplies two-term splits of the fp32 factors (three products) or their hi terms only (one)
        terms = (3 if next(iter(plans.values())).math == B.DAD_BF16 else 1) if bf16 else 1
        flops = sum(2.0 * K * sh.h_in * sh.h_out for sh in layers) * cfg.blocks
        out_bytes = sum(4.0 * sh.h_in * sh.h_out for sh in layers) * cfg.blocks
        in_bytes = sum((2.0 * terms if bf16 else 4.0) * K * (sh.h_in + sh.h_out) for sh in layers) * cfg.blocks
        t = rec["ms_per_step"] * 1e-3
        tf_exec = terms * flops / t / 1e12
        reconstruct = {"kernel": "gemm_tn_tc" if bf16 else "gemm_tn_simt", "contraction": K, "products": terms,
                       "ms_per_step": rec["ms_per_step"], "tflops_algorithmic": flops / t / 1e12,
                       "tflops_executed": tf_exec,
                       "frac_tensor_executed": tf_exec / peaks["bf16_tflops"] if bf16 else None,
                       # the product is timed inside the step's event pass, i.e. under the power cap of a long run: its
                       # measured counterpart is the sustained cuBLAS figure, given beside the burst one above
                       "frac_tensor_executed_of_sustained": tf_exec / peaks["bf16_tflops_sustained"] if bf16 else None,
                       "gbs": (out_bytes + in_bytes) / t / 1e9, "frac_hbm": (out_bytes + in_bytes) / t / 1e9 / peaks["hbm_gbs"],
                       "bound": "tensor" if bf16 and terms * flops / (peaks["bf16_tflops"] * 1e12) >
                                (out_bytes + in_bytes) / (peaks["hbm_gbs"] * 1e9) else "hbm"}

    # ---- the uncompressed dAD gradient (sum_s A_s^T D_s) of each layer shape: the tensor-bound product ----
    full_grad = None
    if not args.no_full_grad:
        rows = []
        flops_total, ms_total = 0.0, 0.0
        for ui, (sh, groups) in enumerate(units):
            A, D, _ = data[0][ui]
            # Layers of one shape whose single gradient is too few output tiles for the GPU share a launch
            # (dad_full_grad_grouped): as many of the call's stacked layers as bring the tiles of 256 x 256 to about 64.
            tiles1 = -(-sh.h_in // 256) * -(-sh.h_out // 256)
            gg = 1
            while gg * 2 <= groups and groups % (gg * 2) == 0 and tiles1 * gg * 2 <= 64:
                gg *= 2
            A1, D1 = A[:cfg.S * gg], D[:cfg.S * gg]          # gg layers' slices
            L1 = B.make_layer(A1, D1)
            g = torch.empty(gg, sh.h_in, sh.h_out, device=dev, dtype=torch.float32)
            ws = B.new_workspace(max(256, B.dad_full_grad_grouped_workspace_bytes(L1, gg)), dev)
            for _ in range(2):
                B.dad_full_grad_grouped(L1, gg, A1, D1, g, None, ws, stream)
            f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            reps = 5
            torch.cuda.synchronize()
            f0.record(stream)
            for _ in range(reps):
                B.dad_full_grad_grouped(L1, gg, A1, D1, g, None, ws, stream)
            f1.record(stream)
            torch.cuda.synchronize()
            B.dad_check(ws)
            t_ms = f0.elapsed_time(f1) / reps / gg          # per layer
            fl = 2.0 * cfg.S * cfg.N * sh.h_in * sh.h_out
            flops_total += fl * sh.count
            ms_total += t_ms * sh.count
            rows.append({"layer": f"{sh.h_in}->{sh.h_out}", "us": t_ms * 1e3, "tflops": fl / (t_ms * 1e-3) / 1e12,
                         "layers_per_call": gg})
        tf = flops_total / (ms_total * 1e-3) / 1e12
        full_grad = {"bound": "tensor" if cfg.dtype == "bf16" else "alu", "achieved": tf, "peak": peaks["bf16_tflops"],
                     "unit": "TFLOP/s", "frac": tf / peaks["bf16_tflops"], "peak_source": peaks["source"] + " (burst)",
                     "layers_per_s": sum(sh.count for sh in cfg.layers) / (ms_total * 1e-3), "per_shape": rows}

    # ---- end to end: the C-ABI host entry point; inputs start in pinned host memory, the gradient ends there ----
    e2e = None
    if not args.no_e2e:
        math = B.DAD_F32 if cfg.dtype == "f32" else B.DAD_BF16
        # Two streams take the layers in turn, each with its own device scratch and pinned result buffer, so that one
        # layer's host-to-device copies run under the other's kernels and device-to-host copy.
        lanes = [stream, torch.cuda.Stream(device=dev)]
        host, scratch = [], {}
        for li, sh in enumerate(cfg.layers):      # one pinned input set per layer shape, reused for every such layer
            seed = wl.seed_for(cfg.index, 900 + li, rank)
            if cfg.index == 1:
                A, D = wl.gaussian_layer(cfg.S, cfg.N, sh.h_in, sh.h_out, seed, cfg.torch_dtype, dev)
            else:
                A, D = wl.decaying_layer(cfg.S, cfg.N, sh.h_in, sh.h_out, seed, cfg.torch_dtype, dev)
            Q0 = wl.start_block(cfg.S, r, sh.h_out, seed, dev)
            a, d, q = A.cpu().pin_memory(), D.cpu().pin_memory(), Q0.cpu().pin_memory()
            L1 = B.make_layer(a, d)
            gh = [torch.empty(sh.h_in, sh.h_out, dtype=torch.float32).pin_memory() for _ in lanes]
            for k in range(len(lanes)):
                scratch[(li, k)] = torch.empty(B.dad_rank_dad_host_scratch_bytes(L1, r, iters, math), dtype=torch.uint8,
                                               device=dev)
            host.append((L1, a, d, q, gh))
            del A, D, Q0
        h2d = sum((a.numel() * a.element_size() + d.numel() * d.element_size() + q.numel() * 4) * sh.count
                  for (L1, a, d, q, gh), sh in zip(host, cfg.layers)) * cfg.blocks
        d2h = sum(sh.h_in * sh.h_out * 4 for sh in layers) * cfg.blocks

        def e2e_step():
            k = 0
            for b in range(cfg.blocks):
                for li, sh in enumerate(cfg.layers):
                    L1, a, d, q, gh = host[li]
                    for _ in range(sh.count):
                        B.dad_rank_dad_host(L1, a, d, q, r, iters, math, gh[k], scratch[(li, k)], None, lanes[k])
                        k = (k + 1) % len(lanes)

        e2e_step()
        sync_all()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        lanes[1].wait_stream(stream)       # the second stream starts inside the timed region ...
        for _ in range(args.e2e_steps):
            e2e_step()
        stream.wait_stream(lanes[1])       # ... and ends inside it
        e1.record(stream)
        sync_all()
        ems = multi.max_over_ranks(e0.elapsed_time(e1), dev)
        e2e = {"value": multi.whole_job_rate(n_layers * args.e2e_steps, world, ems * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": args.e2e_steps,
               "call": "dad_rank_dad_host per layer (host A, Delta, Q0 in; host gradient out), layers alternate over two streams"}

    # ---- launches of one compress call, the pipeline each plan takes, and one sampled site against the oracle ----
    sh0, groups0 = units[0]
    key0 = (sh0.h_in, sh0.h_out, groups0)
    A0, D0, Q00 = data[(n_super - 1) % RB][0]          # what the plan of the first unit saw last
    plan0 = plans[key0]
    torch.cuda.synchronize()
    c0 = B.dad_launch_count()
    B.dad_rank_compress(plan0.layer, A0, D0, r, iters, Q00, plan0.P, plan0.Q, plan0.sigma, plan0.ws, stream)
    torch.cuda.synchronize()
    launches_per_compress = B.dad_launch_count() - c0
    names = {B.DAD_PATH_GENERAL: "general", B.DAD_PATH_TENSOR: "tensor", B.DAD_PATH_FUSED: "fused",
             B.DAD_PATH_FUSED_L2: "fused_l2", B.DAD_PATH_TENSOR_PAIRED: "tensor_paired"}
    compress_path = {f"{k[0]}->{k[1]} x{k[2]}": names.get(B.dad_compress_path(pl.layer, r, iters)[0], "?")
                     for k, pl in plans.items()}
    check = None
    if rank == 0 and not args.no_check:
        check = oracle_check(cfg, r, iters, plan0, A0, D0, Q00)
        check["layer"] = f"{sh0.h_in}->{sh0.h_out}"

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import dad_oracle
        dad_oracle.build()
        # repeat the sample until about ten seconds of oracle time have gone by (at most 8 times)
        inv, secs, reps, sample = 0.0, 0.0, 0, ""
        while reps < 8 and (secs < 10.0 or reps == 0):
            lps, s1, sample = oracle_sample(cfg, r, iters)
            inv += 1.0 / lps
            secs += s1
            reps += 1
        cpu = {"value": reps / inv, "unit": UNIT, "cores": min(dad_oracle.max_threads(), cfg.S), "kind": "oracle",
               "sample": f"{reps}x [{sample}]", "seconds": secs}

    if rank == 0:
        # Conservative bound beside the streamed one: every element of A and Delta has to cross HBM at least once
        # per layer (the passes re-read them 2*iters+1 times; nothing of a 64-256-slice launch survives in L2).
        b_min = sum((sh.h_in + sh.h_out) * cfg.S * cfg.N * cfg.elem_bytes for sh in layers) * cfg.blocks
        t_min_ms = b_min / (peaks["hbm_gbs"] * 1e9) * 1e3
        compulsory = {"bytes_per_step": b_min, "t_min_ms": t_min_ms, "frac": t_min_ms / ms_per_step,
                      "note": "t_min = bytes of A and Delta read once / measured HBM rate; the method's passes re-read them"}
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "f32" if cfg.dtype == "f32" else "bf16", "data": "synthetic",
                "config": {"workload": workload_name(cfg, r, iters),
                           "l2": f"inputs larger than L2: {RB} resident input set(s) of {G} block(s), {input_bytes / 1e9:.2f} GB, cycled",
                           "calls": ("one call per layer" if args.no_group else
                                     f"same-shape layers of {G} consecutive block(s) stacked as extra slices of one call: " +
                                     ", ".join(f"{g}x {sh.h_in}->{sh.h_out}" for sh, g in units) +
                                     (f"; the {n_super} calls of a shape per step compress and gather, one batched "
                                      "reconstruction per shape ends the step" if defer else "")),
                           "launch": ("CUDA graph replay" if args.cuda_graph else "stream launches") +
                                     ("" if n_streams == 1 else
                                      f", the step's independent calls dealt over {n_streams} streams"),
                           "factors": "fp32", "accumulate": "f64" if cfg.dtype == "f32" else "f32"},
                "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roofline, "cpu_baseline": cpu,
                "kernels": kernels, "reconstruct": reconstruct, "dad_full_grad": full_grad, "compulsory_traffic": compulsory,
                "stream_gbs": sum(sum(v for k, v in stream_bytes_per_layer(cfg, sh, iters).items() if not k.endswith("launches"))
                                  for sh in layers) * cfg.blocks / (ms_per_step * 1e-3) / 1e9,
                "launches_per_compress": launches_per_compress, "compress_path": compress_path, "check": check}
        return line
    return None


if __name__ == "__main__":
    a = parse_args()
    if a.impl == "reference":
        run_reference(a)
    else:
        run_ours(a)
