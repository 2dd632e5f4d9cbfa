#!/usr/bin/env python
"""Benchmark of the SPADE hot path on B200: one step = one attention layer (plan + summarize +
select + attn) over one batch of seeded synthetic Q/K/V.

    python bench.py --gpus N --steps K --warmup W [--workload NAME] [--impl reference]

Prints ONE JSON line.  `value` is the dense-equivalent throughput 4*N^2*d*heads / t_layer
summed over all ranks (ranks run independent replicas: the path has no exchange step).
`--impl reference` times the CPU oracle (as it stands) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2608_03335_b200.workloads import WORKLOADS, bf16_bits, make_qkv, sweep_workload  # noqa: E402

METRIC = "attention_layer_effective_tflops"
UNIT = "TFLOP/s (dense-equivalent, 4*N^2*d*heads per layer)"


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm=p["hbm_gbs"], bf16=p["bf16_tflops"], bf16_sustained=p["bf16_tflops_sustained"], kind="of measured")
    return dict(hbm=6650.0, bf16=1590.0, bf16_sustained=1400.0, kind="of fallback")


def _workload(name):
    if name.startswith("sweep_c"):                       # e.g. sweep_c1_s85
        c, s = name[len("sweep_c"):].split("_s")
        return sweep_workload(int(c), int(s) / 100.0), [int(c)]
    return WORKLOADS[name], None


class ClockSampler:
    """Samples nvidia-smi SM clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "50", "-i", str(self.gpu)], stdout=subprocess.PIPE, text=True)
            self.th = threading.Thread(target=lambda: self.lines.extend(self.proc.stdout), daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        self.th.join(timeout=2)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


def executed_units(plan, w):
    """128-row x 64-key units the attention kernel multiplies, from the GPU's own lists: two per listed
    block for 128-token schemes; for 64-token schemes the merged list of each query tile (two blocks of a
    2 x 2 x 2 cell of the block grid, paired along the axis the head chose for that cell; lone blocks where
    a cell is a single block; text blocks pair among themselves)."""
    t = plan.tables()
    scheme = t["scheme"].cpu().tolist()
    cell_axis = t["cell_axis"].long()
    total = 0
    tables = {}
    for bh, c in enumerate(scheme):
        g = plan.geometry(c)
        nb, nbv = g["NB"], g["NBv"]
        cnt = t["kv_cnt"][bh, :nb].long()
        if g["BS"] == 128:
            total += 2 * int(cnt.sum())
            continue
        idx = t["kv_idx"][bh, :nb].long()
        valid = torch.arange(idx.shape[1], device=idx.device)[None, :] < cnt[:, None]
        mask = torch.zeros(nb, nb + 1, dtype=torch.bool, device=idx.device)
        mask.scatter_(1, torch.where(valid, idx, torch.full_like(idx, nb)), True)
        mask = mask[:, :nb]
        if c not in tables:
            tc, pr = plan.pair_table(c)
            tables[c] = (tc.to(idx.device), pr.to(idx.device))
        tile_cell, pairs = tables[c]
        axis = cell_axis[bh][tile_cell]                                   # [tiles]
        e = pairs.gather(1, axis[:, None])[:, 0]
        qb0, qb1 = e & 0xffff, e >> 16
        qb1 = torch.where(qb1 == 0xffff, qb0, qb1)
        total += int((mask[qb0] | mask[qb1]).sum())
        tm = mask[nbv:]
        if tm.shape[0]:
            if tm.shape[0] % 2:
                tm = torch.cat([tm, torch.zeros_like(tm[:1])], 0)
            total += int((tm[0::2] | tm[1::2]).sum())
    return total


def listed_pair_flops(plan, w):
    """4*d * sum over (query block, listed KV block) of BS*BS: what the lists ask for with every block padded
    to its nominal size, before 64-token query blocks are paired into 128-row tiles."""
    t = plan.tables()
    total = 0.0
    for bh, c in enumerate(t["scheme"].cpu().tolist()):
        g = plan.geometry(c)
        total += float(t["kv_cnt"][bh, :g["NB"]].sum()) * g["BS"] * g["BS"]
    return 4.0 * w.d * total


def achieved_sparsity(plan, w):
    """1 - kept token pairs / N^2 (fraction of pruned attention scores), from the GPU's lists."""
    t = plan.tables()
    T, H, W = w.grid
    kept = 0.0
    for bh, c in enumerate(t["scheme"].cpu().tolist()):
        bt, bh_, bw = w.candidates[c]
        g = plan.geometry(c)

        def sizes(n, b):
            return np.minimum(b, n - b * np.arange(-(-n // b)))

        n = (sizes(T, bt)[:, None, None] * sizes(H, bh_)[None, :, None] * sizes(W, bw)[None, None, :]).reshape(-1)
        if g["NBt"]:
            n = np.concatenate([n, np.minimum(g["BS"], w.n_text - g["BS"] * np.arange(g["NBt"]))])
        nt = torch.tensor(n, dtype=torch.float64, device=t["kv_idx"].device)
        nb = g["NB"]
        idx = t["kv_idx"][bh, :nb].long()
        cnt = t["kv_cnt"][bh, :nb].long()
        valid = torch.arange(idx.shape[1], device=idx.device)[None, :] < cnt[:, None]
        cols = torch.where(valid, nt[idx.clamp(0, nb - 1)], torch.zeros((), dtype=torch.float64, device=idx.device))
        kept += float((cols.sum(1) * nt).sum())
    return 1.0 - kept / (float(w.n_tokens) ** 2 * w.heads * w.batch)


def oracle_sample_seconds(w, forced, Qb, Kb, Vb, n_blocks=4, threads=0):
    """The CPU oracle on a bounded sample: selection in full for head 0, attention on `n_blocks`
    query blocks of head 0; returns (seconds extrapolated to the whole layer, description, cores)."""
    from oracle import spade_oracle as so
    cores = os.cpu_count() or 1
    t0 = time.perf_counter()
    if forced is None:
        p = so.plan_head(Qb[0], Kb[0], w.grid, w.n_text, w.candidates, threads=threads)
        c = p["scheme"]
    else:
        c = forced[0]
    t_plan = time.perf_counter() - t0
    blk = w.candidates[c]
    t0 = time.perf_counter()
    sel = so.select_head(Qb[0], Kb[0], w.grid, w.n_text, blk, w.mode, float(np.float32(w.value)), threads=threads)
    t_sel = time.perf_counter() - t0
    nb = sel["geo"]["NB"]
    rng = np.random.default_rng(0)
    qbl = sorted(int(x) for x in rng.choice(nb, min(n_blocks, nb), replace=False))
    t0 = time.perf_counter()
    so.attention_blocks(Qb[0], Kb[0], Vb[0], w.grid, w.n_text, blk, qbl, sel["kv_idx"], sel["kv_cnt"], threads=threads)
    t_att = time.perf_counter() - t0
    heads = w.heads * w.batch
    total = heads * (t_plan + t_sel + t_att * nb / len(qbl))
    desc = (f"head 0 of {heads}: scheme generation + summaries + estimator + index search in full, "
            f"attention on {len(qbl)} of {nb} query blocks; time extrapolated to all blocks and heads")
    return total, desc, cores


def _config(w, forced, args, **extra):
    """The `config` object both arms print (same keys, so the two lines can be matched)."""
    cfg = dict(workload=w.name, heads=w.heads, grid=list(w.grid), n_text=w.n_text, N=w.n_tokens, d=w.d,
               candidates=[list(c) for c in w.candidates], mode=w.mode, budget=w.value,
               forced_scheme=None if forced is None else forced[0], amplitude=w.amplitude,
               static_masks=dict(window=args.window, sink_tokens=args.sink, intra_threshold=args.intra),
               estimator=args.estimator)
    cfg.update(extra)
    return cfg


def run_reference(args, w, forced):
    """`--impl reference`: the oracle, as it stands, on the host cores (rank 0 only).  Each step is a bounded
    sample of the workload (head 0: selection in full, attention on 16 query blocks); the printed
    ms_per_step is that sample's time scaled to all blocks and heads, and says so."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    # the same generator stream as the GPU arm when a device is there (so head 0 holds the same bytes);
    # torch's CPU stream of the same seed otherwise
    gen_dev = "cuda" if torch.cuda.is_available() else "cpu"
    Q, K, V = make_qkv(w, gen_dev, heads=[0])
    Qb, Kb, Vb = (bf16_bits(x[:, :1])[0] for x in (Q, K, V))
    del Q, K, V
    times, sample_s = [], []
    desc, cores = "", 1
    for i in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        sec, desc, cores = oracle_sample_seconds(w, forced, Qb, Kb, Vb, n_blocks=16)
        if i >= args.warmup:
            times.append(sec)
            sample_s.append(time.perf_counter() - t0)
    sec = sum(times) / len(times)
    val = w.dense_flops() / sec / 1e12
    line = dict(impl="reference", metric=METRIC, value=val, unit=UNIT, n_gpus=args.gpus, steps=args.steps,
                warmup=args.warmup, ms_per_step=sec * 1e3, extrapolated=True,
                measured_sample_ms_per_step=sum(sample_s) / len(sample_s) * 1e3,
                higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="f64", data="synthetic",
                config=_config(w, forced, args, sample=desc,
                               generator=f"torch {gen_dev} generator streams of seed {w.seed} (head 0 only)"),
                cpu_baseline=dict(value=val, unit=UNIT, cores=cores, kind="oracle", sample=desc, extrapolated=True),
                e2e=dict(value=val, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0), gpu_launches=0)
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="wan14b")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--heads", type=int, default=0, help="run a slice of the workload with this many heads (profiling captures)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--window", type=int, default=-1, help="local-window radius in blocks (static mask), < 0 = off")
    ap.add_argument("--sink", type=int, default=0, help="attention-sink tokens (static mask)")
    ap.add_argument("--intra", type=float, default=0.0, help="intra-block threshold on the mean pairwise cosine")
    ap.add_argument("--estimator", default="mean", choices=["mean", "dsa", "dsa2"],
                    help="inter-block estimator: mean summaries (default) or the max/min-summary forms")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    w, forced = _workload(args.workload)
    if args.heads > 0:
        w = w.replace(name=f"{w.name}_heads{args.heads}", heads=args.heads)
    if forced is not None:
        forced = forced * (w.heads * w.batch)

    if args.impl == "reference":
        run_reference(args, w, forced)
        return

    from paper_2608_03335_b200 import multi
    rank, local_rank, world = multi.rank_info()
    torch.cuda.set_device(local_rank)
    dist = multi.init("nccl", torch.device("cuda", local_rank))

    from paper_2608_03335_b200 import binding
    from paper_2608_03335_b200.build import build_library
    if rank == 0:
        build_library()
    if dist is not None:
        dist.barrier()

    dev = torch.device("cuda", local_rank)
    wr = w.replace(index=w.index + multi.replica_seed_offset(rank)) if world > 1 else w       # every rank its own replica
    Q, K, V = make_qkv(wr, dev)
    O = torch.empty_like(Q)
    plan = binding.Plan(w.batch, w.heads, w.grid, w.n_text, w.candidates, w.mode, w.value, device=local_rank,
                        intra_threshold=args.intra, window=args.window, sink_tokens=args.sink, estimator=args.estimator)
    stream = torch.cuda.current_stream()

    def step(events=None):
        if events is None:
            plan.spade_forward(Q, K, V, O, forced_scheme=forced)
            return
        events[0].record(stream)
        plan.spade_plan(Q, K, forced_scheme=forced); events[1].record(stream)
        plan.spade_summarize(Q, K); events[2].record(stream)
        plan.spade_select(); events[3].record(stream)
        plan.spade_attn(Q, K, V, O); events[4].record(stream)

    for _ in range(args.warmup):
        step()
    plan.spade_status()
    torch.cuda.synchronize()

    # ---- timed region: K whole layers, device-timed, max over ranks -------------------------------
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(args.steps)]
    sampler = ClockSampler(local_rank)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    for i in range(args.steps):
        step(evs[i])
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    clocks = sampler.stop()
    plan.spade_status()
    total_ms = evs[0][0].elapsed_time(evs[-1][4])
    stage_ms = [sum(e[i].elapsed_time(e[i + 1]) for e in evs) / args.steps for i in range(4)]
    total_ms = multi.max_over_ranks(total_ms, dist, dev)
    ms_per_step = total_ms / args.steps
    value = multi.aggregate_throughput(w.dense_flops(), world, ms_per_step) / 1e12

    # ---- roofline of the dominant kernel (attention): executed tensor FLOPs / its launch time --------
    peaks = _peaks()
    units = executed_units(plan, w)
    exec_flops = 4.0 * w.d * units * 128 * 64
    listed_flops = listed_pair_flops(plan, w)
    attn_ms = stage_ms[3]
    achieved = exec_flops / (attn_ms * 1e-3) / 1e12
    sparsity = achieved_sparsity(plan, w)
    useful_flops = (1.0 - sparsity) * w.dense_flops()
    useful = useful_flops / (attn_ms * 1e-3) / 1e12
    # DRAM traffic of one launch: only from an ncu capture of this very workload (profiles/), else null
    traffic = None
    prof = os.path.join(ROOT, "profiles", f"k_attn_{w.name}.txt")
    if os.path.exists(prof):
        for ln in open(prof):
            if ln.startswith("dram_bytes_per_launch:"):
                traffic = float(ln.split(":")[1].split()[0])
    # Which measured peak the run compares with follows from the run: the burst figure when the timed region
    # is short or the clocks stayed at their maximum without the power cap, the sustained one otherwise.
    sm, smax = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
    at_max = sm is not None and smax is not None and sm >= 0.985 * smax and "sw_power_cap" not in clocks.get("reasons", [])
    burst = total_ms < 1000.0 or at_max
    peak = peaks["bf16"] if burst else peaks["bf16_sustained"]
    roofline = dict(bound="tensor", kernel="k_attn", achieved=achieved, peak=peak, unit="TFLOP/s",
                    frac=achieved / peak, peak_kind=("bf16 burst, " if burst else "bf16 sustained, ") + peaks["kind"],
                    frac_of_burst_peak=achieved / peaks["bf16"], frac_of_sustained_peak=achieved / peaks["bf16_sustained"],
                    useful_frac=useful / peak, traffic=traffic,
                    executed_tflop_per_launch=exec_flops / 1e12, launch_ms=attn_ms,
                    launch_ms_x_sm_mhz=None if sm is None else attn_ms * sm,
                    algorithmic_dram_bytes_per_launch=4.0 * w.heads * w.batch * w.n_tokens * w.d * 2)
    # selection stages (plan + summarize + select): algorithmic bytes = Q and K read once, the chosen
    # scheme's summaries and the index lists written once
    t_tab = plan.tables()
    list_bytes = 4.0 * float(t_tab["kv_cnt"].sum())
    summ_bytes = 2.0 * 512.0 * sum(plan.geometry(c)["NB"] for c in t_tab["scheme"].cpu().tolist())
    qk_bytes = 2.0 * w.heads * w.batch * w.n_tokens * w.d * 2
    sel_bytes = qk_bytes + summ_bytes + list_bytes
    sel_ms = stage_ms[0] + stage_ms[1] + stage_ms[2]
    stages = dict(achieved_sparsity=sparsity, useful_tflops=useful,
                  executed_split=dict(valid_token_pairs=useful_flops / exec_flops,
                                      edge_padding_of_listed_blocks=(listed_flops - useful_flops) / exec_flops,
                                      unlisted_half_of_paired_tiles=(exec_flops - listed_flops) / exec_flops),
                  plan_ms=stage_ms[0], summarize_ms=stage_ms[1], select_ms=stage_ms[2], attn_ms=stage_ms[3],
                  plan_summarize_hbm_gbs=(qk_bytes + summ_bytes) / ((stage_ms[0] + stage_ms[1]) * 1e-3) / 1e9,
                  selection_ms=sel_ms, selection_algorithmic_bytes=sel_bytes,
                  selection_hbm_gbs=sel_bytes / (sel_ms * 1e-3) / 1e9,
                  selection_hbm_frac=sel_bytes / (sel_ms * 1e-3) / 1e9 / peaks["hbm"],
                  hbm_peak_gbs=peaks["hbm"])

    t = plan.tables()
    schemes_chosen = t["group_count"].cpu().tolist()[:len(w.candidates)]
    pairing_axes = [0, 0, 0]            # cells of the 64-token heads that pair along t, h, w
    for bh, c in enumerate(t["scheme"].cpu().tolist()):
        pt = plan.pair_table(c)
        if pt is not None:
            ncell = int(pt[0].max()) + 1
            for a in range(3):
                pairing_axes[a] += int((t["cell_axis"][bh, :ncell] == a).sum())
    kernel_launches = plan.launch_count()

    # ---- end to end through the host-buffer entry point (it lays the workspace out per head chunk) ----
    e2e = None
    nbytes = Q.numel() * 2
    if not args.no_e2e:
        hq, hk, hv = (x.cpu().pin_memory() for x in (Q, K, V))
        ho = torch.empty_like(hq).pin_memory()
        plan.spade_forward_host(hq, hk, hv, ho, Q, K, V, O, forced_scheme=forced)
        if dist is not None:
            dist.barrier()
        n_e2e = max(3, min(args.steps, 5))
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            plan.spade_forward_host(hq, hk, hv, ho, Q, K, V, O, forced_scheme=forced)
        e2e_ms = (time.perf_counter() - t0) * 1e3 / n_e2e
        e2e_ms = multi.max_over_ranks(e2e_ms, dist, dev)
        e2e = dict(value=multi.aggregate_throughput(w.dense_flops(), world, e2e_ms) / 1e12, unit=UNIT, ms_per_step=e2e_ms,
                   h2d_bytes_per_step=3 * nbytes, d2h_bytes_per_step=nbytes)

    # ---- the oracle on this machine's host cores (rank 0, single-GPU runs only) ----------------------------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        Qb, Kb, Vb = (bf16_bits(x[:, :1])[0] for x in (Q, K, V))
        sec, desc, cores = oracle_sample_seconds(w, forced, Qb, Kb, Vb, n_blocks=32)
        cpu = dict(value=w.dense_flops() / sec / 1e12, unit=UNIT, cores=cores, kind="oracle", sample=desc,
                   extrapolated_ms_per_layer=sec * 1e3)

    if rank == 0:
        line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
                    ms_per_step=ms_per_step, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16",
                    data="synthetic",
                    config=_config(w, forced, args, l2="inputs larger than L2 (Q+K+V+O = %.0f MB)" % (4 * nbytes / 1e6),
                                   schemes_chosen=schemes_chosen, pairing_axes=pairing_axes),
                    roofline=roofline, stages=stages, cpu_baseline=cpu, e2e=e2e, clocks=clocks,
                    gpu_launches=args.steps * kernel_launches,
                    executed_tflops=achieved,
                    useful_note="executed = 128x64 units as multiplied; executed_split says how much of it is valid token "
                                "pairs, zero-filled edge padding of listed blocks, and the half of a paired 64-token tile "
                                "that does not list the unit")
        print(json.dumps(line))
    plan.close()
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
