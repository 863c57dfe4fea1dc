#!/usr/bin/env python
"""Benchmark of the grouped LM-head draft step on B200.

One "step" is one draft call (gate -> top-k groups -> gathered GEMV of the
selected groups -> log-sum-exp -> top-k tokens) over one batch of M query rows.
Headline workload: the Llama3-8B-shaped draft head of the paper's Table 1
(H=4096, V=128256) in 64 groups with the top 8 active (the N=64/top8 cell of
its Table 4), M=8 tree-node rows, 10 candidates per row; seeded synthetic
bf16 weights N(0, 0.02) and hidden states N(0, 1).

value = algorithmic bytes of the step (bytes of the groups actually touched +
gate + hidden + outputs) / step time, summed over ranks: achieved HBM GB/s.
The same line carries the step latency, the dense head (all groups active and
a torch matmul comparator), other M, the dominant kernel's roofline fraction,
an end-to-end number through the host-buffer entry point, and the CPU oracle
timed on the host cores.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "grouped LM-head draft-step HBM GB/s (algorithmic bytes of touched groups / step time)"
UNIT = "GB/s"
WORKLOAD = "llama3_8b"
N_BATCHES = 8            # distinct hidden batches rotated through the steps
# DRAM bytes per algorithmic byte of the dominant kernel, from the ncu capture summarised in
# profiles/head_stream_kernel_llama3_M8.md ((read + write) / weight bytes of the touched groups, two launches).
# Set to None whenever that kernel changes until the capture is redone.
STREAM_TRAFFIC_RATIO = 1.015
FLUSH_BYTES = 512 << 20  # > 2x the 126 MB L2: written, then read back, between timed steps


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 6:
                continue
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except ValueError:
                continue
            for n, val in zip(names, r[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def _visible_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except (ValueError, IndexError):
            return local_rank
    return local_rank


def aggregate_over_ranks(dist, local_ms: float, local_bytes: float, device=None):
    """Whole-job figures: time = max over ranks, bytes = sum over ranks (no data-path collective)."""
    import torch
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    b = torch.tensor([local_bytes], dtype=torch.float64, device=device)
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(b, op=dist.ReduceOp.SUM)
    return float(t.item()), float(b.item())


def batches_for_rank(rank: int, world: int, n_batches: int = N_BATCHES):
    """Every rank drafts for its own sequences: disjoint hidden batches per rank."""
    return [rank * n_batches + i for i in range(n_batches)]


def run_oracle_baseline(cfg, W, gm, Wg, hidden_batches, steps, warmup=0):
    """Times the CPU oracle, as it stands, on whole draft steps of the same workload."""
    from oracle import lmhead_oracle as orc
    times, touched = [], []
    for i in range(warmup + steps):
        hb = hidden_batches[i % len(hidden_batches)]
        t0 = time.perf_counter()
        r = orc.draft(W, gm, Wg, hb, cfg.k_groups, cfg.k_tokens, want_logits=False)
        dt = time.perf_counter() - t0
        if i >= warmup:
            times.append(dt)
            touched.append(len(set(r.groups.ravel().tolist())))
    return times, touched, orc.threads()


def workload_label(cfg):
    """The same string in both arms' `config.workload`."""
    return (f"{cfg.name}: H={cfg.H} V={cfg.V} N={cfg.N} top-{cfg.k_groups} M={cfg.M} k_tokens={cfg.k_tokens}, "
            f"seed {cfg.seed}")


def bench_config(cfg, world):
    """`config` of the JSON line, the same in both arms."""
    return {"workload": workload_label(cfg),
            "l2": f"flush: {FLUSH_BYTES >> 20} MiB written then read before every timed step; {N_BATCHES} hidden "
                  "batches rotated",
            "parallelism": f"replicas x{world}, rows sharded by sequence, no collective"}


def algorithmic_bytes(cfg, groups_touched, M):
    return groups_touched * cfg.v * cfg.H * 2 + cfg.N * cfg.H * 2 + M * cfg.H * 2 + M * cfg.k_tokens * 8


def main_reference(args, rank):
    """--impl reference: the CPU oracle on the host cores (rank 0 only)."""
    if rank != 0:
        return
    from paper_2502_16880_b200 import synth
    cfg = synth.CONFIGS[WORKLOAD].with_(M=args.rows)
    W, gm, Wg = synth.make_w_vocab(cfg), synth.make_group_map(cfg), synth.make_w_gate(cfg)
    hbs = [synth.make_hidden(cfg, cfg.M, batch=b) for b in range(N_BATCHES)]
    times, touched, cores = run_oracle_baseline(cfg, W, gm, Wg, hbs, args.steps, args.warmup)
    total = sum(times)
    byts = sum(algorithmic_bytes(cfg, u, cfg.M) for u in touched)
    val = byts / total / 1e9
    sample = f"whole draft steps, M={cfg.M}, {args.steps} steps"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": total / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": bench_config(cfg, args.gpus),
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--rows", type=int, default=8, help="M of the headline workload")
    ap.add_argument("--quick", action="store_true", help="headline only: skip the other M, dense and CPU legs")
    ap.add_argument("--large-m-only", type=int, default=0, metavar="M",
                    help="run only the tensor-core leg with M rows (a short run for profilers) and print its line")
    ap.add_argument("--vocab-shard-only", type=int, default=0, metavar="M",
                    help="run only the vocab-sharded step with M rows: every rank reads its own groups, one all-gather "
                         "of the per-row records, merge (strong scaling: all ranks draft for the same rows)")
    ap.add_argument("--csra-only", type=int, default=0, metavar="N",
                    help="run only the CSRA objective (Eq. 2) with N positions, 4 key blocks, D = H (a short run for profilers)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        main_reference(args, rank)
        return

    import torch
    import torch.distributed as dist
    from paper_2502_16880_b200 import lmhead, synth

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    lmhead.load_library()

    cfg = synth.CONFIGS[WORKLOAD].with_(M=args.rows)
    headline_cfg = cfg
    if args.csra_only:
        n_c, v_c, D_c = args.csra_only, 4, cfg.H
        rng_c = np.random.default_rng([cfg.seed, 77])
        mk = lambda rows: torch.from_numpy(synth.fp32_to_bf16_bits(rng_c.standard_normal((rows, D_c), dtype=np.float32))
                                           .view(np.int16)).to(dev).view(torch.bfloat16)
        Qc, Kc = mk(n_c), mk(n_c * v_c)
        ws_c = torch.empty(lmhead.coral_csra_workspace_bytes(n_c, v_c, D_c), dtype=torch.uint8, device=dev)
        loss_c = torch.empty(1, dtype=torch.float32, device=dev)
        ts = []
        for i in range(args.warmup + args.steps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            lmhead.coral_csra_infonce(Qc, Kc, v_c, 0.07, ws_c, loss_c)
            b.record()
            torch.cuda.synchronize()
            if i >= args.warmup:
                ts.append(a.elapsed_time(b))
        print(json.dumps({"csra_only": n_c, "views": v_c, "D": D_c, "us": float(np.mean(ts)) * 1e3,
                          "tflops": 2.0 * n_c * n_c * v_c * D_c / (float(np.mean(ts)) * 1e-3) / 1e12,
                          "loss": float(loss_c.item()), "status": lmhead.coral_csra_status(ws_c)}))
        return
    W, gm, Wg = synth.make_w_vocab(cfg), synth.make_group_map(cfg), synth.make_w_gate(cfg)

    def dev_bf16(bits):
        return torch.from_numpy(bits.view(np.int16)).to(dev).view(torch.bfloat16)

    Wd = dev_bf16(W)
    if args.large_m_only:
        Mb = args.large_m_only
        big = lmhead.LMHead(Wd, torch.from_numpy(gm), dev_bf16(Wg), max_M=Mb, max_k_groups=cfg.k_groups,
                            max_k_tokens=cfg.k_tokens)
        hb = dev_bf16(synth.make_hidden(cfg, Mb, batch=100))
        ids_b = torch.empty((Mb, cfg.k_tokens), dtype=torch.int32, device=dev)
        lps_b = torch.empty((Mb, cfg.k_tokens), dtype=torch.float32, device=dev)
        ts = []
        for i in range(args.warmup + args.steps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            lmhead.coral_lmhead_draft(big.handle, hb, cfg.k_groups, cfg.k_tokens, ids_b, lps_b)
            b.record()
            torch.cuda.synchronize()
            if i >= args.warmup:
                ts.append(a.elapsed_time(b))
        st = big.stats()
        lmhead.coral_lmhead_set_kernel_timing(big.handle, True)      # stage split, from events inside the call
        stg = []
        for i in range(10):
            lmhead.coral_lmhead_draft(big.handle, hb, cfg.k_groups, cfg.k_tokens, ids_b, lps_b)
            torch.cuda.synchronize()
            if i >= 3:
                stg.append(lmhead.coral_lmhead_stage_ms(big.handle))
        lmhead.coral_lmhead_set_kernel_timing(big.handle, False)
        print(json.dumps({"large_m_only": Mb, "path": int(st.path), "us_per_step": float(np.mean(ts)) * 1e3,
                          "stage_us": {k: float(np.mean([x[j] for x in stg])) * 1e3
                                       for j, k in enumerate(("router", "head_kernels", "merge"))},
                          "status": big.status()}))
        big.close()
        return
    if args.vocab_shard_only:
        Ms = args.vocab_shard_only
        sh = lmhead.LMHead(Wd, torch.from_numpy(gm), dev_bf16(Wg), max_M=Ms, max_k_groups=cfg.k_groups,
                           max_k_tokens=cfg.k_tokens, shard=(rank, world) if world > 1 else None)   # stores its own groups only
        hs = [dev_bf16(synth.make_hidden(cfg, Ms, batch=b)) for b in range(N_BATCHES)]     # same rows on every rank
        Wrec = 2 + 2 * cfg.k_tokens
        rec = torch.empty((Ms, Wrec), dtype=torch.int32, device=dev)
        gathered = torch.empty((world, Ms, Wrec), dtype=torch.int32, device=dev)
        ids_s = torch.empty((Ms, cfg.k_tokens), dtype=torch.int32, device=dev)
        lps_s = torch.empty((Ms, cfg.k_tokens), dtype=torch.float32, device=dev)
        flush_s = torch.empty(FLUSH_BYTES // 8, dtype=torch.int64, device=dev)

        def step(i):
            lmhead.coral_lmhead_draft_partial(sh.handle, hs[i % len(hs)], cfg.k_groups, cfg.k_tokens, rec)
            if world > 1:
                dist.all_gather_into_tensor(gathered.view(world * Ms, Wrec), rec)
            else:
                gathered[0].copy_(rec)
            lmhead.coral_lmhead_merge_partials(gathered, cfg.k_tokens, ids_s, lps_s)

        ts, touched_s = [], []
        for i in range(max(args.warmup, 3) + args.steps):
            flush_s.fill_(i)
            torch.sum(flush_s)
            if world > 1:
                dist.barrier()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            step(i)
            b.record()
            torch.cuda.synchronize()
            if i >= max(args.warmup, 3):
                ts.append(a.elapsed_time(b))
                touched_s.append(sh.stats().groups_touched)
        local_ms = float(sum(ts))
        local_bytes = float(sum(u * cfg.v * cfg.H * 2 for u in touched_s))
        tot_ms, tot_bytes = aggregate_over_ranks(dist if world > 1 else None, local_ms, local_bytes, dev)
        if rank == 0:
            print(json.dumps({"vocab_shard_only": Ms, "n_gpus": world, "scaling": "strong",
                              "us_per_step": tot_ms / args.steps * 1e3,
                              "GBps_all_ranks": tot_bytes / (tot_ms * 1e-3) / 1e9,
                              "groups_touched_rank0_mean": float(np.mean(touched_s)),
                              "exchange_bytes_per_rank": Ms * Wrec * 4, "status": sh.status()}))
        sh.close()
        if world > 1:
            dist.destroy_process_group()
        return
    head = lmhead.LMHead(Wd, torch.from_numpy(gm), dev_bf16(Wg), max_M=64, max_k_groups=cfg.N, max_k_tokens=cfg.k_tokens)
    default_head = head
    flush = torch.empty(FLUSH_BYTES // 8, dtype=torch.int64, device=dev)
    stream = torch.cuda.current_stream()

    def flush_l2(i):
        """Cold L2 before a timed step, outside the event pair: overwrite a buffer larger than L2, then read
        it back so that the lines left in L2 are clean (dirty lines would be written back to HBM during the
        timed kernels and charged to them)."""
        flush.fill_(i)
        torch.sum(flush)

    def time_steps(M, k_groups, steps, warmup, batches, kernel_timing=False, rho=0.0, zipf_s=0.0, on=None, cold=True,
                   shape=None, stages=None):
        """Per-step CUDA-event times (ms) with an L2 flush before every step, outside the event pair.  With
        kernel_timing the library records events around its stages (which keeps the kernels of a call from
        overlapping, so step times come from runs without it); `stages`, a list, receives (route, head, merge) ms."""
        head = on if on is not None else default_head
        cfg = shape if shape is not None else headline_cfg
        hb_bits = [synth.make_hidden(cfg.with_(rho=rho, zipf_s=zipf_s), M, batch=b) for b in batches]
        hds = [dev_bf16(b) for b in hb_bits]
        ids = torch.empty((M, cfg.k_tokens), dtype=torch.int32, device=dev)
        lps = torch.empty((M, cfg.k_tokens), dtype=torch.float32, device=dev)
        lmhead.coral_lmhead_set_kernel_timing(head.handle, kernel_timing)
        ms, kms, touched, launches = [], [], [], 0
        ev0 = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        ev1 = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        for i in range(warmup):
            if cold:
                flush_l2(i)
            lmhead.coral_lmhead_draft(head.handle, hds[i % len(hds)], k_groups, cfg.k_tokens, ids, lps, stream)
        # union size per batch (the stats call synchronises; done outside the timed steps)
        per_batch_union = []
        for hd in hds:
            lmhead.coral_lmhead_draft(head.handle, hd, k_groups, cfg.k_tokens, ids, lps, stream)
            st = head.stats()
            per_batch_union.append(st.groups_touched)
            per_launch = st.kernel_launches
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        for i in range(steps):
            if cold:
                flush_l2(i)
            ev0[i].record(stream)
            lmhead.coral_lmhead_draft(head.handle, hds[i % len(hds)], k_groups, cfg.k_tokens, ids, lps, stream)
            ev1[i].record(stream)
            launches += per_launch
            touched.append(per_batch_union[i % len(hds)])
            if kernel_timing:
                kms.append(lmhead.coral_lmhead_head_kernel_ms(head.handle))
                if stages is not None:
                    stages.append(lmhead.coral_lmhead_stage_ms(head.handle))
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        ms = [a.elapsed_time(b) for a, b in zip(ev0, ev1)]
        lmhead.coral_lmhead_set_kernel_timing(head.handle, False)
        assert head.status() == 0
        return ms, kms, touched, launches, hb_bits

    NOMINAL_HBM_GBPS = 7700.0     # HBM3e nameplate of the HGX B200 (context; the fractions that are judged use the measured copy peak)

    def copy_floor_us(on, nbytes, in_flight=0, repeats=1, cold=True, n=13):
        """Mean time (us) of the do-nothing bulk-copy stream over the first nbytes of `on`'s packed head."""
        nbytes = int(nbytes) // 16384 * 16384
        ts = []
        for i in range(n):
            if cold:
                flush_l2(i)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            lmhead.coral_lmhead_copy_floor(on.handle, nbytes, stream, in_flight=in_flight, repeats=repeats)
            b.record(stream)
            torch.cuda.synchronize()
            if i >= 3:
                ts.append(a.elapsed_time(b))
        assert on.status() == 0
        return float(np.mean(ts)) * 1e3

    def timed_case(on, shape, M, k_groups, steps):
        """One (shape, M, k_groups) point, cold L2: whole-step time, the three stages timed by events inside the
        call (a separate run), and the copy floor of the same weight bytes."""
        ms_m, _, t_m, _, _ = time_steps(M, k_groups, steps, 3, my_batches, on=on, shape=shape)
        stg = []
        _, kms, _, _, _ = time_steps(M, k_groups, min(steps, 30), 3, my_batches, kernel_timing=True, on=on,
                                     shape=shape, stages=stg)
        c2 = shape.with_(M=M, k_groups=k_groups)
        b_m = float(np.mean([algorithmic_bytes(c2, u, M) for u in t_m]))
        w_m = float(np.mean([u * c2.v * c2.H * 2 for u in t_m]))
        us = float(np.mean(ms_m)) * 1e3
        k_us = float(np.mean(kms)) * 1e3
        floor = copy_floor_us(on, w_m)
        return {"M": M, "k_groups": k_groups, "path": int(on.stats().path), "us_per_step": us,
                "us_per_step_median": float(np.median(ms_m)) * 1e3, "GBps": b_m / us / 1e3,
                "hbm_frac": b_m / us / 1e3 / peak, "hbm_frac_of_nominal": b_m / us / 1e3 / NOMINAL_HBM_GBPS,
                "groups_touched_mean": float(np.mean(t_m)), "roofline_us_at_measured_peak": b_m / peak / 1e3,
                "stage_us": {"router": float(np.mean([x[0] for x in stg])) * 1e3,
                             "head_kernel": float(np.mean([x[1] for x in stg])) * 1e3,
                             "merge": float(np.mean([x[2] for x in stg])) * 1e3},
                "head_kernel_us": k_us, "head_kernel_GBps": w_m / k_us / 1e3, "head_kernel_hbm_frac": w_m / k_us / 1e3 / peak,
                "copy_floor_us_same_bytes": floor, "head_kernel_frac_of_copy_floor": floor / k_us}

    my_batches = batches_for_rank(rank, world)
    sampler = ClockSampler(_visible_index(local_rank))
    sampler.start()            # runs across every timed GPU leg below
    ms, _, touched, launches, hb_bits = time_steps(cfg.M, cfg.k_groups, args.steps, max(args.warmup, 3), my_batches)
    local_ms = float(sum(ms))
    local_bytes = float(sum(algorithmic_bytes(cfg, u, cfg.M) for u in touched))
    tot_ms, tot_bytes = aggregate_over_ranks(dist if world > 1 else None, local_ms, local_bytes, dev)
    value = tot_bytes / (tot_ms * 1e-3) / 1e9

    # dominant kernel: the weight-streaming kernel, timed alone with events inside the library call
    peak, peak_kind = _peaks()
    ksteps = min(args.steps, 100)
    _, kms, ktouched, _, _ = time_steps(cfg.M, cfg.k_groups, ksteps, 3, my_batches, kernel_timing=True)
    k_bytes = float(np.mean([u * cfg.v * cfg.H * 2 + cfg.M * cfg.H * 2 for u in ktouched]))
    k_ms = float(np.mean(kms))
    achieved = k_bytes / (k_ms * 1e-3) / 1e9
    # floor for that kernel: a do-nothing bulk-copy stream of the same number of bytes of the packed head, cold L2
    copy_floor_us_ = copy_floor_us(head, k_bytes, n=23)
    roofline = {"bound": "hbm", "kernel": "head_stream_kernel", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "copy_floor_us_same_bytes": copy_floor_us_, "frac_of_copy_floor": copy_floor_us_ / (k_ms * 1e3),
                "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                "frac_of_nominal_hbm3e": achieved / NOMINAL_HBM_GBPS, "nominal_hbm3e_GBps": NOMINAL_HBM_GBPS,
                "traffic": None if STREAM_TRAFFIC_RATIO is None else STREAM_TRAFFIC_RATIO * k_bytes,
                "traffic_source": "bytes x the DRAM-bytes-per-algorithmic-byte ratio of the ncu capture in profiles/ "
                                  "(not measured in this run)",
                "avg_launch_us": k_ms * 1e3, "algorithmic_bytes_per_launch": k_bytes}

    # end to end through the host-buffer entry point (pinned host memory; copies inside the timed region)
    hh = [torch.from_numpy(b.view(np.int16)).pin_memory() for b in hb_bits]
    ids_h = torch.empty((cfg.M, cfg.k_tokens), dtype=torch.int32).pin_memory()
    lps_h = torch.empty((cfg.M, cfg.k_tokens), dtype=torch.float32).pin_memory()
    e2e_steps = min(args.steps, 100)
    for i in range(3):
        lmhead.coral_lmhead_draft_host(head.handle, hh[i % len(hh)], cfg.k_groups, cfg.k_tokens, ids_h, lps_h, stream)
    e2e_t = 0.0
    for i in range(e2e_steps):
        flush_l2(i)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        lmhead.coral_lmhead_draft_host(head.handle, hh[i % len(hh)], cfg.k_groups, cfg.k_tokens, ids_h, lps_h, stream)
        e2e_t += time.perf_counter() - t0
    e2e_bytes = float(sum(algorithmic_bytes(cfg, touched[i % len(touched)], cfg.M) for i in range(e2e_steps)))
    e2e_ms, e2e_tot_bytes = aggregate_over_ranks(dist if world > 1 else None, e2e_t * 1e3, e2e_bytes, dev)
    e2e = {"value": e2e_tot_bytes / (e2e_ms * 1e-3) / 1e9, "unit": UNIT, "us_per_step": e2e_ms / e2e_steps * 1e3,
           "h2d_bytes_per_step": cfg.M * cfg.H * 2, "d2h_bytes_per_step": cfg.M * cfg.k_tokens * 8}

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": tot_ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16 inputs, f32 accumulate", "data": "synthetic",
        "config": bench_config(cfg, world),
        "us_per_step": tot_ms / args.steps * 1e3,
        "us_per_step_median": float(np.median(ms)) * 1e3,
        "us_per_step_p10": float(np.percentile(ms, 10)) * 1e3,
        "us_per_step_p90": float(np.percentile(ms, 90)) * 1e3,
        "groups_touched_mean": float(np.mean(touched)),
        "hbm_frac_whole_step": value / (peak * world),
        "hbm_frac_whole_step_of_nominal": value / (NOMINAL_HBM_GBPS * world),
        "roofline": roofline, "e2e": e2e, "gpu_launches": launches,
    }

    if rank == 0 and world == 1 and not args.quick:
        extra_steps = min(args.steps, 50)
        # warm L2 (no flush; the same 8 batches rotate, so parts of the head are still in the 126 MB L2): labelled,
        # not the headline - in a real draft cycle the other layers' weights stream through L2 between head calls
        ms_w, _, _, _, _ = time_steps(cfg.M, cfg.k_groups, extra_steps, 3, my_batches, cold=False)
        out["warm_l2_us_per_step"] = float(np.mean(ms_w)) * 1e3
        out["other_M"] = [timed_case(head, cfg, M, cfg.k_groups, extra_steps) for M in (1, 60)]
        # the paper's two-layer router (Eq. 7: scores = W2 (act(W1 h) + h)): W1 is H x H, 33.5 MB more to read per call
        W1d = dev_bf16(synth._normal_bf16(np.random.default_rng([cfg.seed, 91]), cfg.H, cfg.H, 0.01))
        lmhead.coral_lmhead_set_router_mlp(head.handle, W1d)
        eq7 = []
        for M7 in (1, 8, 60):
            ms7, _, t7, _, _ = time_steps(M7, cfg.k_groups, min(extra_steps, 30), 3, my_batches)
            b7 = float(np.mean([algorithmic_bytes(cfg.with_(M=M7), u, M7) for u in t7])) + 2.0 * cfg.H * cfg.H
            eq7.append({"M": M7, "us_per_step": float(np.mean(ms7)) * 1e3, "groups_touched_mean": float(np.mean(t7)),
                        "algorithmic_bytes_with_W1": b7, "GBps": b7 / (float(np.mean(ms7)) * 1e-3) / 1e9,
                        "hbm_frac": b7 / (float(np.mean(ms7)) * 1e-3) / 1e9 / peak})
        lmhead.coral_lmhead_set_router_mlp(head.handle, None)
        out["eq7_two_layer_router"] = eq7
        del W1d
        # extra (not a workload of the list): rows correlated like tree siblings of one parent, where the union
        # of selected groups no longer saturates (Appendix B: the worst case is unlikely in practice)
        ms_c, _, t_c, _, _ = time_steps(60, cfg.k_groups, extra_steps, 3, my_batches, rho=0.3)
        b_c = float(np.mean([algorithmic_bytes(cfg.with_(M=60), u, 60) for u in t_c]))
        out["correlated_rows_M60_rho0.3"] = {"us_per_step": float(np.mean(ms_c)) * 1e3,
                                             "groups_touched_mean": float(np.mean(t_c)),
                                             "GBps": b_c / (float(np.mean(ms_c)) * 1e-3) / 1e9}
        # the same with the kernel chosen on the device from the rows per group (CORAL_PATH_ADAPTIVE), and what
        # that mode costs where the streaming kernel stays the right choice (iid rows, M=60)
        head.set_path(lmhead.CORAL_PATH_ADAPTIVE)
        ms_ca, _, _, _, _ = time_steps(60, cfg.k_groups, extra_steps, 3, my_batches, rho=0.3)
        took_c = int(head.stats().path)
        ms_ia, _, _, _, _ = time_steps(60, cfg.k_groups, extra_steps, 3, my_batches)
        took_i = int(head.stats().path)
        head.set_path(lmhead.CORAL_PATH_AUTO)
        out["correlated_rows_M60_rho0.3"]["adaptive_us_per_step"] = float(np.mean(ms_ca)) * 1e3
        out["correlated_rows_M60_rho0.3"]["adaptive_path"] = took_c
        out["adaptive_iid_M60"] = {"us_per_step": float(np.mean(ms_ia)) * 1e3, "path": took_i}
        # extra: the paper's frequency-ordered contiguous grouping (Appendix B), modelled by a contiguous group map
        # and a Zipf-like prior on low-index groups in the gate (synth.py), against the random map above
        zcfg = cfg.with_(zipf_s=1.5)
        zhead = lmhead.LMHead(Wd, torch.from_numpy(synth.make_group_map(cfg, contiguous=True)),
                              dev_bf16(synth.make_w_gate(zcfg)), max_M=64, max_k_groups=cfg.k_groups,
                              max_k_tokens=cfg.k_tokens)
        zleg = []
        for M in (8, 60):
            ms_z, _, t_z, _, _ = time_steps(M, cfg.k_groups, extra_steps, 3, my_batches, zipf_s=1.5, on=zhead)
            b_z = float(np.mean([algorithmic_bytes(cfg.with_(M=M), u, M) for u in t_z]))
            zhead.set_path(lmhead.CORAL_PATH_ADAPTIVE)
            ms_za, _, _, _, _ = time_steps(M, cfg.k_groups, extra_steps, 3, my_batches, zipf_s=1.5, on=zhead)
            took_z = int(zhead.stats().path)
            zhead.set_path(lmhead.CORAL_PATH_AUTO)
            lmhead.coral_lmhead_set_hot_groups(zhead.handle, 4)     # the four most frequent groups stay in L2
            ms_zh, _, _, _, _ = time_steps(M, cfg.k_groups, extra_steps, 3, my_batches, zipf_s=1.5, on=zhead)
            lmhead.coral_lmhead_set_hot_groups(zhead.handle, 0)
            zleg.append({"M": M, "us_per_step": float(np.mean(ms_z)) * 1e3, "groups_touched_mean": float(np.mean(t_z)),
                         "hot4_persisting_us_per_step": float(np.mean(ms_zh)) * 1e3,
                         "GBps": b_z / (float(np.mean(ms_z)) * 1e-3) / 1e9,
                         "adaptive_us_per_step": float(np.mean(ms_za)) * 1e3, "adaptive_path": took_z})
        assert zhead.status() == 0
        zhead.close()
        out["contiguous_groups_zipf1.5"] = zleg
        # dense head on the same GPU: (i) this library with every group active, (ii) torch bf16 matmul comparator
        ms_d, _, t_d, _, _ = time_steps(cfg.M, cfg.N, extra_steps, 3, my_batches)
        dense_bytes = algorithmic_bytes(cfg, cfg.N, cfg.M)
        hd = dev_bf16(hb_bits[0])
        tms = []
        for i in range(extra_steps + 3):
            flush_l2(i)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            z = torch.matmul(hd, Wd.T).float()
            torch.topk(torch.log_softmax(z, dim=1), cfg.k_tokens, dim=1)
            b.record()
            torch.cuda.synchronize()
            if i >= 3:
                tms.append(a.elapsed_time(b))
        out["dense_head"] = {
            "all_groups_active_us": float(np.mean(ms_d)) * 1e3,
            "all_groups_active_GBps": dense_bytes / (float(np.mean(ms_d)) * 1e-3) / 1e9,
            "torch_matmul_logsoftmax_topk_us": float(np.mean(tms)) * 1e3,
            "grouped_vs_dense_speedup": float(np.mean(ms_d)) / (tot_ms / args.steps),
        }
        # large-M routed grouped GEMM (16 sequences x 60 tree nodes) on the tensor-core path, next to a dense
        # 960 x V x H bf16 GEMM by torch (comparator only)
        M_big = 960
        big = lmhead.LMHead(Wd, torch.from_numpy(gm), dev_bf16(Wg), max_M=M_big, max_k_groups=cfg.k_groups,
                            max_k_tokens=cfg.k_tokens)
        hbig = [dev_bf16(synth.make_hidden(cfg, M_big, batch=100 + b)) for b in range(2)]
        ids_b = torch.empty((M_big, cfg.k_tokens), dtype=torch.int32, device=dev)
        lps_b = torch.empty((M_big, cfg.k_tokens), dtype=torch.float32, device=dev)
        lmhead.coral_lmhead_set_kernel_timing(big.handle, True)
        t_step, t_head = [], []
        for i in range(13):
            flush_l2(i)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            lmhead.coral_lmhead_draft(big.handle, hbig[i & 1], cfg.k_groups, cfg.k_tokens, ids_b, lps_b, stream)
            b.record()
            torch.cuda.synchronize()
            if i >= 3:
                t_step.append(a.elapsed_time(b))
                t_head.append(lmhead.coral_lmhead_stage_ms(big.handle)[1])
        assert big.status() == 0
        st_big = big.stats()
        flops = 2.0 * cfg.H * (M_big * cfg.N + M_big * cfg.k_groups * cfg.v)
        pk = {}
        if os.path.exists(os.path.join(ROOT, "MEASURED_PEAKS.json")):
            with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
                pk = json.load(f)
        tf_sust = float(pk.get("bf16_tflops_sustained", 1400.0))
        tg = []
        for i in range(8):
            flush_l2(i)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            torch.matmul(hbig[0], Wd.T)
            b.record()
            torch.cuda.synchronize()
            if i >= 3:
                tg.append(a.elapsed_time(b))
        head_us = float(np.mean(t_head)) * 1e3
        out["large_m"] = {
            "M": M_big, "path": int(st_big.path), "groups_touched": int(st_big.groups_touched),
            "us_per_step": float(np.mean(t_step)) * 1e3, "grouped_gemm_stage_us": head_us,
            "GBps_whole_step": st_big.algorithmic_bytes / (float(np.mean(t_step)) * 1e-3) / 1e9,
            "GBps_grouped_gemm": st_big.weight_bytes / (head_us * 1e-6) / 1e9,
            "hbm_frac_grouped_gemm": st_big.weight_bytes / (head_us * 1e-6) / 1e9 / peak,
            "algorithmic_tflops_grouped_gemm": flops / (head_us * 1e-6) / 1e12,
            "tensor_frac_of_sustained_peak": flops / (head_us * 1e-6) / 1e12 / tf_sust,
            "tensor_frac_ceiling_at_hbm_roofline": flops / (st_big.weight_bytes / (peak * 1e9)) / 1e12 / tf_sust,
            "torch_dense_gemm_960xVxH_us": float(np.mean(tg)) * 1e3,
        }
        # what issuing the tensor-core path's MMAs costs by itself (tcgen05.mma of a CTA pair, 256 x n x 16, four
        # per commit as in the kernel's 64-column step, nothing loaded): ns per MMA for one and two issuing
        # threads, next to the time the tensor pipe needs at its nominal rate
        ns_out = torch.zeros(2, dtype=torch.int64, device=dev)
        issue = []
        for n_i, iss in ((32, 1), (128, 1), (256, 1), (32, 2), (128, 2), (256, 2)):
            for _ in range(2):
                lmhead.coral_lmhead_tc_issue_probe(big.handle, n_i, 4, iss, 2000, ns_out, stream)
                torch.cuda.synchronize()
            t_issue, t_done = [float(x) for x in ns_out.cpu().tolist()]
            issue.append({"n": n_i, "issuers": iss, "mmas_per_commit": 4,
                          "ns_per_round_of_one_issuer": t_issue / 2000.0, "ns_per_mma_over_all_issuers": t_done / 2000.0 / 4 / iss,
                          "ns_per_mma_at_nominal_tensor_rate": 128.0 * n_i * 16 / 4096.0 / 1.965})
        out["tc_issue_probe"] = issue
        assert big.status() == 0
        big.close()
        # supplementary points with more rows per group (240 and 480): the same path above the machine ridge
        supp = []
        for M_s in (1920, 3840):
            bg = lmhead.LMHead(Wd, torch.from_numpy(gm), dev_bf16(Wg), max_M=M_s, max_k_groups=cfg.k_groups,
                               max_k_tokens=cfg.k_tokens)
            h_s = dev_bf16(synth.make_hidden(cfg, M_s, batch=200))
            ids_s = torch.empty((M_s, cfg.k_tokens), dtype=torch.int32, device=dev)
            lps_s = torch.empty((M_s, cfg.k_tokens), dtype=torch.float32, device=dev)
            lmhead.coral_lmhead_set_kernel_timing(bg.handle, True)
            ts_, th_ = [], []
            for i in range(8):
                flush_l2(i)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                lmhead.coral_lmhead_draft(bg.handle, h_s, cfg.k_groups, cfg.k_tokens, ids_s, lps_s, stream)
                b.record()
                torch.cuda.synchronize()
                if i >= 3:
                    ts_.append(a.elapsed_time(b))
                    th_.append(lmhead.coral_lmhead_stage_ms(bg.handle)[1])
            assert bg.status() == 0
            fl_s = 2.0 * cfg.H * (M_s * cfg.N + M_s * cfg.k_groups * cfg.v)
            supp.append({"M": M_s, "us_per_step": float(np.mean(ts_)) * 1e3,
                         "grouped_gemm_stage_us": float(np.mean(th_)) * 1e3,
                         "tensor_frac_of_sustained_peak": fl_s / (float(np.mean(th_)) * 1e-3) / 1e12 / tf_sust})
            bg.close()
            del h_s, ids_s, lps_s
        out["large_m_supplementary"] = supp
        # the other shapes of the workload list (paper Table 1: H, V; Table 4: N, top-n), same cold-L2 protocol
        def torch_dense_us(Wt, hidden_bits, k_tokens):
            hd_ = dev_bf16(hidden_bits)
            tms_ = []
            for i in range(13):
                flush_l2(i)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                torch.topk(torch.log_softmax(torch.matmul(hd_, Wt.T).float(), dim=1), k_tokens, dim=1)
                b.record()
                torch.cuda.synchronize()
                if i >= 3:
                    tms_.append(a.elapsed_time(b))
            return float(np.mean(tms_)) * 1e3

        for name, cases in (("llama2_7b", [(1, 4), (8, 4), (60, 4), (8, 32)]),
                            ("qwen25_7b", [(60, 2), (60, 4), (60, 8), (60, 16), (60, 64)])):
            scfg = synth.CONFIGS[name]
            Ws = dev_bf16(synth.make_w_vocab(scfg))
            shead = lmhead.LMHead(Ws, torch.from_numpy(synth.make_group_map(scfg)), dev_bf16(synth.make_w_gate(scfg)),
                                  max_M=64, max_k_groups=scfg.N, max_k_tokens=scfg.k_tokens)
            pts = [timed_case(shead, scfg, M, kg, extra_steps) for M, kg in cases]
            for pt in pts:
                if pt["k_groups"] == scfg.N:
                    pt["dense_equivalent"] = True
                    pt["torch_matmul_logsoftmax_topk_us"] = torch_dense_us(
                        Ws, synth.make_hidden(scfg, pt["M"], batch=my_batches[0]), scfg.k_tokens)
            out[name] = {"shape": f"H={scfg.H} V={scfg.V} N={scfg.N} v={scfg.v} k_tokens={scfg.k_tokens}", "points": pts}
            assert shead.status() == 0
            shead.close()
            del Ws, shead
        # what an SM can take in: the do-nothing bulk-copy stream (one CTA per SM, 16 KiB copies) with 4, 8 and 13
        # copies in flight, from HBM (cold L2, the touched bytes of the headline call) and from L2 (a 48 MiB region
        # swept 9 times against once: the 8 extra sweeps hit L2)
        l2_region = 48 << 20
        ingest = []
        for fl in (4, 8, 13):
            t_h = copy_floor_us(head, k_bytes, in_flight=fl)
            t1 = copy_floor_us(head, l2_region, in_flight=fl, repeats=1, cold=False)
            t9 = copy_floor_us(head, l2_region, in_flight=fl, repeats=9, cold=False)
            ingest.append({"copies_in_flight_per_sm": fl, "hbm_to_smem_GBps": (int(k_bytes) // 16384 * 16384) / t_h / 1e3,
                           "l2_to_smem_GBps": 8.0 * l2_region / max(t9 - t1, 1e-3) / 1e3,
                           "l2_to_smem_GBps_per_sm": 8.0 * l2_region / max(t9 - t1, 1e-3) / 1e3 / torch.cuda.get_device_properties(dev).multi_processor_count})
        out["smem_ingest_probe"] = ingest
        # extra (second workload, training side): the CSRA objective of Eq. 2 on synthetic features - 4096
        # positions, keys = three other steps and the targets, D = 4096 - a tensor-bound contraction
        n_c, v_c, D_c = 4096, 4, cfg.H
        rng_c = np.random.default_rng([cfg.seed, 77])
        base_c = rng_c.standard_normal((n_c, D_c), dtype=np.float32)
        Qc = dev_bf16(synth.fp32_to_bf16_bits(0.6 * base_c + 0.8 * rng_c.standard_normal((n_c, D_c), dtype=np.float32)))
        Kc = torch.cat([dev_bf16(synth.fp32_to_bf16_bits(0.6 * base_c + 0.8 * rng_c.standard_normal((n_c, D_c), dtype=np.float32)))
                        for _ in range(v_c)])
        ws_c = torch.empty(lmhead.coral_csra_workspace_bytes(n_c, v_c, D_c), dtype=torch.uint8, device=dev)
        loss_c = torch.empty(1, dtype=torch.float32, device=dev)
        tc_, tt_ = [], []
        for i in range(8):
            flush_l2(i)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            lmhead.coral_csra_infonce(Qc, Kc, v_c, 0.07, ws_c, loss_c, stream=stream)
            b.record(stream)
            torch.cuda.synchronize()
            if i >= 3:
                tc_.append(a.elapsed_time(b))
        assert lmhead.coral_csra_status(ws_c) == 0
        for i in range(8):          # comparator: the same objective with torch ops (bf16 matmul, fp32 softmax)
            flush_l2(i)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            qn_ = torch.nn.functional.normalize(Qc.float(), dim=1).to(torch.bfloat16)
            kn_ = torch.nn.functional.normalize(Kc.float(), dim=1).to(torch.bfloat16)
            lg_ = torch.matmul(qn_, kn_.T).float() / 0.07
            idx_ = torch.arange(n_c, device=dev)
            pos_ = torch.stack([lg_[idx_, idx_ + s_ * n_c] for s_ in range(v_c)], 1).mean(1)
            loss_t = (torch.logsumexp(lg_, dim=1) - pos_).mean()
            b.record()
            torch.cuda.synchronize()
            if i >= 3:
                tt_.append(a.elapsed_time(b))
        fl_c = 2.0 * n_c * (n_c * v_c) * D_c
        out["csra_infonce"] = {"n": n_c, "views": v_c, "D": D_c, "us": float(np.mean(tc_)) * 1e3,
                               "tflops": fl_c / (float(np.mean(tc_)) * 1e-3) / 1e12,
                               "tensor_frac_of_sustained_peak": fl_c / (float(np.mean(tc_)) * 1e-3) / 1e12 / tf_sust,
                               "loss": float(loss_c.item()), "torch_ops_us": float(np.mean(tt_)) * 1e3,
                               "torch_ops_loss": float(loss_t.item())}
        del Qc, Kc, ws_c
        out["clocks"] = sampler.stop()
        # CPU oracle on the host cores: whole steps of the same workload, bounded
        o_steps = 3
        times, o_touched, cores = run_oracle_baseline(cfg, W, gm, Wg, hb_bits, o_steps, warmup=1)
        o_bytes = sum(algorithmic_bytes(cfg, u, cfg.M) for u in o_touched)
        out["cpu_baseline"] = {"value": o_bytes / sum(times) / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
                               "sample": f"{o_steps} whole draft steps of the same workload (M={cfg.M})",
                               "us_per_step": sum(times) / o_steps * 1e6}
    if "clocks" not in out:
        out["clocks"] = sampler.stop()
    if rank == 0:
        print(json.dumps(out))
    head.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
