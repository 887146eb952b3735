#!/usr/bin/env python
"""Benchmark of the LSA layer-group forward (indexer + sparse attention, one index set reused by R layers).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config cfg3] [--impl reference]

A step is one lsa_layer_group call over the whole synthetic workload (coarse page scores, page
top-M, fine scores, top-K_sparse, conversion, R attention layers).  Default workload: cfg3, the 128K
prefill the headline metric is quoted on.  Prints one JSON line (rank 0).  With N > 1 every rank runs
its own independent sequence (weak scaling, no data-path collective).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "LSA layer-group tokens/sec (128K prefill)"
UNIT = "tokens/s"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", default="cfg3")
    ap.add_argument("--impl", default="lsa", choices=["lsa", "reference"])
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--cpu-queries", type=int, default=256,
                    help="queries the CPU oracle is timed on for the cpu_baseline leg (about 10 s of host work at cfg3)")
    ap.add_argument("--no-decode", action="store_true", help="skip the cfg4 decode side measurement of the default run")
    ap.add_argument("--phase", default="group", choices=["group", "index"],
                    help="group: whole lsa_layer_group step; index: indexer only (no attention tensors are allocated; for profiling)")
    ap.add_argument("--attn-tc", type=int, default=-1, help="override LSA_TUNE_ATTN_TC (0 or 1)")
    ap.add_argument("--seq-len", type=int, default=0, help="override the prefill length L of the config (profiling sweeps)")
    ap.add_argument("--q-tail", type=int, default=0, help="score only the last N queries of the sequence")
    ap.add_argument("--keep-pages", type=int, default=0, help="override M, the pages recalled by the coarse stage (recall-budget sweeps)")
    ap.add_argument("--batch", type=int, default=0, help="override the decode batch of the config (small profiling captures)")
    ap.add_argument("--layers", type=int, default=0, help="override R, the layers per group (small profiling captures)")
    ap.add_argument("--flat", action="store_true", help="hi_enable = 0: flat indexer (Eq. 7) instead of the hierarchy")
    ap.add_argument("--attn-split", type=int, default=0, help="override LSA_TUNE_ATTN_SPLIT (decode row splits)")
    ap.add_argument("--attn-pv-wait", type=int, default=-1, help="override LSA_TUNE_ATTN_PV_WAIT (0 or 1)")
    ap.add_argument("--attn-gather", type=int, default=-1, help="override LSA_TUNE_ATTN_GATHER (0: cp.async rows, 1: TMA gather4)")
    ap.add_argument("--fine-paged-tc", type=int, default=-1, help="override LSA_TUNE_FINE_PAGED_TC (0, 1 or 2)")
    ap.add_argument("--coarse-groups", type=int, default=0, help="override LSA_TUNE_COARSE_GROUPS (1 or 2)")
    return ap.parse_args()


# ------------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons every 200 ms while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def __exit__(self, *exc):
        if self.proc is not None:
            time.sleep(0.25)
            self.proc.terminate()          # the exact child started above
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
            self.thread.join(timeout=2)

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
# algorithmic work
# ------------------------------------------------------------------------------------------------
def attn_rows_per_query(cfg, t):
    n_sink = min(cfg.S, t + 1)
    n_win = t - max(cfg.S, t - cfg.W + 1) + 1
    n_sp = min(cfg.Ksp, max(0, t - cfg.W - cfg.S + 1))
    return n_sink + max(0, n_win) + n_sp


def attn_flops_per_launch(cfg, positions):
    """2*H*(d_qk+d_v) flops per (query, attended row): QK^T and PV of Eq. 3, one layer."""
    return float(sum(2 * cfg.H * (cfg.d_qk + cfg.d_v) * attn_rows_per_query(cfg, int(t)) for t in positions))


def attn_bytes_per_launch(cfg, positions):
    """Decode: every attended cache row is read once, plus q and out."""
    rows = sum(attn_rows_per_query(cfg, int(t)) for t in positions)
    return float(rows * cfg.d_qk * 2 + len(positions) * cfg.H * (cfg.d_qk + cfg.d_v) * 2)


# DRAM traffic of one attention launch, from the ncu capture of the same kernel on cfg3 cut to 16384 queries
# (profiles/sparse_attn_tc_cfg3_16k.md: dram__bytes_read.sum 1.344671 GB + dram__bytes_write.sum 1.047908 GB).
# Traffic there is q + out (the KV latent stays in L2), so it scales with the number of queries of a launch.
NCU_ATTN_DRAM_BYTES_PER_QUERY = (1.344671e9 + 1.047908e9) / 16384
# Decode: DRAM bytes of one attention launch per sequence, from the ncu capture at batch 16
# (profiles/sparse_attn_tc_cfg4_decode_batch16.md: dram__bytes_read.sum 43.95 MB + dram__bytes_write.sum 0.47 MB).
NCU_DECODE_ATTN_DRAM_BYTES_PER_SEQ = (43949568 + 472832) / 16


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": d["hbm_gbs"], "tensor_tflops": d["bf16_tflops_sustained"], "source": "measured"}
    return {"hbm_gbs": 6650.0, "tensor_tflops": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------------------------------------
# CPU oracle legs
# ------------------------------------------------------------------------------------------------
CORES_NOTE = ("threads of the BLAS pool behind numpy's matrix products; the oracle walks over the sampled queries "
              "one after another in a single Python process")


def oracle_sample(cfg, wl, n_queries, seed=0):
    """Times the oracle (as it stands) on n_queries sampled queries of the workload: selection plus the R
    attention layers.  Returns (queries per second, seconds, threads used)."""
    import numpy as np
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import parity_util as pu
    from oracle import reference_run as ref
    try:
        from threadpoolctl import threadpool_info
        threads = max([i.get("num_threads", 1) for i in threadpool_info()] or [1])
    except Exception:
        threads = os.cpu_count() or 1
    rng = np.random.default_rng(seed)
    kw = dict(P=cfg.P, B=cfg.B, M=cfg.M, Ksp=cfg.Ksp, S=cfg.S, W=cfg.W)
    if cfg.mode == "prefill":
        caches = ref.HostCaches(pu.to_np(wl.keys["k"]), pu.to_np(wl.keys["scale"]) if "scale" in wl.keys else None,
                                [pu.to_np(k) for k in wl.k], [pu.to_np(v) for v in wl.v], cfg.B, n_key=wl.n_key)
        qs = [int(x) for x in rng.integers(wl.q_pos0, wl.q_pos0 + wl.n_query, n_queries)]
        host = [(t, pu.to_np(wl.q_idx[t - wl.q_pos0]), pu.to_np(wl.w[t - wl.q_pos0]),
                 [pu.to_np(q[t - wl.q_pos0]) for q in wl.q]) for t in qs]
        t0 = time.perf_counter()
        for t, qi, w, ql in host:
            sparse, _ = ref.select_query(t, qi, w, caches, hi_enable=cfg.hi_enable, **kw)
            ref.attend_query(t, ql, caches, sparse, S=cfg.S, W=cfg.W, sm_scale=cfg.sm_scale, d_v=cfg.d_v)
        dt = time.perf_counter() - t0
        return len(host) / dt, dt, threads
    # decode: whole sequences
    seqs = [(seed + i) % cfg.batch for i in range(min(n_queries, cfg.batch))]
    dt = 0.0
    for b in seqs:
        caches, t = pu.decode_caches(wl, b)            # host copies: not part of the timed work
        qi, w, ql = pu.to_np(wl.q_idx[b]), pu.to_np(wl.w[b]), [pu.to_np(q[b]) for q in wl.q]
        t0 = time.perf_counter()
        sparse, _ = ref.select_query(t, qi, w, caches, hi_enable=cfg.hi_enable, **kw)
        ref.attend_query(t, ql, caches, sparse, S=cfg.S, W=cfg.W, sm_scale=cfg.sm_scale, d_v=cfg.d_v)
        dt += time.perf_counter() - t0
    return len(seqs) / dt, dt, threads


# ------------------------------------------------------------------------------------------------
def main():
    args = parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    from paper_2608_01662_b200.configs import CONFIGS
    cfg = CONFIGS[args.config]
    decode = cfg.mode == "decode"
    metric = "LSA layer-group decode us/step" if decode else METRIC
    unit = "us/step" if decode else UNIT

    if args.impl == "reference":
        if rank != 0:
            return
        run_reference(args, cfg, metric, unit, decode)
        return

    import torch
    import torch.distributed as dist
    from paper_2608_01662_b200 import build
    from paper_2608_01662_b200.workload import make_workload
    from paper_2608_01662_b200.distributed import job_throughput, max_over_ranks

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()

    # prefill at cfg5 size keeps only one 16384-query chunk of per-query tensors resident
    kw = {}
    if not decode and cfg.q_chunk and cfg.L > 262144:
        kw = dict(q_pos0=cfg.L - cfg.q_chunk, n_query=cfg.q_chunk)
    if args.seq_len:
        cfg = cfg.replace(L=args.seq_len)
    if args.keep_pages:
        cfg = cfg.replace(M=args.keep_pages)
    if args.batch:
        cfg = cfg.replace(batch=args.batch)
    if args.layers:
        cfg = cfg.replace(R=args.layers)
    if args.flat:
        cfg = cfg.replace(hi_enable=False)
    if args.q_tail:
        kw = dict(q_pos0=cfg.L - args.q_tail, n_query=args.q_tail)
    if args.phase == "index":
        cfg = cfg.replace(R=0)
        args.no_e2e = True
    wl = make_workload(cfg, dev, with_lse=False, **kw)
    if args.phase == "index":
        wl.step = wl.index
    wl.prepare()
    if args.coarse_groups:
        wl.ctx.tune(0, args.coarse_groups)
    if args.attn_tc >= 0:
        wl.ctx.tune(1, args.attn_tc)
    if args.attn_split:
        wl.ctx.tune(2, args.attn_split)
    if args.attn_pv_wait >= 0:
        wl.ctx.tune(3, args.attn_pv_wait)
    if args.attn_gather >= 0:
        wl.ctx.tune(4, args.attn_gather)
    if args.fine_paged_tc >= 0:
        wl.ctx.tune(5, args.fine_paged_tc)
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        wl.step()
    barrier()
    st = wl.ctx.status()
    assert st == 0, f"device status {st}"

    stream = torch.cuda.current_stream(dev)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    wl.ctx.profile_enable(not decode)      # event pairs around each kernel class (see lsa_profile_enable)
    n0 = wl.ctx.launch_count()
    with ClockSampler(local_rank) as clocks:
        barrier()
        ev0.record(stream)
        for _ in range(args.steps):
            wl.step()
        ev1.record(stream)
        barrier()
    ms = ev0.elapsed_time(ev1)
    launches = wl.ctx.launch_count() - n0
    prof = wl.ctx.profile_read() if not decode else None
    wl.ctx.profile_enable(False)
    if decode:
        # the per-kernel event pairs would perturb a ~100 us step: measure them in a second pass
        wl.ctx.profile_enable(True)
        for _ in range(args.steps):
            wl.step()
        prof = wl.ctx.profile_read()
        wl.ctx.profile_enable(False)

    ms_per_step = max_over_ranks(ms, dev) / args.steps          # the slowest rank bounds the job
    value = ms_per_step * 1e3 if decode else job_throughput(wl.units(), world, ms_per_step)

    if rank != 0:
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel: sparse attention
    peaks = measured_peaks()
    import numpy as np
    if decode:
        positions = (wl.ctx_len.cpu().numpy().astype(np.int64) - 1)
    else:
        positions = np.arange(wl.q_pos0, wl.q_pos0 + wl.n_query)
    attn_ms, attn_n = prof["sparse_attn"]
    roofline = None
    if attn_n > 0:
        dur_s = attn_ms / attn_n * 1e-3
        if decode:
            roofline = decode_attn_roofline(cfg, prof, decode_attn_launch_us(wl), positions, peaks)
        else:
            a = attn_flops_per_launch(cfg, positions) / dur_s / 1e12
            roofline = {"kernel": "sparse_attn_tc_kernel" if cfg.H == 64 else "sparse_attn_kernel", "bound": "tensor", "achieved": a,
                        "peak": peaks["tensor_tflops"], "unit": "TFLOP/s", "frac": a / peaks["tensor_tflops"],
                        "traffic": NCU_ATTN_DRAM_BYTES_PER_QUERY * len(positions) if cfg.H == 64 else None,
                        "traffic_source": "ncu capture at 16384 queries, scaled by queries per launch",
                        "algorithmic_bytes": float(len(positions)) * cfg.H * (cfg.d_qk + cfg.d_v) * 2,
                        "peak_source": peaks["source"], "launch_ms": attn_ms / attn_n}
    kernels = {k: {"ms_per_step": v[0] / args.steps, "launches_per_step": v[1] / args.steps}
               for k, v in prof.items() if v[1] > 0}

    # ---- end to end through the host-buffer entry point (prefill only)
    e2e = None
    if not args.no_e2e and not decode and world == 1:
        e2e = run_e2e(args, cfg, wl, dev)

    cpu = None
    if not args.no_cpu:
        v, secs, threads = oracle_sample(cfg, wl, args.cpu_queries)
        cpu = {"value": (1e6 / v) * cfg.batch if decode else v, "unit": unit, "cores": threads, "kind": "oracle",
               "cores_note": CORES_NOTE,
               "sample": f"{args.cpu_queries if not decode else min(args.cpu_queries, cfg.batch)} "
                         f"{'sequences' if decode else 'uniformly sampled queries'} of the same workload, selection + "
                         f"{cfg.R} attention layers each, {secs:.1f} s"
                         + ("; value extrapolated to the batch of %d" % cfg.batch if decode else "")}

    # ---- the metric's second half: decode us/step on cfg4, measured in the same run (single GPU, default workload)
    queries_per_step = wl.units()
    decode_line = None
    if not decode and world == 1 and args.config == "cfg3" and args.phase == "group" and not args.no_decode and not (args.seq_len or args.q_tail or args.flat):
        del wl
        import gc
        gc.collect()
        torch.cuda.empty_cache()
        decode_line = measure_decode(CONFIGS["cfg4"], dev, peaks)

    line = {
        "metric": metric, "value": value, "unit": unit, "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": not decode,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": config_dict(cfg, queries_per_step),
        "clocks": clocks.summary(), "gpu_launches": int(launches), "kernels": kernels,
        "roofline": with_nominal(roofline), "e2e": e2e, "cpu_baseline": cpu, "decode": decode_line,
    }
    print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def config_dict(cfg, queries_per_step):
    """The `config` object of the JSON line; both arms print the same keys and values for the same workload."""
    decode = cfg.mode == "decode"
    return {"workload": cfg.name, "mode": cfg.mode, "L": cfg.L, "batch": cfg.batch, "R": cfg.R,
            "indexer_keys": cfg.key_dtype, "P": cfg.P, "B": cfg.B, "M": cfg.M, "K_sparse": cfg.Ksp,
            "K_sink": cfg.S, "K_swa": cfg.W, "queries_per_step": int(queries_per_step),
            "l2": "inputs larger than L2 (per-layer q and out are GBs); no flush" if not decode
                  else "KV pools are GBs per layer, far larger than L2; no flush"}


NOMINAL_BF16_TFLOPS, NOMINAL_HBM_GBS = 2250.0, 8000.0   # dense bf16 and HBM3e data-sheet figures, for context


def with_nominal(roofline):
    """Adds the fraction of the nominal (data-sheet) peak beside the fraction of the measured one."""
    if roofline is not None:
        nominal = NOMINAL_HBM_GBS if roofline["bound"] == "hbm" else NOMINAL_BF16_TFLOPS
        roofline["peak_nominal"] = nominal
        roofline["frac_of_nominal"] = roofline["achieved"] / nominal
    return roofline


def decode_attn_roofline(cfg, prof, launch_us, positions, peaks):
    """Decode roofline of one attention launch (one layer of the group; the layers run one after another because each
    layer's query depends on the layer before).  `launch_us` comes from one event pair around many back-to-back
    launches (decode_attn_launch_us); `launch_us_in_step` is the library's event pair around each launch inside
    lsa_layer_group, which adds front-end time to a launch this short."""
    attn_ms, attn_n = prof["sparse_attn"]
    bytes_per_launch = attn_bytes_per_launch(cfg, positions)
    a = bytes_per_launch / (launch_us * 1e-6) / 1e9
    return with_nominal({"kernel": "sparse_attn_tc_kernel", "bound": "hbm", "achieved": a, "peak": peaks["hbm_gbs"],
                         "unit": "GB/s", "frac": a / peaks["hbm_gbs"],
                         "traffic": NCU_DECODE_ATTN_DRAM_BYTES_PER_SEQ * cfg.batch,
                         "traffic_source": "ncu capture at batch 16, scaled by sequences per launch",
                         "algorithmic_bytes": bytes_per_launch, "peak_source": peaks["source"], "launch_us": launch_us,
                         "launch_us_in_step": attn_ms / attn_n * 1e3,
                         "timing": "one event pair around 10 x R back-to-back launches, each layer on its own cache"})


def decode_attn_launch_us(wl, rounds=10):
    """Average device time of one decode attention launch (a6 with its split merge), timed with one CUDA event pair
    around rounds x R back-to-back lsa_sparse_attn calls on the physical row lists lsa_convert wrote.  Each layer
    has its own multi-GB KV pool, so no launch finds its rows in L2.  An event pair per launch (the per-kernel
    profile) adds several microseconds of front-end time to a launch this short."""
    import torch
    cfg, dev = wl.cfg, wl.device
    ld = cfg.S + cfg.Ksp + cfg.W
    rows = torch.empty((cfg.batch, ld), dtype=torch.int32, device=dev)
    n_rows = torch.empty((cfg.batch,), dtype=torch.int32, device=dev)
    wl.ctx.convert(wl.sparse_idx, wl.n_sparse, 0, cfg.batch, rows, n_rows, None, wl.page_table, wl.ctx_len)

    def one_round():
        for r in range(cfg.R):
            wl.ctx.sparse_attn(wl.q[r], wl.k[r], wl.v[r], wl.sparse_idx, wl.n_sparse, 0, cfg.batch, 0, wl.out[r], None,
                               rows, n_rows, wl.ctx_len, cfg.batch)
    one_round()
    stream = torch.cuda.current_stream(dev)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for _ in range(rounds):
        one_round()
    ev1.record(stream)
    torch.cuda.synchronize()
    return ev0.elapsed_time(ev1) / (rounds * cfg.R) * 1e3


def measure_decode(cfg, dev, peaks, steps=50, warmup=10):
    """cfg4: one lsa_layer_group call per step for the 64-sequence paged batch; returns the side-line dict."""
    import numpy as np
    import torch
    from paper_2608_01662_b200.workload import make_workload
    grow = 32                                  # pages mapped ahead for the running loop below; the step itself is cfg4's
    wl = make_workload(cfg.replace(ctx_grow=grow), dev, with_lse=False)
    wl.prepare()
    for _ in range(warmup):
        wl.step()
    torch.cuda.synchronize()
    st = wl.ctx.status()
    assert st == 0, f"device status {st}"
    stream = torch.cuda.current_stream(dev)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n0 = wl.ctx.launch_count()
    ev0.record(stream)
    for _ in range(steps):
        wl.step()
    ev1.record(stream)
    torch.cuda.synchronize()
    us = ev0.elapsed_time(ev1) / steps * 1e3
    launches = (wl.ctx.launch_count() - n0) // steps
    wl.ctx.profile_enable(True)       # second pass: event pairs would perturb a step this short
    for _ in range(steps):
        wl.step()
    prof = wl.ctx.profile_read()
    wl.ctx.profile_enable(False)
    positions = wl.ctx_len.cpu().numpy().astype(np.int64) - 1
    roofline = decode_attn_roofline(cfg, prof, decode_attn_launch_us(wl), positions, peaks)
    # running loop: every step first appends one token per sequence (indexer key quantised, sub-block mean updated,
    # one latent row per layer), then runs the group on the grown caches
    k_new = (torch.randn((cfg.batch, cfg.d_I), device=dev) / cfg.d_I ** 0.5).to(torch.bfloat16)
    kv_new = [torch.randn((cfg.batch, cfg.d_qk), device=dev).to(torch.bfloat16) for _ in range(cfg.R)]
    wl.ctx.profile_enable(True)
    ev0.record(stream)
    for _ in range(grow):
        wl.ctx.append(k_new, wl.keys["k"], wl.keys.get("scale"), wl.kmean, wl.page_table, wl.ctx_len, wl.ctx_len, kv_new, wl.k)
        wl.step()
    ev1.record(stream)
    torch.cuda.synchronize()
    loop_prof = wl.ctx.profile_read()
    wl.ctx.profile_enable(False)
    st = wl.ctx.status()
    assert st == 0, f"device status {st}"
    running = {"steps": grow, "us_per_step_with_event_pairs": ev0.elapsed_time(ev1) / grow * 1e3,
               "append_us": loop_prof["block_means"][0] / grow * 1e3,
               "what": "lsa_append (key quantised, sub-block mean updated, R latent rows stored) + lsa_layer_group, "
                       "contexts growing by one token per step"}
    return {"metric": "LSA layer-group decode us/step", "value": us, "unit": "us/step", "higher_is_better": False,
            "steps": steps, "gpu_launches_per_step": int(launches),
            "config": {"workload": cfg.name, "batch": cfg.batch, "R": cfg.R, "ctx": [cfg.ctx_lo, cfg.ctx_hi],
                       "l2": "KV pools are GBs per layer, far larger than L2; no flush"},
            "kernels_us_per_step": {k: v[0] / steps * 1e3 for k, v in prof.items() if v[1] > 0},
            "roofline": roofline,
            "running_loop": running}


def run_e2e(args, cfg, wl, dev):
    """Same metric through lsa_layer_group_host: per-query tensors start in pinned host memory, results
    end there; the caches stay resident (they are state of the sequence, not inputs of the step)."""
    import torch
    from paper_2608_01662_b200 import binding
    n = wl.n_query
    q_idx_h = wl.q_idx.cpu().pin_memory()
    w_h = wl.w.cpu().pin_memory()
    q_h = [q.cpu().pin_memory() for q in wl.q]
    out_h = [torch.empty(o.shape, dtype=o.dtype).pin_memory() for o in wl.out]
    sq = 4096
    nbytes = binding.host_stage_bytes(wl.params, sq)
    stage = [torch.empty(nbytes, dtype=torch.uint8, device=dev) for _ in range(2)]
    h2d = q_idx_h.numel() * 2 + w_h.numel() * 4 + sum(q.numel() * 2 for q in q_h)
    d2h = sum(o.numel() * 2 for o in out_h)

    def step():
        wl.ctx.layer_group_host(q_idx_h, w_h, wl.keys["k"], wl.keys.get("scale"), wl.kmean, wl.q_pos0, n, wl.n_key, q_h, wl.k,
                                wl.v, out_h, sq, stage)
    step()
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream(dev)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for _ in range(args.e2e_steps):
        step()
    ev1.record(stream)
    torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1) / args.e2e_steps
    # the device-resident run must have produced the same bytes: every row of every layer, compared on the device in
    # pieces of 8192 queries (a whole layer's output is 8 GiB at cfg3)
    same = True
    for oh, o in zip(out_h, wl.out):
        for i in range(0, n, 8192):
            same = same and torch.equal(oh[i:i + 8192].to(dev, non_blocking=False), o[i:i + 8192])
    return {"value": n / (ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
            "ms_per_step": ms, "steps": args.e2e_steps, "matches_device_run": bool(same),
            "api": "lsa_layer_group_host, pinned host buffers, 4096-query passes"}


def run_reference(args, cfg, metric, unit, decode):
    """The oracle as the reference arm: each step times it on a bounded sample of the workload."""
    import torch
    from paper_2608_01662_b200.workload import make_workload
    dev = torch.device("cuda:0") if torch.cuda.is_available() else torch.device("cpu")
    # the sample's inputs are drawn by the same generators; only the sampled queries are scored
    n_q = 4 if not decode else 1
    kw = {}
    if not decode:
        kw = dict(q_pos0=max(0, cfg.L - 4096), n_query=min(cfg.L, 4096))   # late queries: full-size candidate sets
    wl = make_workload(cfg, dev, with_lse=False, make_ctx=False, **kw)
    # queries one step of the GPU arm processes on this config (the sample below is a bounded part of them)
    units = cfg.batch if decode else (cfg.q_chunk if cfg.q_chunk and cfg.L > 262144 else cfg.L)
    vals, secs_all, threads = [], 0.0, 1
    for i in range(max(0, args.warmup) + args.steps):
        v, secs, threads = oracle_sample(cfg, wl, n_q, seed=i)
        if i >= args.warmup:
            vals.append(v)
            secs_all += secs
    v = len(vals) / sum(1.0 / x for x in vals)              # total queries / total time
    value = (1e6 / v) * cfg.batch if decode else v
    sample = (f"{n_q} sampled late queries per step, selection + {cfg.R} attention layers each" if not decode
              else "1 sequence per step, extrapolated to the batch")
    print(json.dumps({
        "impl": "reference", "metric": metric, "value": value, "unit": unit, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": secs_all / max(1, args.steps) * 1e3, "higher_is_better": not decode,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(cfg, units),
        "cpu_baseline": {"value": value, "unit": unit, "cores": threads, "kind": "oracle", "sample": sample,
                         "cores_note": CORES_NOTE},
        "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


if __name__ == "__main__":
    main()
