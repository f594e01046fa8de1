#!/usr/bin/env python
"""Benchmark of the DReSD retrieval hot path on B200 (one JSON line on stdout).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload NAME] [--rows N]

A *step* is one dresd_retrieve() call -- query preprocessing, scoring of every
key, top-n selection, merge and continuation gather -- for one decode step of
the workload (batch 1 on the 10M x 256 fp16 datastore by default).  `value` is
queries/s with everything resident in HBM; `e2e` is the same through the
host-buffer entry point, copies included.  With --gpus N > 1 every rank (one
process per GPU) serves its own query stream against its own replica of the
datastore; there is no data-path collective, only the timing barrier.  Started
plainly (`python bench.py --gpus N`), the script launches its N ranks itself
through torch.distributed.run; started under torchrun it is one of them.

`--impl reference` times the CPU oracle (plain float64 brute force) on the
host cores, on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2502_15572_b200 import synth  # noqa: E402

METRIC = "retrieval queries/s at 10M x 256 fp16, batch 1 (exact top-10 + 10-token drafts)"
TRAFFIC_RATIO = 1.004     # measured DRAM traffic / algorithmic key bytes (profiles/scan_*_2M_rows.md)
N_QUERIES = 1000          # distinct single queries cycled through (config 2: 1,000 sequential queries)


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2_decode_b1_f16", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--rows", type=int, default=None, help="override N (debugging; not a bench value)")
    ap.add_argument("--batch", type=int, default=None, help="override B (debugging; not a bench value)")
    ap.add_argument("--top-n", type=int, default=None, help="override top_n (debugging; not a bench value)")
    ap.add_argument("--shard-rows", action="store_true",
                    help="N > 1: the rows of ONE datastore are split over the ranks (every rank answers every query "
                         "from its rows, the per-rank results are all-gathered and merged on the device): strong scaling. "
                         "Default: every rank holds a replica and serves its own slice of the query stream (weak)")
    ap.add_argument("--oracle-queries", type=int, default=3)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--build-keys", action="store_true",
                    help="time dresd_build_keys (datastore-side Eq. 1 -> v W -> Eq. 2, a tensor-bound GEMM) instead")
    ap.add_argument("--fit-zscore", action="store_true",
                    help="time dresd_fit_zscore (Eq. 1 statistics over --rows x --d-in bf16 embeddings) instead")
    ap.add_argument("--single-cta", action="store_true",
                    help="--build-keys: one CTA per tile instead of CTA pairs (cta_group::2)")
    ap.add_argument("--no-zscore", action="store_true",
                    help="--build-keys: projection and Eq. 2 only (W is exact in 16 bits: one tensor-core term)")
    ap.add_argument("--d-in", type=int, default=4096)
    ap.add_argument("--d-out", type=int, default=256)
    ap.add_argument("--first-token-filter", action="store_true",
                    help="time dresd_retrieve_filtered: each query wants the first stored token of its source row")
    ap.add_argument("--sorted-store", action="store_true",
                    help="with --first-token-filter: rows sorted by first stored token and indexed, so that a call "
                         "scans only the rows of its queries' tokens (same result as the filtered full scan)")
    ap.add_argument("--probe", type=int, default=1, help="probe-pass tile stride (0 off, 1 default)")
    ap.add_argument("--quantised", type=int, default=0, metavar="M",
                    help="candidates by approximate score over an 8-bit (E4M3) copy of the keys, exact re-ranking "
                         "of the M best (top_n <= M <= 32); reports recall against the exact path")
    ap.add_argument("--keys-as-m", type=int, default=0, choices=[0, 1],
                    help="1: keep the keys as the M operand of the tcgen05 kernel also for 33-64 queries")
    ap.add_argument("--scan-path", type=int, default=0, choices=[0, 1, 2],
                    help="0 auto, 1 streaming mma.sync kernel, 2 tcgen05 kernel (16-bit keys)")
    return ap.parse_args()


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            j = json.load(f)
        return float(j["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, copy read+write)"
    return 6650.0, "fallback (earlier measurement on this pool)"


def metric_name(cfg):
    if cfg["name"] == "c2_decode_b1_f16" and cfg["N"] == synth.WORKLOADS["c2_decode_b1_f16"]["N"]:
        return METRIC
    return (f"retrieval queries/s at {cfg['N']} x {cfg['d']} {cfg['dtype']}, batch {cfg['B']} "
            f"(exact top-{cfg['top_n']} + {cfg['draft_len']}-token drafts)")


def workload_config(cfg):
    return {"workload": cfg["name"], "N": cfg["N"], "d": cfg["d"], "d_in": cfg.get("d_in", cfg["d"]),
            "key_dtype": cfg["dtype"],
            "batch": cfg["B"], "top_n": cfg["top_n"], "draft_len": cfg["draft_len"],
            "first_token_filter": bool(cfg.get("filter_on", False)),
            "multi_gpu": cfg.get("multi_gpu", "replicas: every rank serves its own slice of the query stream"),
            "sorted_by_first_token": "rows_scanned_per_step_mean" in cfg,
            "rows_scanned_per_step_mean": cfg.get("rows_scanned_per_step_mean"),
            "mixture_components": cfg["C"], "query_noise_sigma": cfg["sigma"], "seed": cfg["seed"],
            "l2": "keys are %.2f GB per step, far larger than the 126 MB L2: no flush needed"
                  % (cfg["N"] * cfg["d"] * synth.DTYPE_BYTES[cfg["dtype"]] / 1e9)}


def workload_of(args):
    cfg = dict(synth.WORKLOADS[args.workload], name=args.workload)
    if args.rows:
        cfg["N"] = args.rows
    if args.batch:
        cfg["B"] = args.batch
    if args.top_n:
        cfg["top_n"] = args.top_n
    cfg["n_queries"] = N_QUERIES if cfg["B"] == 1 else cfg["B"] * 16
    return cfg


def make_inputs(args):
    cfg = workload_of(args)
    keys, toks = synth.make_store(cfg["seed"], cfg["N"], cfg["d"], cfg["C"], cfg["dtype"], cfg["stored_len"])
    nq = cfg["n_queries"]
    if "d_in" in cfg:       # queries arrive at the LLM's hidden width and are projected (Section 3.3)
        _, _, W = synth.make_preprocess(cfg["proj_seed"], cfg["d_in"], cfg["d"], cfg["dtype"])
        cfg["W"] = W
        q = synth.make_hidden_queries(cfg["seed"] + 100, nq, cfg["d_in"], cfg["dtype"], scale=1.0, offset=0.0)
    else:
        q, src = synth.make_queries(cfg["seed"] + 100, keys, cfg["dtype"], nq, cfg["sigma"])
        cfg["first_tokens"] = np.ascontiguousarray(toks[src, 0])      # the token the LLM would have produced
        if args.sorted_store:
            keys, toks = synth.sort_by_first_token(keys, toks)
    return cfg, keys, toks, q


def device_inputs(args, rank, world, device="cuda"):
    """The workload as tensors on `device` for this rank: ``(cfg, keys, tokens, queries, shard,
    host)``.  One rank: generated here.  Replicas (N ranks, default): rank 0 generates the
    datastore once and broadcasts it -- the other ranks do no host-side generation.  Sharded
    rows (--shard-rows): every rank generates only ITS rows (the generator is seeded per
    65,536-row chunk) and the queries' source rows are collected from their owners, so that
    all ranks hold the same queries.  `host` = the numpy arrays where this rank has them
    (rank 0 of a replica run, the one rank of a 1-GPU run), else None."""
    import torch
    from paper_2502_15572_b200 import dist_util

    def store_tensor(t, dtype):
        return t.view(torch.bfloat16) if dtype == "bf16" else t.view(torch.float16) if dtype == "f16" else t

    def upload(a, dtype):
        if a.dtype in (np.float16, np.uint16):
            a = a.view(np.int16)
        return store_tensor(torch.from_numpy(np.ascontiguousarray(a)).to(device), dtype)

    if args.shard_rows and world > 1:
        cfg = workload_of(args)
        if "d_in" in cfg:
            raise SystemExit("--shard-rows: workloads with a projection are timed on replicas")
        dtype = cfg["dtype"]
        shard = dist_util.shard_rows(cfg["N"], rank, world)
        keys, toks = synth.make_store(cfg["seed"], cfg["N"], cfg["d"], cfg["C"], dtype, cfg["stored_len"],
                                      rows=(shard.start, shard.stop))
        src = synth.query_sources(cfg["seed"] + 100, cfg["N"], cfg["n_queries"])
        src_keys = dist_util.collect_rows(keys, shard.start, src, device=device)
        q = synth.queries_from_rows(cfg["seed"] + 100, src_keys, dtype, cfg["N"], cfg["sigma"])
        return cfg, upload(keys, dtype), torch.from_numpy(toks).to(device), upload(q, dtype), shard, None
    host = None
    if rank == 0:
        cfg, keys, toks, q = make_inputs(args)
        host = (keys, toks, q)
    else:
        cfg, keys, toks, q = workload_of(args), None, None, None
        if "d_in" in cfg:
            _, _, cfg["W"] = synth.make_preprocess(cfg["proj_seed"], cfg["d_in"], cfg["d"], cfg["dtype"])
    dtype = cfg["dtype"]
    shard = dist_util.shard_rows(cfg["N"], 0, 1) if args.shard_rows else None
    if world == 1:
        return cfg, upload(keys, dtype), torch.from_numpy(np.ascontiguousarray(toks)).to(device), upload(q, dtype), shard, host
    dkeys = store_tensor(dist_util.broadcast_array(keys, 0, device), dtype)
    dtoks = dist_util.broadcast_array(toks, 0, device)
    dq = store_tensor(dist_util.broadcast_array(q, 0, device), dtype)
    if "d_in" not in cfg:
        ft = dist_util.broadcast_array(cfg.get("first_tokens"), 0, device)
        cfg["first_tokens"] = ft.cpu().numpy()
    return cfg, dkeys, dtoks, dq, shard, host


def relaunch_command(argv, n_gpus, port):
    """The command that starts `n_gpus` ranks of this script on this node (one process per GPU)."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_gpus}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *argv]


def maybe_relaunch(args, argv):
    """`python bench.py --gpus N` with N > 1, started plainly: start the N ranks and pass their
    output and exit code on.  Returns None when this process is already one of the ranks."""
    if args.gpus <= 1 or "WORLD_SIZE" in os.environ:
        return None
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    return subprocess.call(relaunch_command(argv, args.gpus, port))


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.path = tempfile.mktemp(prefix="dresd_clocks_", suffix=".csv")
        self.proc = None
        self.gpu_index = gpu_index

    def start(self):
        try:
            self.f = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"], stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if not self.proc:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.f.close()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as f:
            for line in f:
                p = [x.strip() for x in line.split(",")]
                if len(p) < 9:
                    continue
                try:
                    sm.append(float(p[1]))
                    mx.append(float(p[2]))
                except ValueError:
                    continue
                for name, val in zip(names, p[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        os.unlink(self.path)
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), samples=len(sm),
                       reasons=sorted(reasons))
        return out


# ----------------------------------------------------------------------------- CPU oracle legs
def time_oracle(cfg, keys, toks, q, n_queries):
    import oracle
    threads = oracle.dresd_oracle.default_threads()
    oracle.build()
    nq = max(1, n_queries)
    t0 = time.perf_counter()
    r = oracle.retrieve(keys, toks, cfg["dtype"], q[:nq], cfg["top_n"], cfg["draft_len"], W=cfg.get("W"),
                        threads=threads)
    dt = time.perf_counter() - t0
    return nq / dt, threads, nq, dt, r


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg, keys, toks, q = make_inputs(args)
    steps = max(1, min(args.steps, 3))
    for _ in range(min(args.warmup, 1)):
        time_oracle(cfg, keys, toks, q, 1)
    t0 = time.perf_counter()
    qps, threads, nq, dt, _ = time_oracle(cfg, keys, toks, q, steps)
    ms = (time.perf_counter() - t0) * 1e3 / steps
    sample = f"{nq} queries of the workload, whole datastore each (float64 brute force + full sort)"
    print(json.dumps({
        "impl": "reference", "metric": metric_name(cfg), "value": qps, "unit": "queries/s",
        "n_gpus": args.gpus, "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": workload_config(cfg),
        "cpu_baseline": {"value": qps, "unit": "queries/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": qps, "unit": "queries/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ----------------------------------------------------------------------------- the CUDA path
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2502_15572_b200 import binding, build as lib_build

    from paper_2502_15572_b200 import dist_util
    rank, local, world = dist_util.rank_info()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the retrieval path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        lib_build.build()
    if world > 1:
        dist.barrier()

    if args.shard_rows and (args.first_token_filter or args.quantised):
        raise SystemExit("--shard-rows times the exact, unfiltered call")
    # datastore and queries resident in HBM; `shard` = this rank's contiguous rows of the one datastore
    cfg, dkeys, dtoks, dq, shard, host = device_inputs(args, rank, world)
    keys, toks, q = host if host is not None else (None, None, None)
    cfg["filter_on"] = args.first_token_filter
    B, n, L, dtype = cfg["B"], cfg["top_n"], cfg["draft_len"], cfg["dtype"]
    if shard is not None:
        cfg["multi_gpu"] = "rows of one datastore sharded over the ranks; all-gather of the per-rank results + device merge"
    if shard is None:
        # every rank serves its own slice of the query stream against its own replica
        batches = dist_util.query_slice(dq.shape[0] // B, rank, world)
    else:
        batches = range(dq.shape[0] // B)                  # every rank sees every query
    nq, q_first = max(1, len(batches)), batches.start
    store = binding.Store(dkeys, dtoks, dtype)
    if "W" in cfg:
        dW = binding.to_device(cfg["W"], dtype)
        store.set_preprocess(cfg["d_in"], W=dW)
    store.set_option("scan_path", args.scan_path)
    store.set_option("probe", args.probe)
    store.set_option("keys_as_m", args.keys_as_m)
    dft = None
    if args.first_token_filter:
        if "first_tokens" not in cfg:
            raise SystemExit("--first-token-filter needs a workload whose queries have source rows")
        store.enable_first_token_filter()
        dft = torch.from_numpy(cfg["first_tokens"]).cuda()
        if args.sorted_store:
            store.index_first_tokens()
    out = (torch.empty((B, n), dtype=torch.int32, device="cuda"),
           torch.empty((B, n), dtype=torch.float32, device="cuda"),
           torch.empty((B, n, L), dtype=torch.int32, device="cuda"))

    recall = None
    if args.quantised:
        store.attach_quantised()
        # recall of the exact neighbours (the exact path is the parity-checked one)
        hit = tot = 0
        for i in range(min(nq, 64)):
            j = (q_first + i) * B
            ftk = None if dft is None else dft[j:j + B]
            ex = (store.retrieve(dq[j:j + B], n, L) if dft is None
                  else store.retrieve_filtered(dq[j:j + B], ftk, n, L))[0].cpu().numpy()
            ap_ = store.retrieve_quantised(dq[j:j + B], n, L, args.quantised, first_tokens=ftk)[0].cpu().numpy()
            for b in range(B):
                want = set(ex[b].tolist()) - {-1}
                hit += len(want & set(ap_[b].tolist()))
                tot += len(want)
        recall = hit / tot

    sharded = None if shard is None else dist_util.ShardedRetriever(store, shard.start, n, L)

    def step(i):
        j = (q_first + i % nq) * B
        if args.quantised:
            store.retrieve_quantised(dq[j:j + B], n, L, args.quantised, out=out,
                                     first_tokens=None if dft is None else dft[j:j + B])
        elif shard is not None:
            sharded(dq[j:j + B])
        elif dft is None:
            store.retrieve(dq[j:j + B], n, L, out=out)
        else:
            store.retrieve_filtered(dq[j:j + B], dft[j:j + B], n, L, out=out)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    barrier()
    store.status()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)

    # ---- device-resident timed region (CUDA events on the launching stream) ----
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record()
    for i in range(args.steps):
        step(args.warmup + i)
    ev1.record()
    barrier()
    ms_total = ev0.elapsed_time(ev1)
    launches = (store.last_launches() + (1 if shard is not None else 0)) * args.steps   # + the shard merge kernel
    passes = store.last_key_passes()                       # passes over the keys per call
    store.status()

    # ---- the scoring kernel by itself: a pass of its own, right after the timed region, in which EVERY
    # call carries a CUDA-event pair around its scoring launches (recorded by the library on the launching
    # stream).  The pass has a fixed length, whatever --steps is, and its own step time is taken by an outer
    # event pair over the same calls, so the kernel's time and the step time it is compared with come from
    # ONE measurement.  The events sit between the kernels of a call and switch off the overlap of a
    # kernel's set-up with its predecessor's tail: these calls are a little slower than the timed region's.
    PROFILED_CALLS = 64
    store.set_option("profile_stride", 1)
    store.set_option("profile", PROFILED_CALLS)
    pv0, pv1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    pv0.record()
    for i in range(PROFILED_CALLS):
        step(args.warmup + i)
    pv1.record()
    torch.cuda.synchronize()
    pass_ms_step = pv0.elapsed_time(pv1) / PROFILED_CALLS
    scan_ms, scan_calls = store.profile_read()
    store.set_option("profile", 0)
    store.status()

    # ---- latency per decode step (a synchronisation after every call) and the scan floor ----
    lat = []
    for i in range(min(args.steps, 200)):
        t0 = time.perf_counter()
        step(args.warmup + i)
        torch.cuda.synchronize()
        lat.append((time.perf_counter() - t0) * 1e3)
    # The cost of selection, merge and gather: the same call with a filter that nothing passes (keys
    # streamed and scored; no candidate queued, merged or gathered beyond empty lists) against the normal
    # call, in ALTERNATING bursts on the same stream (the SM clock drifts with the power state over a run,
    # so the two are compared burst by burst; medians).
    floor_ms = normal_ms = None
    if dtype != "f32" and args.scan_path != 1:
        burst, rounds = max(4, min(args.steps, 20)), 12
        t_floor, t_norm = [], []
        for r in range(rounds):
            order = ((1, t_floor), (0, t_norm)) if r % 2 == 0 else ((0, t_norm), (1, t_floor))
            for flag, acc in order:
                store.set_option("debug_no_select", flag)
                step(r)
                f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                f0.record()
                for i in range(burst):
                    step(args.warmup + i)
                f1.record()
                torch.cuda.synchronize()
                acc.append(f0.elapsed_time(f1) / burst)
        store.set_option("debug_no_select", 0)
        step(0)
        torch.cuda.synchronize()
        floor_ms, normal_ms = float(np.median(t_floor)), float(np.median(t_norm))

    # ---- end to end: pinned host buffers in and out through dresd_retrieve_host ----
    hq = (dq.view(torch.int16) if dtype != "f32" else dq).cpu().pin_memory()     # the query stream in host memory
    hout = (torch.empty((B, n), dtype=torch.int32).pin_memory(),
            torch.empty((B, n), dtype=torch.float32).pin_memory(),
            torch.empty((B, n, L), dtype=torch.int32).pin_memory())
    dq_stage = dq[:B].clone()
    hft = None if dft is None else torch.from_numpy(cfg["first_tokens"]).pin_memory()
    ft_stage = None if dft is None else dft[:B].clone()

    def host_call(j):
        if shard is not None:
            dq_stage.view(torch.int16 if dtype != "f32" else torch.float32).copy_(
                hq[j:j + B].view(torch.int16 if dtype != "f32" else torch.float32), non_blocking=True)
            res = sharded(dq_stage)
            for h, o_ in zip(hout, res):
                h.copy_(o_, non_blocking=True)
            torch.cuda.synchronize()
            return
        if not args.quantised and dft is None:
            store.retrieve_host(hq[j:j + B], n, L, hout)
            return
        # the quantised and the filtered calls take device buffers: the same copies, issued here
        dq_stage.view(torch.int16 if dtype != "f32" else torch.float32).copy_(
            hq[j:j + B].view(torch.int16 if dtype != "f32" else torch.float32), non_blocking=True)
        if dft is not None:
            ft_stage.copy_(hft[j:j + B], non_blocking=True)
        if args.quantised:
            store.retrieve_quantised(dq_stage, n, L, args.quantised, out=out, first_tokens=ft_stage)
        else:
            store.retrieve_filtered(dq_stage, ft_stage, n, L, out=out)
        for h, o_ in zip(hout, out):
            h.copy_(o_, non_blocking=True)
        torch.cuda.synchronize()

    for i in range(min(args.warmup, 3)):
        host_call((q_first + i % nq) * B)
    barrier()
    t0 = time.perf_counter()
    for i in range(args.steps):
        host_call((q_first + (args.warmup + i) % nq) * B)
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    barrier()
    clocks = sampler.stop() if rank == 0 else None

    ms_total, e2e_ms_total, scan_ms_avg, pass_ms_step = dist_util.max_over_ranks(
        [ms_total, e2e_s * 1e3, scan_ms / max(scan_calls, 1), pass_ms_step], device="cuda")
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    ms_step = ms_total / args.steps
    # replicas: every rank answered its own B queries per step; sharded rows: all ranks together answered B
    qps = dist_util.aggregate_throughput(B, args.steps, 1 if shard is not None else world, ms_total)
    e2e_qps = dist_util.aggregate_throughput(B, args.steps, 1 if shard is not None else world, e2e_ms_total)
    eb = synth.DTYPE_BYTES[dtype]
    key_bytes = cfg["N"] * cfg["d"] * (1 if args.quantised else eb)   # algorithmic bytes of one scoring launch
    if shard is not None:
        key_bytes = len(shard) * cfg["d"] * eb             # rank 0's kernel reads its shard
    if args.sorted_store and dft is not None:
        # only the rows of the batch's distinct first tokens are scored: mean over the timed steps
        counts = np.bincount(dtoks[:, 0].cpu().numpy())
        rows = [sum(int(counts[t]) for t in set(cfg["first_tokens"][j:j + B].tolist()))
                for j in ((q_first + (args.warmup + i) % nq) * B for i in range(args.steps))]
        cfg["rows_scanned_per_step_mean"] = float(np.mean(rows))
        key_bytes = cfg["rows_scanned_per_step_mean"] * cfg["d"] * (1 if args.quantised else eb)
    peak, peak_src = peaks()
    achieved = passes * key_bytes / (scan_ms_avg * 1e-3) / 1e9
    line = {
        "metric": metric_name(cfg) + (" -- 8-bit candidates, exact re-rank of %d" % args.quantised
                                      if args.quantised else "")
                  + (" -- rows sorted by first token, only the queries' token windows scanned"
                     if "rows_scanned_per_step_mean" in cfg else ""), "value": qps, "unit": "queries/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "strong" if shard is not None else "weak", "vs_baseline": None, "dtype": "f32 accumulate over %s keys" % dtype,
        "data": "synthetic", "config": workload_config(cfg),
        "e2e": {"value": e2e_qps, "unit": "queries/s",
                "h2d_bytes_per_step": B * cfg.get("d_in", cfg["d"]) * eb + (4 * B if dft is not None else 0),
                "d2h_bytes_per_step": B * n * (8 + 4 * L) + 4},
        "gpu_launches": launches,
        "clocks": {k: clocks[k] for k in ("sm_mhz", "sm_max_mhz", "reasons")},
        "roofline": {"bound": "hbm", "kernel": "scan (K2+K3: score every key + per-CTA top-n)",
                     "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_source": peak_src, "traffic": TRAFFIC_RATIO * passes * key_bytes,
                     "traffic_source": "ncu dram__bytes_read+write of the same kernel on a 2M-row case of this "
                                       "workload (1.004 x algorithmic), scaled by rows scanned; see profiles/",
                     "bytes_per_launch": key_bytes, "launches_per_step": passes,
                     "ms_per_launch": scan_ms_avg / max(1, round(passes)),
                     "frac_of_nominal_8TBs": achieved / 8000.0,
                     "timing": "CUDA-event pairs around the scoring launches of %d calls issued right after the "
                               "timed region (same stream, same inputs, every call profiled); ms_per_step_same_pass "
                               "is the step time of those same calls.  Events between the kernels of a call switch "
                               "off the overlap of a kernel's set-up with its predecessor's tail, so these calls are "
                               "slower than ms_per_step and `achieved` is a lower bound of the kernel's rate in the "
                               "timed region; achieved_if_step_were_all_scan is the other lower bound, the timed "
                               "region's whole step charged to the kernel" % scan_calls,
                     "ms_per_step_same_pass": pass_ms_step,
                     "non_scan_share_of_step": 1.0 - scan_ms_avg / pass_ms_step,
                     "achieved_if_step_were_all_scan": passes * key_bytes / (ms_step * 1e-3) / 1e9},
        "datastore_gbs_per_step": key_bytes / (ms_step * 1e-3) / 1e9,
        "latency_ms": {"p50": float(np.percentile(lat, 50)), "p99": float(np.percentile(lat, 99)),
                       "note": "wall clock per call with a device synchronisation after each"},
        "selection_overhead": None if floor_ms is None else {
            "floor_ms_per_step": floor_ms, "normal_ms_per_step": normal_ms, "frac": normal_ms / floor_ms - 1.0,
            "note": "floor = the same call with a filter that nothing passes (keys streamed and scored, "
                    "no candidate queued, merged or gathered beyond empty lists); floor and normal calls "
                    "timed in alternating bursts, medians"},
    }
    if args.quantised:
        line["quantised"] = {"candidates": args.quantised, "recall_at_n_vs_exact_path": recall,
                             "queries_compared": min(nq, 64) * B, "key_format": "E4M3 (k8 = e4m3(256 k))"}
        line["dtype"] = "f32 accumulate over E4M3 keys, exact re-rank over %s keys" % dtype
    if world == 1 and not args.no_cpu_baseline:
        o_qps, threads, o_nq, o_dt, _ = time_oracle(cfg, keys, toks, q, args.oracle_queries)
        line["cpu_baseline"] = {"value": o_qps, "unit": "queries/s", "cores": threads, "kind": "oracle",
                                "sample": f"{o_nq} queries of the workload over the whole datastore, {o_dt:.1f} s"}
    print(json.dumps(line))
    store.close()
    if world > 1:
        dist.destroy_process_group()


def run_build_keys(args):
    """Datastore-side preprocessing: rows/s and achieved tensor throughput of dresd_build_keys."""
    import torch
    from paper_2502_15572_b200 import binding, build as lib_build
    lib_build.build()
    torch.cuda.set_device(0)
    torch.manual_seed(1234)
    N, d_in, d = args.rows or 2_000_000, args.d_in, args.d_out
    H = torch.randn((N, d_in), device="cuda", dtype=torch.bfloat16)
    W = (torch.randn((d_in, d), device="cuda") / d_in ** 0.5).to(torch.bfloat16)
    mean = 0.5 * torch.randn(d_in, device="cuda")
    var = 0.5 + torch.rand(d_in, device="cuda")
    out = torch.empty((N, d), device="cuda", dtype=torch.bfloat16)
    s = torch.cuda.current_stream().cuda_stream
    terms = 1 if args.no_zscore else 2
    binding.dresd_set_global_option("build_keys_pairs", 0 if args.single_cta else 1)
    m_ptr, v_ptr = (None, None) if args.no_zscore else (mean.data_ptr(), var.data_ptr())

    def step():
        binding.dresd_build_keys(H.data_ptr(), N, d_in, binding.DRESD_BF16, m_ptr, v_ptr, 1e-5,
                                 W.data_ptr(), d, None, out.data_ptr(), s)

    steps, warm = min(args.steps, 20), max(3, min(args.warmup, 5))
    for _ in range(warm):
        step()
    sampler = ClockSampler(0)
    sampler.start()
    time.sleep(0.3)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    ev0.record()
    for _ in range(steps):
        step()
    ev1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = ev0.elapsed_time(ev1) / steps            # includes the per-call scratch set-up of W
    flops = 2.0 * N * d_in * d * terms            # with Eq. 1, both 16-bit terms of W / sigma are multiplied
    peak = 1404.5
    pk = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(pk):
        peak = float(json.load(open(pk))["bf16_tflops_sustained"])
    tf = flops / (ms * 1e-3) / 1e12
    print(json.dumps({
        "metric": "datastore rows preprocessed/s (Eq. 1 -> v W -> Eq. 2), bf16 hidden states",
        "value": N / (ms * 1e-3), "unit": "rows/s", "n_gpus": 1, "steps": steps, "warmup": warm,
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32 accumulate over bf16 operands", "data": "synthetic",
        "config": {"workload": "build_keys", "N": N, "d_in": d_in, "d": d, "zscore": not args.no_zscore,
                   "tensor_terms": terms, "cta_pairs": not args.single_cta,
                   "l2": "hidden states are %.1f GB per step: no flush needed" % (N * d_in * 2 / 1e9)},
        "gpu_launches": 2 * steps,
        "clocks": {k: clocks[k] for k in ("sm_mhz", "sm_max_mhz", "reasons")},
        "roofline": {"bound": "tensor", "kernel": "build_keys (tcgen05 GEMM + fused normalisation)",
                     "achieved": tf, "peak": peak, "unit": "TFLOP/s", "frac": tf / peak,
                     # the method's own flops, 2 N d_in d: with Eq. 1 the kernel multiplies TWO 16-bit terms of
                     # W / sigma to keep fp32-level weights, and `achieved` counts both
                     "frac_algorithmic": tf / terms / peak,
                     "peak_source": "measured (MEASURED_PEAKS.json bf16_tflops_sustained)", "traffic": None,
                     "hbm_read_gbs": N * d_in * 2 / (ms * 1e-3) / 1e9},
    }))


def run_fit_zscore(args):
    """Statistics of Eq. 1 over a sample of embeddings: rows/s and achieved HBM bandwidth of dresd_fit_zscore."""
    import torch
    from paper_2502_15572_b200 import binding, build as lib_build
    lib_build.build()
    torch.cuda.set_device(0)
    torch.manual_seed(4321)
    N, d_in = args.rows or 1_000_000, args.d_in
    V = (torch.randn((N, d_in), device="cuda") * 2.0 + 0.5).to(torch.bfloat16)
    mean = torch.empty(d_in, device="cuda")
    var = torch.empty(d_in, device="cuda")
    s = torch.cuda.current_stream().cuda_stream

    def step():
        binding.dresd_fit_zscore(V.data_ptr(), N, d_in, binding.DRESD_BF16, mean.data_ptr(), var.data_ptr(), s)

    steps, warm = min(args.steps, 50), max(3, min(args.warmup, 5))
    for _ in range(warm):
        step()
    sampler = ClockSampler(0)
    sampler.start()
    time.sleep(0.3)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    ev0.record()
    for _ in range(steps):
        step()
    ev1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = ev0.elapsed_time(ev1) / steps            # three launches and the call's stream synchronisation
    peak, src = 6650.0, "fallback"
    pk = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(pk):
        peak, src = float(json.load(open(pk))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    gbs = N * d_in * 2 / (ms * 1e-3) / 1e9
    print(json.dumps({
        "metric": "sample rows reduced/s (Eq. 1 statistics E[V], Var[V]), bf16 embeddings",
        "value": N / (ms * 1e-3), "unit": "rows/s", "n_gpus": 1, "steps": steps, "warmup": warm,
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32 chunk sums folded into f64", "data": "synthetic",
        "config": {"workload": "fit_zscore", "N": N, "d_in": d_in,
                   "l2": "the sample is %.1f GB per step: no flush needed" % (N * d_in * 2 / 1e9)},
        "gpu_launches": 3 * steps,
        "clocks": {k: clocks[k] for k in ("sm_mhz", "sm_max_mhz", "reasons")},
        "roofline": {"bound": "hbm", "kernel": "fit_sums_kernel (whole call timed)", "achieved": gbs, "peak": peak,
                     "unit": "GB/s", "frac": gbs / peak, "peak_source": src, "traffic": None},
    }))


if __name__ == "__main__":
    a = parse_args()
    rc = maybe_relaunch(a, sys.argv[1:])
    if rc is not None:
        sys.exit(rc)
    if a.fit_zscore:
        run_fit_zscore(a)
    elif a.build_keys:
        run_build_keys(a)
    elif a.impl == "reference":
        run_reference(a)
    else:
        run_ours(a)
