#!/usr/bin/env python
"""Benchmark of the ASL prefill hot path (score -> pool -> rank statistic ->
per-head top-k -> K/V compaction) on synthetic long-context tensors.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C3] [--impl ours|reference]

One "step" = one pass of the whole path over one layer's tensors of the
workload.  Prints ONE JSON line.  Inputs are seeded synthetic tensors shaped
like the 128K-token single-request workload (32 q heads / 8 kv heads, d=128,
w=64, budget 4096); several layers' tensors stay resident and the steps rotate
through them, so every step streams a K larger than L2 that it has not touched
for at least two steps.
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
sys.path.insert(0, ROOT)

from paper_2601_07667_b200 import inputs as I   # noqa: E402

METRIC = "obs-window score+select+compact: context tokens/s/layer"
UNIT = "tokens/s/layer"
# dram__bytes_read.sum + dram__bytes_write.sum of one scorer launch: read from the committed summary of the ncu
# capture (its "traffic_bytes_per_launch:" line), so that the figure and the evidence cannot drift apart
SCORER_TRAFFIC_FILES = {"C3": os.path.join(ROOT, "profiles", "score_tc_kernel_c3_128k_dram_traffic.txt")}


def scorer_traffic_bytes(workload_name):
    path = SCORER_TRAFFIC_FILES.get(workload_name)
    if not path or not os.path.exists(path):
        return None
    with open(path) as f:
        for line in f:
            if line.startswith("traffic_bytes_per_launch:"):
                return float(line.split(":")[1])
    return None
# default launch configuration of the timed steps (the GPU parity tests build their paths from the same two values)
DEFAULT_WORKLOAD = "C3"
DEFAULT_SCORE_CTAS = -16       # persistent scorer: this many CTAs fewer than SMs (0 = one per SM)
DEFAULT_LSE_SCORE_CTAS = -32   # the same for the one-pass step (supplied log-sum-exp) where a kv head has at most 256 query
                               # rows: its scorer is short enough for the rest of the layer to want more SMs; else as above
DEFAULT_TAIL_STREAMS = 2       # side streams for the rest of the layer
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["source"] = "fallback"
    return p


def algorithmic_work(wl, fp8_keys=False):
    """Algorithmic bytes and flops of one layer's pass: K read once, Q once, only
    kept K/V rows gathered (read + write), score vectors written and re-read by
    the pooling, ranking and selection stages, one QK^T."""
    d, Hk, Hq, w = wl.head_dim, wl.n_kv_heads, wl.n_q_heads, wl.window
    n_tot = wl.total_tokens
    T_tot = n_tot - wl.batch * w
    kept = sum(wl.kept(b) for b in range(wl.batch))
    k_bytes = n_tot * Hk * d * (1 if fp8_keys else 2)
    q_bytes = wl.batch * w * Hq * d * 2
    gather = (2 if fp8_keys else 4) * kept * Hk * d + 4 * kept * Hk * d      # K rows (1 or 2 bytes/element) + V rows, read + write
    score = 3 * (Hk + 1) * T_tot * 4 + kept * Hk * 4
    flops = 2.0 * w * d * n_tot * Hq
    return {"bytes": k_bytes + q_bytes + gather + score, "k_bytes": k_bytes, "flops": flops,
            "exps": float(w) * Hq * n_tot}


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.samples = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        mhz, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for s in self.samples:
            f = [x.strip() for x in s.split(",")]
            if len(f) < 7:
                continue
            try:
                mhz.append(float(f[0])); mx.append(float(f[1])); power.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(mhz)) if mhz else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(mhz), "reasons": sorted(reasons)}


def default_launch(sm_count: int, one_pass: bool = False) -> dict:
    """LayerPath keywords of the launch configuration this benchmark times by default (``one_pass``: of its
    one-pass step, scoring with a supplied log-sum-exp)."""
    want = DEFAULT_LSE_SCORE_CTAS if one_pass else DEFAULT_SCORE_CTAS
    ctas = want if want > 0 else max(1, sm_count + want)
    return {"score_ctas": ctas, "tail_streams": DEFAULT_TAIL_STREAMS}


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def rank_seed(seed: int, rank: int) -> int:
    """Requests are sharded by rank with no exchange: each rank draws its own seeded inputs."""
    return seed + rank


def max_over_ranks(ms: float, world: int, device="cuda") -> float:
    """Time of the slowest rank (the only reduction on the multi-GPU path)."""
    if world == 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_tokens_per_s(tokens_per_rank: int, world: int, ms_per_step: float) -> float:
    """Whole-job throughput: every rank's tokens over the slowest rank's step time."""
    return world * tokens_per_rank / (ms_per_step * 1e-3)


def spawn_replicas(n: int, argv) -> int:
    """Starts ``n`` ranks of this script on this node (rank r on GPU r), one process each, with the
    rendezvous variables a launcher would set, and waits for them.  Returns the worst exit code.
    Rank 0's JSON line goes to this process's stdout; the other ranks print nothing."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + list(argv), env=env))
    worst = 0
    for p in procs:
        rc = p.wait()
        worst = rc if rc != 0 and worst == 0 else worst
    return worst


def run_dry(args):
    """Rendezvous only (no kernel runs, no GPU needed): every rank joins the process group (NCCL on a
    CUDA box, gloo otherwise), the per-rank times 1+rank ms are MAX-reduced as the timed region's
    would be, and rank 0 prints the distributed fields of the JSON line."""
    import torch
    import torch.distributed as dist
    rank, world, local = dist_env()
    cuda = torch.cuda.is_available()
    if cuda:
        torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl" if cuda else "gloo")
    ms = max_over_ranks(1.0 + rank, world, device="cuda" if cuda else "cpu")
    if rank == 0:
        print(json.dumps({"dry_run": True, "n_gpus": world, "ms_per_step": ms, "seed_of_last_rank": rank_seed(args.seed, world - 1),
                          "value": aggregate_tokens_per_s(1000, world, ms), "scaling": "weak"}), flush=True)
    if world > 1:
        dist.destroy_process_group()


# --------------------------------------------------------------------------------------
def oracle_step(wl, x, layer, controllers, heads=None):
    """One layer of the path by the fp64 oracle (optionally only the first `heads` kv heads)."""
    from oracle import asl_oracle as O
    cu = wl.cu_seqlens()
    Hk = wl.n_kv_heads if heads is None else heads
    for b in range(wl.batch):
        n, w = wl.seqlens[b], wl.window
        q = O.widen_bf16(x["q_obs"][b][: Hk * wl.group])
        k = O.widen_bf16(x["k"][cu[b]:cu[b + 1], :Hk])
        P, agg = O.score_layer(q, k, wl.group, wl.pool_kernel, wl.pool_mode)
        controllers[b].step(layer, agg)
        kk = O.kept_count(wl.budgets[b], n, w)
        for h in range(Hk):
            idx = O.select_topk(P[h], kk, n, w)
            O.compact_rows(x["k"][cu[b]:cu[b + 1]], idx, h)
            O.compact_rows(x["v"][cu[b]:cu[b + 1]], idx, h)


def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
        return int(n)
    except Exception:
        return os.cpu_count() or 1


def time_oracle(wl, layer_sets, steps, warmup, heads):
    from oracle import asl_oracle as O
    ctl = [O.SelectionController(wl.budgets[b], wl.window, wl.l_min, wl.l_obs, wl.tau) for b in range(wl.batch)]
    for i in range(warmup):
        oracle_step(wl, layer_sets[i % len(layer_sets)], i, ctl, heads)
    t0 = time.perf_counter()
    for i in range(steps):
        oracle_step(wl, layer_sets[i % len(layer_sets)], warmup + i, ctl, heads)
    dt = (time.perf_counter() - t0) / max(steps, 1)
    frac = heads / wl.n_kv_heads
    return wl.total_tokens * frac / dt, dt


def make_workload(args):
    """The named workload, optionally with other context lengths (profiling-sized cases)."""
    base = I.workload(args.workload, seed=args.seed)
    if not args.seqlens and not args.budgets and not args.heads:
        return base
    seqlens = tuple(int(x) for x in args.seqlens.split(",")) if args.seqlens else base.seqlens
    if args.budgets:
        budgets = tuple(int(x) for x in args.budgets.split(","))
    else:                                          # keep the workload's first budget, one per request
        budgets = tuple(min(base.budgets[0], n) for n in seqlens)
    heads = {}
    if args.heads:
        hq, hk = (int(x) for x in args.heads.split(","))
        heads = {"n_q_heads": hq, "n_kv_heads": hk}
    return I.workload(args.workload, seed=args.seed, seqlens=seqlens, budgets=budgets, **heads)


def run_reference(args):
    rank, world, _ = dist_env()
    if rank != 0:
        return
    wl = make_workload(args)
    heads = 1
    sets = [I.layer_inputs(wl, l, args.seed) for l in range(2)]
    np.dot(np.ones((64, 64)), np.ones((64, 64)))
    value, dt = time_oracle(wl, sets, args.steps, args.warmup, heads)
    cores = oracle_threads()
    sample = (f"each step: the whole path of one layer for kv head 0 and its {wl.group} query heads "
              f"(1/{wl.n_kv_heads} of the scoring, top-k and compaction; the rank statistic in full), "
              f"value scaled by that fraction")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "seqlens": list(wl.seqlens), "window": wl.window,
                       "budgets": list(wl.budgets), "heads": f"{wl.n_q_heads}q/{wl.n_kv_heads}kv", "d": wl.head_dim},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2601_07667_b200 import binding as B

    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    wl = make_workload(args)
    sms = torch.cuda.get_device_properties(local).multi_processor_count
    if args.score_ctas < 0:
        args.score_ctas = max(1, sms + args.score_ctas)
    if args.lse_score_ctas is None and (wl.n_q_heads // wl.n_kv_heads) * wl.window <= 256:
        args.lse_score_ctas = DEFAULT_LSE_SCORE_CTAS
    if args.lse_score_ctas is None:
        args.lse_score_ctas = args.score_ctas
    elif args.lse_score_ctas < 0:
        args.lse_score_ctas = max(1, sms + args.lse_score_ctas)
    fp8 = args.k_dtype == "fp8"
    work = algorithmic_work(wl, fp8)
    pk = peaks()

    # resident inputs: a few layers' tensors, rotated (each rank draws its own seed: independent requests)
    n_sets = args.layer_sets
    host_sets = [I.layer_inputs(wl, l, rank_seed(args.seed, rank)) for l in range(n_sets)]
    k_scale = None
    if fp8:
        # a quantised K cache: one scale per kv head for the whole run (the scales belong to the plan)
        amax = np.max([np.abs(I.bf16_bits_to_f32(x["k"])).max(axis=(0, 2)) for x in host_sets], axis=0)
        k_scale = (amax / 448.0).astype(np.float32)
        for x in host_sets:
            x["k"] = I.keys_to_fp8(x["k"], k_scale)[0]
    pin = lambda a: torch.from_numpy(a if a.dtype == np.uint8 else a.view(np.int16)).pin_memory()
    host_pinned = [{k: pin(x[k]) for k in ("q_obs", "k", "v")} for x in host_sets]
    as_dev = lambda t: t.cuda(non_blocking=True) if t.dtype == torch.uint8 else t.cuda(non_blocking=True).view(torch.bfloat16)
    dev_sets = [{k: as_dev(t) for k, t in hp.items()} for hp in host_pinned]
    torch.cuda.synchronize()

    def make_path(score_ctas):
        return B.LayerPath(n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads, head_dim=wl.head_dim, window=wl.window,
                           pool_kernel=wl.pool_kernel, pool_mode=wl.pool_mode, seqlens=wl.seqlens, budgets=wl.budgets,
                           l_min=wl.l_min, l_obs=wl.l_obs, tau=wl.tau, device=local, score_ctas=score_ctas,
                           tail_streams=args.tail_streams, k_dtype=B.ASL_K_FP8_E4M3 if fp8 else B.ASL_K_BF16,
                           k_scale=None if k_scale is None else [float(s) for s in k_scale])

    path = make_path(args.score_ctas)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    stream = torch.cuda.current_stream()
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def step(i, marks=None):
        s = dev_sets[i % n_sets]
        if marks is None:
            path.run_layer(s["q_obs"], s["k"], s["v"], i)
            return
        # same calls as run_layer, with events between the stages (stage timing run only)
        ctx, ws, wsb = path.ctx, path.workspace, path.ws_bytes
        rows = path.n_rows(i)
        e = [ev() for _ in range(5)]
        e[0].record(stream)
        B.asl_score_layer(ctx, s["q_obs"], s["k"], path.scores_kv, path.scores_agg, ws, wsb)
        e[1].record(stream)
        B.asl_rank_stat(ctx, path.scores_agg, i, rows, path.rank_ring, path.stat, ws, wsb)
        e[2].record(stream)
        B.asl_select_topk(ctx, path.scores_kv, wl.n_kv_heads, path.idx, ws, wsb)
        e[3].record(stream)
        B.asl_compact_kv(ctx, s["k"], s["v"], path.idx, path.k_out, path.v_out)
        e[4].record(stream)
        marks.append(e)

    # ---- warm-up, then the timed region: EXACTLY `steps` steps ----
    for i in range(args.warmup):
        step(i)
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    # The K steps are issued either call by call, or (default) as one CUDA graph recorded from those
    # very calls: one launch for the whole sequence, side streams included.
    step_args = lambda i: tuple(dev_sets[i % n_sets][k] for k in ("q_obs", "k", "v")) + (i,)
    graph = None
    launches0 = B.asl_launch_count(path.ctx)
    issue = "call by call"
    if args.graph:
        try:
            graph = path.capture([step_args(args.warmup + i) for i in range(args.steps)])
            launches = B.asl_launch_count(path.ctx) - launches0      # kernels recorded = kernels per replay
            graph.replay()                                           # untimed: uploads the graph
            torch.cuda.synchronize()
            issue = "one CUDA graph of the K steps"
        except RuntimeError as e:                                    # capture refused: time the calls themselves
            graph = None
            args.graph = False
            issue = "call by call (graph capture failed: %s)" % str(e).splitlines()[0][:80]
            torch.cuda.synchronize()
            path._fresh_events()
            launches0 = B.asl_launch_count(path.ctx)
    t_start, t_end = ev(), ev()
    barrier()
    t_start.record(stream)
    if graph is not None:
        graph.replay()
    else:
        for i in range(args.steps):
            path.run_layer(*step_args(args.warmup + i))
        path.join()
    t_end.record(stream)
    barrier()
    if graph is None:
        launches = B.asl_launch_count(path.ctx) - launches0
    time.sleep(0.2)
    clocks = sampler.stop() if rank == 0 else None
    ms_total = t_start.elapsed_time(t_end)
    ms_total = max_over_ranks(ms_total, world)
    ms_step = ms_total / args.steps
    value = aggregate_tokens_per_s(wl.total_tokens, world, ms_step)

    # ---- the scorer kernel's own duration while it shares the GPU with the rest (events around the
    #      scoring call, same overlapped sequence issued call by call; outside the timed region) ----
    score_marks = []
    for i in range(args.steps):
        path.run_layer(*step_args(args.warmup + i), score_marks=score_marks)
    path.join()
    torch.cuda.synchronize()
    score_ms = float(np.mean([a.elapsed_time(b_) for a, b_ in score_marks]))

    # ---- per-stage times (serialised, outside the timed region) ----
    marks = []
    for i in range(min(args.steps, 8)):
        step(args.warmup + args.steps + i, marks)
    torch.cuda.synchronize()
    stage_ms = [float(np.mean([m[j].elapsed_time(m[j + 1]) for m in marks])) for j in range(4)]

    # ---- the same step when the caller supplies the window rows' log-sum-exp (one pass over K) ----
    lp = path if args.lse_score_ctas == args.score_ctas else make_path(args.lse_score_ctas)
    lse_sets = []
    for ds in dev_sets:
        B.asl_score_layer(lp.ctx, ds["q_obs"], ds["k"], lp.scores_kv, lp.scores_agg, lp.workspace, lp.ws_bytes)
        lse = torch.empty((wl.batch, wl.n_q_heads, wl.window), dtype=torch.float32, device="cuda")
        B.asl_window_lse(lp.ctx, lp.workspace, lp.ws_bytes, lse)
        lse_sets.append(lse)
    lp.reset()
    for i in range(args.warmup):
        lp.run_layer(dev_sets[i % n_sets]["q_obs"], dev_sets[i % n_sets]["k"], dev_sets[i % n_sets]["v"], i,
                       lse=lse_sets[i % n_sets])
    lp.join()
    barrier()
    lse_graph = None
    if args.graph:
        lse_graph = lp.capture([step_args(args.warmup + i) + (lse_sets[(args.warmup + i) % n_sets],)
                                  for i in range(args.steps)])
        lse_graph.replay()
        barrier()
    l0, l1 = ev(), ev()
    l0.record(stream)
    if lse_graph is not None:
        lse_graph.replay()
    else:
        for i in range(args.steps):
            j = (args.warmup + i) % n_sets
            lp.run_layer(dev_sets[j]["q_obs"], dev_sets[j]["k"], dev_sets[j]["v"], args.warmup + i, lse=lse_sets[j])
        lp.join()
    l1.record(stream)
    barrier()
    lse_ms = max_over_ranks(l0.elapsed_time(l1), world) / args.steps
    if lp is not path:
        lp.close()

    # ---- end to end through the C ABI with host buffers ----
    e2e_steps = max(2, min(args.steps, args.e2e_steps))
    q_d, k_d, v_d = (torch.empty_like(dev_sets[0][k]) for k in ("q_obs", "k", "v"))
    idx_h = torch.empty(path.idx.shape, dtype=torch.int32).pin_memory()
    ko_h = torch.empty(path.k_out.shape, dtype=path.k_out.dtype).pin_memory()
    vo_h = torch.empty(path.v_out.shape, dtype=torch.bfloat16).pin_memory()
    st_h = torch.empty(path.stat.shape, dtype=torch.uint8).pin_memory()

    def e2e_step(i):
        hp = host_pinned[i % n_sets]
        for dst, key in ((q_d, "q_obs"), (k_d, "k"), (v_d, "v")):
            (dst if dst.dtype == torch.uint8 else dst.view(torch.int16)).copy_(hp[key], non_blocking=True)
        path.run_layer(q_d, k_d, v_d, i)
        path.join()                     # top-k, compaction and the statistic run on side streams
        idx_h.copy_(path.idx, non_blocking=True)
        ko_h.copy_(path.k_out, non_blocking=True)
        vo_h.copy_(path.v_out, non_blocking=True)
        st_h.copy_(path.stat, non_blocking=True)

    path.reset()
    e2e_step(0)
    barrier()
    e0, e1 = ev(), ev()
    e0.record(stream)
    for i in range(e2e_steps):
        e2e_step(1 + i)
    e1.record(stream)
    barrier()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1), world) / e2e_steps
    # the leg checks what it timed: the host copies are the device results of the last step
    if not (torch.equal(idx_h, path.idx.cpu()) and torch.equal(ko_h.view(torch.uint8), path.k_out.cpu().view(torch.uint8))
            and torch.equal(st_h, path.stat.cpu())):
        raise SystemExit("end-to-end leg: host copies differ from the device results")
    h2d = sum(host_pinned[0][k].numel() * host_pinned[0][k].element_size() for k in ("q_obs", "k", "v"))
    d2h = idx_h.numel() * 4 + ko_h.numel() * ko_h.element_size() + vo_h.numel() * 2 + st_h.numel()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the whole step and of the scorer ----
    hbm = pk["hbm_gbs"]
    tf = pk["bf16_tflops"] * (2.0 if fp8 else 1.0)      # 8-bit operands: the measured bf16 peak times the nominal fp8/bf16 ratio
    t_hbm = work["bytes"] / (hbm * 1e9)
    t_mma = work["flops"] / (tf * 1e12)
    bound = "hbm" if t_hbm >= t_mma else "tensor"
    if bound == "hbm":
        achieved = work["k_bytes"] / (score_ms * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": achieved, "peak": hbm, "unit": "GB/s", "frac": achieved / hbm}
    else:
        achieved = work["flops"] / (score_ms * 1e-3) / 1e12
        roof = {"bound": "tensor", "achieved": achieved, "peak": tf, "unit": "TFLOP/s", "frac": achieved / tf}
    default_shape = not args.seqlens and not args.budgets and not args.heads and not fp8
    roof.update({"traffic": scorer_traffic_bytes(wl.name) if default_shape else None, "kernel": "score_tc_kernel (asl_score_columns: both softmax passes, one persistent launch)", "kernel_ms": score_ms,
                 "peak_source": pk["source"], "step_roofline_us": max(t_hbm, t_mma) * 1e6,
                 "step_frac": max(t_hbm, t_mma) / (ms_step * 1e-3)})

    # ---- the oracle on the host cores, bounded sample ----
    cpu = None
    if world == 1 and not args.no_cpu_baseline and not fp8:
        v, dt = time_oracle(wl, host_sets, 2, 1, 1)
        cpu = {"value": v, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
               "sample": f"2 layers, kv head 0 with its {wl.group} query heads (1/{wl.n_kv_heads} of scoring, top-k and "
                         f"compaction, rank statistic in full), scaled by that fraction; {dt:.2f} s per sampled layer"}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "fp8" if fp8 else "bf16", "data": "synthetic",
            "config": {"workload": wl.name, "seqlens": list(wl.seqlens), "window": wl.window,
                       "budgets": list(wl.budgets), "heads": f"{wl.n_q_heads}q/{wl.n_kv_heads}kv", "d": wl.head_dim,
                       "pool": [wl.pool_kernel, "avg" if wl.pool_mode == 0 else "max"], "k_dtype": args.k_dtype,
                       "l2": (f"inputs larger than L2: {n_sets} resident layer sets rotated, K = "
                              f"{work['k_bytes'] / 1e6:.0f} MB per layer") if work["k_bytes"] * n_sets > 126e6 else
                             (f"small workload: {n_sets} layer sets of {work['k_bytes'] / 1e6:.1f} MB K stay in L2 "
                              f"(launch-latency bound, a parity configuration)"),
                       "score_ctas": args.score_ctas, "tail_streams": args.tail_streams, "issue": issue, "parallelism": f"replicas x{world}"},
            "roofline": roof, "cpu_baseline": cpu,
            "e2e": {"value": aggregate_tokens_per_s(wl.total_tokens, world, e2e_ms), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms},
            "one_pass_lse": {"ms_per_step": lse_ms, "score_ctas": args.lse_score_ctas, "value": aggregate_tokens_per_s(wl.total_tokens, world, lse_ms),
                             "unit": UNIT, "step_frac": max(t_hbm, t_mma) / (lse_ms * 1e-3),
                             "note": "asl_score_layer_lse: the caller supplies the window rows' log-sum-exp"},
            "gpu_launches": int(launches), "clocks": clocks,
            "stages_ms": {"score+pool": stage_ms[0], "rank_stat": stage_ms[1], "topk": stage_ms[2],
                          "compact": stage_ms[3]}}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--layer-sets", type=int, default=3)
    ap.add_argument("--e2e-steps", type=int, default=4)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", dest="graph", action="store_false",
                    help="issue the timed steps call by call instead of replaying one CUDA graph of them")
    ap.add_argument("--tail-streams", type=int, default=DEFAULT_TAIL_STREAMS, choices=[1, 2],
                    help="side streams for the rest of the layer: 2 = statistic and top-k/compaction side by side")
    ap.add_argument("--score-ctas", type=int, default=DEFAULT_SCORE_CTAS,
                    help="CTAs of the persistent scorer: 0 = one per SM, negative = that many fewer than SMs.  Fewer "
                         "leaves SMs to the previous layer's statistic, top-k and compaction, which run on a side stream")
    ap.add_argument("--lse-score-ctas", type=int, default=None,
                    help="the same for the one-pass step (scoring with a supplied log-sum-exp); default: "
                         f"{DEFAULT_LSE_SCORE_CTAS} where a kv head has at most 256 query rows, else --score-ctas")
    ap.add_argument("--seqlens", type=str, default=None,
                    help="comma-separated context lengths replacing the workload's (smaller cases for profiling)")
    ap.add_argument("--budgets", type=str, default=None, help="comma-separated KV budgets, one per request")
    ap.add_argument("--heads", type=str, default=None, help="query,kv head counts replacing the workload's (e.g. 28,4)")
    ap.add_argument("--k-dtype", default="bf16", choices=["bf16", "fp8"],
                    help="fp8: K as E4M3 codes with one scale per kv head (a quantised K cache); the headline workload is bf16")
    ap.add_argument("--dry-run", action="store_true",
                    help="ranks only rendezvous and reduce a fixed time (checks the multi-rank launch; runs no kernel)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
        return
    world_env = os.environ.get("WORLD_SIZE")
    if world_env is None and args.gpus > 1:
        # started without a launcher: this process becomes the launcher of the N replicas
        raise SystemExit(spawn_replicas(args.gpus, sys.argv[1:]))
    if world_env is not None and int(world_env) != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but the launcher started WORLD_SIZE={world_env} ranks")
    if args.dry_run:
        run_dry(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
