#!/usr/bin/env python
"""Benchmark of the mixed-state block-denoising engine on one node.

A "step" is one complete pass of the hot path over one batch of synthetic
input: the whole workload (default: the Dream-7B-shaped batch of 16, the
configuration the headline metric is quoted on) is admitted, then block-cycles
run until the pending queue and the active set are empty.  `value` is committed
tokens per second with the requests already resident in HBM; `e2e` is the same
metric through the public C ABI with host buffers (bs_admit from pinned host
memory and bs_read_tokens inside the timed region).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 1..5] [--impl ours|reference]

With N > 1 every rank serves its own independently drawn batch on its own GPU
(request-sharded replicas, no collective on the data path); times are the max
over ranks.  The ranks either come from torch.distributed.run (RANK /
LOCAL_RANK / WORLD_SIZE / MASTER_* in the environment), or, when the script is
started plainly with --gpus N > 1, it starts the N ranks itself.
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
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import bs_inputs  # noqa: E402

METRIC = "committed_tokens_per_s"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel, from the ncu capture summarised
# in profiles/gemm_pair_gate_up_m256.md (gate/up GEMM at M = 256: algorithmic 283.1 MB, measured 277.9 MB)
NCU_TRAFFIC_BYTES_PER_LAUNCH = 277925888
GEMM_FAMILIES = ("gemm_qkv", "gemm_o", "gemm_gate_up", "gemm_down", "gemm_lm_head")


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows, self.proc, self.thread, self.gpu = [], None, None, gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "200"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for nme, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nme)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def shard_seed(base_seed: int, rank: int) -> int:
    """Replicas: rank r draws its own batch (weak scaling, per-GPU work fixed)."""
    return base_seed + 7919 * rank


def max_over_ranks(value: float, world: int, device) -> float:
    if world == 1:
        return value
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, world: int, device) -> float:
    if world == 1:
        return value
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def kv_capacity_for(wl) -> int:
    rows = sorted((r.p + r.g for r in wl.requests), reverse=True)[:wl.max_batch]
    cap = sum(rows)
    if wl.token_budget > 0:
        cap = min(cap, 98304)
    return max(cap, wl.max_row_tokens)


def run_ours(args):
    rank, world, local = dist_env()
    torch.cuda.set_device(local)
    device = torch.device(f"cuda:{local}")
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    from paper_2607_08930_b200 import build
    if rank == 0 or not os.path.exists(os.path.join(ROOT, "paper_2607_08930_b200", "libblockserve.so")):
        build.build()
    barrier(world)
    from paper_2607_08930_b200 import binding as B

    wl = bs_inputs.workload(args.workload, seed=shard_seed(0, rank))
    weights = bs_inputs.make_weights(wl.shape, wl.weight_seed, device=str(device))
    torch.cuda.synchronize()
    cap = kv_capacity_for(wl)
    target = wl.committed_target()

    def new_engine(**kw):
        return B.engine_for_workload(wl, weights, kv_capacity_tokens=cap, device=str(device), **kw)

    def admit_all(eng, prompts):
        for r, pr in zip(wl.requests, prompts):
            eng.admit(r.req_id, pr, r.g, r.alpha, r.start_block, r.gen_prefix)

    def serve(eng):
        eng.run()

    # prompts live in pinned host memory (the e2e arm copies them in the timed region)
    pinned = []
    for r in wl.requests:
        t = torch.from_numpy(r.prompt.copy()).pin_memory()
        pinned.append(t.numpy())
    h2d = sum(4 * (r.p + r.g) for r in wl.requests)
    d2h = h2d

    t_start = time.perf_counter()

    def phase(msg):          # progress on stderr (BS_BENCH_VERBOSE=1): the JSON line stays alone on stdout
        if rank == 0 and os.environ.get("BS_BENCH_VERBOSE"):
            print(f"[bench {time.perf_counter() - t_start:8.1f} s] {msg}", file=sys.stderr, flush=True)

    # ---- warm-up (whole jobs) ----
    for _ in range(args.warmup):
        e = new_engine()
        admit_all(e, pinned)
        serve(e)
        assert e.stats().committed == target
        e.close()
        del e
        phase("warm-up job done")
    torch.cuda.synchronize()

    # ---- device-resident arm: requests admitted (copied to HBM) before the clock starts.  One engine is alive at a
    # time (a KV arena can take 45 GB): each job is bracketed by barrier + synchronize and timed with CUDA events on
    # the launching stream; the timed region is the sum over the K jobs.
    def timed_jobs(n_jobs: int, profile: bool, **engine_kw):
        stream = torch.cuda.current_stream()
        total_ms, stats, profs = 0.0, [], []
        for _ in range(n_jobs):
            e = new_engine(**engine_kw)
            admit_all(e, pinned)
            e.set_profiling(profile)
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            barrier(world)
            torch.cuda.synchronize()
            ev0.record(stream)
            serve(e)
            ev1.record(stream)
            torch.cuda.synchronize()
            barrier(world)
            total_ms += ev0.elapsed_time(ev1)
            stats.append(e.stats())
            if profile:
                profs.append(e.profile())
            e.close()
            del e
        return total_ms, stats, profs

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ms_local, job_stats, _ = timed_jobs(args.steps, profile=False)
    phase(f"timed jobs done ({ms_local:.0f} ms)")
    ms_total = max_over_ranks(ms_local, world, device)
    clocks = sampler.stop() if rank == 0 else None
    committed = sum(st.committed for st in job_stats)
    assert committed == target * args.steps, "engine did not commit exactly g_i tokens per request"
    launches = sum(st.kernel_launches for st in job_stats)
    steps_run = sum(st.steps for st in job_stats)
    cycles = sum(st.cycles for st in job_stats)
    sum_active = sum(st.sum_active for st in job_stats)
    torch.cuda.empty_cache()
    total_committed = sum_over_ranks(float(committed), world, device)
    value = total_committed / (ms_total * 1e-3)

    # ---- one more job with the per-family CUDA-event timers on: the roofline numbers.  The timers add two event
    # records per kernel family per layer and keep neighbouring kernels from overlapping their launches, so this
    # job runs a few percent slower than the timed ones; its time is reported beside them.
    prof, prof_ms_job = {}, None
    if not args.no_profile:
        prof_ms_job, _, profs = timed_jobs(1, profile=True)
        for pr in profs:
            for fam, v in pr.items():
                acc = prof.setdefault(fam, dict(ms=0.0, launches=0, flops=0.0, bytes=0.0))
                for k in acc:
                    acc[k] += v[k]
        torch.cuda.empty_cache()
        phase("profiled job done")

    # ---- the same jobs under the per-row block advance (a policy beyond Algorithm 1's synchronous cycles; reported
    # beside the headline, never instead of it)
    async_ms, async_stats, _ = timed_jobs(max(1, min(args.steps, 3)), profile=False, async_advance=True)
    async_ms = max_over_ranks(async_ms, world, device)
    async_committed = sum_over_ranks(float(sum(st.committed for st in async_stats)), world, device)
    assert sum(st.committed for st in async_stats) == target * len(async_stats)
    phase("per-row advance jobs done")

    # ---- end-to-end arm: host buffers in, host buffers out, through the C ABI (engine set-up is not timed) ----
    e2e_local = 0.0
    for _ in range(args.steps):
        e = new_engine()
        torch.cuda.synchronize()
        barrier(world)
        t0 = time.perf_counter()
        admit_all(e, pinned)
        serve(e)
        for r in wl.requests:
            toks, state = e.read_tokens(r.req_id)
        torch.cuda.synchronize()
        e2e_local += time.perf_counter() - t0
        e.close()
        del e
    e2e_s = max_over_ranks(e2e_local, world, device)
    phase("end-to-end jobs done")
    e2e_value = total_committed / e2e_s

    if rank != 0:
        return
    pk, pk_kind = peaks()
    if args.no_profile:
        print(json.dumps({"metric": METRIC, "value": value, "unit": UNIT, "ms_per_step": ms_total / args.steps,
                          "e2e": e2e_value, "note": "per-family timers off"}))
        return
    prof_ms = sum(v["ms"] for v in prof.values())

    def roof_of(fams, label):
        """Roofline figures of a set of kernel families: algorithmic flops and bytes of their launches over the device
        time the family timers measured for them."""
        ms = sum(prof[f]["ms"] for f in fams)
        fl = sum(prof[f]["flops"] for f in fams)
        by = sum(prof[f]["bytes"] for f in fams)
        n = sum(prof[f]["launches"] for f in fams)
        if fl / (pk["bf16_tflops_sustained"] * 1e12) >= by / (pk["hbm_gbs"] * 1e9):
            r = {"bound": "tensor", "achieved": fl / (ms * 1e-3) / 1e12, "peak": pk["bf16_tflops_sustained"],
                 "unit": "TFLOP/s"}
        else:
            r = {"bound": "hbm", "achieved": by / (ms * 1e-3) / 1e9, "peak": pk["hbm_gbs"], "unit": "GB/s"}
        r.update(frac=r["achieved"] / r["peak"], peak_kind=pk_kind, kernel=label, launches=n,
                 avg_launch_us=1e3 * ms / max(n, 1), share_of_step=ms / max(prof_ms, 1e-9),
                 # the same work over (these kernels' share of the profiled job) x (the un-profiled job time)
                 achieved_at_timed_speed=r["achieved"] * prof_ms_job / max(ms_total / args.steps, 1e-9),
                 tflops=fl / (ms * 1e-3) / 1e12, gbs=by / (ms * 1e-3) / 1e9)
        return r

    # the dominant kernel: the SwiGLU gate/up projection (the largest share of every workload's device time); the ncu
    # traffic figure below is a capture of that same kernel
    dominant = max(GEMM_FAMILIES, key=lambda f: prof[f]["ms"])
    roof = roof_of([dominant], {"gemm_gate_up": "projection GEMM, SwiGLU gate/up (k_gemm_pair<3> / k_gemm_tc<3>)"}
                   .get(dominant, f"projection GEMM ({dominant})") + ", from one extra job with per-family timers")
    roof.update(traffic=NCU_TRAFFIC_BYTES_PER_LAUNCH if dominant == "gemm_gate_up" else None,
                traffic_note="ncu DRAM bytes of one gate/up launch at M = 256 (algorithmic 283.1 MB)",
                profiled_job_ms=prof_ms_job)
    roof_all = roof_of(GEMM_FAMILIES, "all five projection GEMM shapes")
    families = {f: {"ms": round(v["ms"], 3), "launches": v["launches"],
                    "tflops": round(v["flops"] / max(v["ms"], 1e-9) / 1e9, 2),
                    "gbs": round(v["bytes"] / max(v["ms"], 1e-9) / 1e6, 1)} for f, v in prof.items()}
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": wl.name, "requests_per_gpu": len(wl.requests), "block_len": wl.block_len,
                   "tau": wl.tau, "token_budget": wl.token_budget, "max_batch": wl.max_batch,
                   "committed_tokens_per_step": target, "denoise_steps_per_step": steps_run / args.steps,
                   "block_cycles_per_step": cycles / args.steps,
                   "effective_compute_ratio": sum_active / max(cycles, 1) / wl.max_batch,
                   "l2": "inputs exceed L2 (weights %.1f GB streamed every denoise step)" %
                         (wl.shape.weight_bytes_bf16() / 1e9),
                   "parallelism": "replicas only" if world > 1 else "1 gpu"},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": int(launches),
        "per_row_advance": {"value": async_committed / (async_ms * 1e-3), "unit": UNIT,
                            "ms_per_step": async_ms / len(async_stats),
                            "denoise_steps_per_step": sum(st.steps for st in async_stats) / len(async_stats),
                            "note": "bs_config.async_advance = 1: rows start their next block the step after their "
                                    "own block completes; not part of the headline value"},
        "clocks": clocks,
        "roofline": roof,
        "roofline_all_gemms": roof_all,
        "families": families,
    }
    if world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(wl, weights, args.cpu_seconds)
    print(json.dumps(out))


# ---------------------------------------------------------------------------------------------------------
# the CPU oracle, timed as it stands on the host cores (a reported baseline, and the --impl reference arm)
# ---------------------------------------------------------------------------------------------------------

class _LazyOracleModel:
    """Feeds the oracle fp32 copies of the weights, widening one layer at a time; the widening time is
    input preparation and is kept out of the oracle's clock."""

    def __init__(self, shape, weights):
        from oracle import blockserve_oracle as O
        self.convert_s = 0.0
        w = weights

        def f32(t):
            t0 = time.perf_counter()
            a = t.detach().to("cpu", torch.float32).numpy()
            self.convert_s += time.perf_counter() - t0
            return a

        nq, nk = shape.n_q_heads * shape.head_dim, shape.n_kv_heads * shape.head_dim

        def layer(l):
            wqkv = f32(w["wqkv"][l])
            return dict(wq=wqkv[:nq], wk=wqkv[nq:nq + nk], wv=wqkv[nq + nk:], wo=f32(w["wo"][l]),
                        w_gate=f32(w["w_gate"][l]), w_up=f32(w["w_up"][l]), w_down=f32(w["w_down"][l]),
                        norm1=f32(w["norm1"][l]), norm2=f32(w["norm2"][l]))

        self.model = O.Model(shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                             shape.d_ffn, shape.vocab, shape.vocab - 1, shape.rms_eps, shape.rope_theta,
                             f32(w["embed"]), f32(w["lm_head"]), f32(w["final_norm"]), layer)
        self.convert_s = 0.0


def oracle_sample(wl, weights, budget_s: float, lazy=None):
    """Runs the oracle on the workload's shortest request: denoise steps of its first block-cycle (the
    first one refreshes the whole row) until `budget_s` seconds of oracle time are spent or the block ends."""
    from oracle import blockserve_oracle as O
    lazy = lazy or _LazyOracleModel(wl.shape, weights)
    r = min(wl.requests, key=lambda q: q.p + q.g)
    req = O.new_request(lazy.model, r.req_id, r.prompt, r.g, r.alpha, wl.block_len, r.start_block, r.gen_prefix)
    req.kv_base = 0
    O.start_block_state(req, wl.block_len)
    spent, steps, committed = 0.0, 0, 0
    while req.mask and (steps == 0 or spent < budget_s):
        lazy.convert_s = 0.0
        t0 = time.perf_counter()
        rec = O.denoise_step(lazy.model, req, wl.block_len, wl.tau)
        spent += time.perf_counter() - t0 - lazy.convert_s
        committed += int(rec.committed.sum())
        steps += 1
    return dict(seconds=spent, steps=steps, committed=committed,
                sample=f"request {r.req_id} of {wl.name} (p={r.p}, g={r.g}, start block {r.start_block}): "
                       f"{steps} denoise step(s) of its first block-cycle, first one a whole-row refresh"), lazy


def cpu_baseline(wl, weights, budget_s: float):
    res, _ = oracle_sample(wl, weights, budget_s)
    return {"value": res["committed"] / res["seconds"], "unit": UNIT, "cores": torch.get_num_threads(),
            "kind": "oracle", "sample": res["sample"], "seconds": res["seconds"]}


def run_reference(args):
    rank, world, local = dist_env()
    if rank != 0:
        return
    wl = bs_inputs.workload(args.workload, seed=0)
    dev = f"cuda:{local}" if torch.cuda.is_available() else "cpu"
    weights = bs_inputs.make_weights(wl.shape, wl.weight_seed, device=dev)
    per_step = max(2.0, min(args.cpu_seconds, 150.0 / max(1, args.steps + args.warmup)))
    lazy = None
    for _ in range(args.warmup):
        _, lazy = oracle_sample(wl, weights, 0.0, lazy)
    t_total, committed, sample = 0.0, 0, ""
    for _ in range(args.steps):
        res, lazy = oracle_sample(wl, weights, per_step, lazy)
        t_total += res["seconds"]
        committed += res["committed"]
        sample = res["sample"]
    value = committed / t_total
    cores = torch.get_num_threads()
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * t_total / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32 arithmetic, activations rounded to bf16 at six points per layer",
        "data": "synthetic",
        "config": {"workload": wl.name, "sample_per_step": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def launch_ranks(n: int, argv, worker=None, check_devices: bool = True, timeout_s: float = 7200.0):
    """Starts `n` ranks of this script (or of `worker`, a command list, for tests) on one node, one GPU each, with
    the rendezvous variables torch.distributed expects, and returns [(returncode, stdout)] by rank.  Rank 0's
    stdout carries the JSON line."""
    import socket
    if n < 1:
        raise SystemExit("--gpus must be at least 1")
    if check_devices:
        have = torch.cuda.device_count()
        if n > have:
            raise SystemExit(f"--gpus {n} but this node has {have} CUDA device(s)")
    with socket.socket() as sock:          # a free port for the rendezvous
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = list(worker) if worker is not None else [sys.executable, os.path.abspath(__file__)]
    procs = []
    for rank in range(n):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(n), LOCAL_WORLD_SIZE=str(n),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen(cmd + list(argv), env=env, stdout=subprocess.PIPE, text=True))
    out = []
    for p in procs:
        try:
            so, _ = p.communicate(timeout=timeout_s)
        except subprocess.TimeoutExpired:
            p.kill()
            so, _ = p.communicate()
        out.append((p.returncode, so))
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", type=int, default=2)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-profile", action="store_true", help="skip the per-family CUDA-event timers (no roofline)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started plainly: this process only launches the ranks and relays rank 0's line
        results = launch_ranks(args.gpus, sys.argv[1:], check_devices=args.impl != "reference")
        sys.stdout.write(results[0][1])
        sys.stdout.flush()
        raise SystemExit(max(abs(rc) for rc, _ in results))
    if args.impl == "reference":
        run_reference(args)
    else:
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device: the engine has no CPU fallback")
        run_ours(args)


if __name__ == "__main__":
    main()
