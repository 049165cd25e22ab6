"""Throughput-only ablations of the serving policy on a synthetic workload (Section 4's research questions on queue
order and block length, in the form that needs no trained weights): sorted vs submission-order queue, suffix
visibility FULL vs NONE, block length L, and optionally the transfer quota S < L of Section 2.5.  Prints one JSON line per variant and a markdown table.

    python -m paper_2607_08930_b200.ablate --workload 3
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import sys

import torch

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bs_inputs  # noqa: E402
from paper_2607_08930_b200 import binding as B, build  # noqa: E402


def run_variant(wl, weights, sort_queue: bool, suffix_mode: int, steps_per_block: int = 0,
                static_groups: bool = False, async_advance: bool = False, kv_capacity_tokens=None,
                refresh_policy: int = 0):
    eng = B.engine_for_workload(wl, weights, sort_queue=sort_queue, suffix_mode=suffix_mode,
                                steps_per_block=steps_per_block, static_groups=static_groups,
                                async_advance=async_advance, kv_capacity_tokens=kv_capacity_tokens,
                                refresh_policy=refresh_policy)
    for r in wl.requests:
        eng.admit(r.req_id, r.prompt, r.g, r.alpha, r.start_block, r.gen_prefix)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    ev0.record()
    eng.run()
    ev1.record()
    torch.cuda.synchronize()
    st = eng.stats()
    assert st.committed == wl.committed_target()
    ms = ev0.elapsed_time(ev1)
    out = dict(tokens_per_s=st.committed / (ms * 1e-3), job_s=ms * 1e-3, cycles=st.cycles, steps=st.steps,
               packed_tokens=st.packed_tokens, mean_active=st.sum_active / max(st.cycles, 1),
               effective_compute_ratio=st.sum_active / max(st.cycles, 1) / wl.max_batch,
               mean_active_per_step=st.active_row_steps / max(st.steps, 1),
               rows_working_per_step=st.row_steps / max(st.active_row_steps, 1))
    eng.close()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", type=int, default=3)
    ap.add_argument("--block-lens", type=int, nargs="*", default=[32, 16])
    ap.add_argument("--static-groups", action="store_true",
                    help="add the comparison policy: fixed groups in submission order, no refill until a group is done")
    ap.add_argument("--requests", type=int, default=0, help="use only the first N requests of the workload")
    ap.add_argument("--async-advance", action="store_true",
                    help="add the per-row block advance and the refresh-at-admission variant (sorted queue, full "
                         "suffix) beside the synchronous cycles")
    ap.add_argument("--kv-rows", type=int, default=0, help="rows of the KV arena (0: sized from the workload)")
    ap.add_argument("--steps-per-block", type=int, nargs="*", default=[],
                    help="extra variants with a transfer quota S < L (sorted queue, full suffix)")
    args = ap.parse_args()
    build.build()
    base = bs_inputs.workload(args.workload)
    if args.requests:
        base = dataclasses.replace(base, requests=base.requests[:args.requests])
    weights = bs_inputs.make_weights(base.shape, base.weight_seed, device="cuda:0")
    rows = []
    for L in args.block_lens:
        if L != base.block_len and any(r.start_block for r in base.requests):
            continue            # pre-committed start blocks are stated in units of the workload's own L
        wl = dataclasses.replace(base, block_len=L)
        for sort_queue in (True, False):
            for suffix_mode in (B.SUFFIX_FULL, B.SUFFIX_NONE):
                run_variant(wl, weights, sort_queue, suffix_mode)          # warm-up
                res = run_variant(wl, weights, sort_queue, suffix_mode)
                res.update(workload=wl.name, block_len=L, queue="sorted" if sort_queue else "submission order",
                           suffix="full" if suffix_mode == B.SUFFIX_FULL else "none")
                print(json.dumps(res), flush=True)
                rows.append(res)
    for S in args.steps_per_block:
        run_variant(base, weights, True, B.SUFFIX_FULL, S)
        res = run_variant(base, weights, True, B.SUFFIX_FULL, S)
        res.update(workload=base.name, block_len=base.block_len, queue=f"sorted, S = {S}", suffix="full")
        print(json.dumps(res), flush=True)
        rows.append(res)
    if args.async_advance:
        for name, kw in (("sorted, synchronous block cycles (Algorithm 1)", dict()),
                         ("sorted, per-row block advance", dict(async_advance=True)),
                         ("sorted, cache rebuilt at admission only", dict(refresh_policy=B.REFRESH_AT_ADMISSION)),
                         ("sorted, per-row advance + cache rebuilt at admission only",
                          dict(async_advance=True, refresh_policy=B.REFRESH_AT_ADMISSION))):
            kw.update(kv_capacity_tokens=args.kv_rows or None)
            run_variant(base, weights, True, B.SUFFIX_FULL, **kw)
            res = run_variant(base, weights, True, B.SUFFIX_FULL, **kw)
            res.update(workload=base.name, block_len=base.block_len, queue=name, suffix="full")
            print(json.dumps(res), flush=True)
            rows.append(res)
    if args.static_groups:
        for name, kw in (("block-boundary refill, submission order", dict(sort_queue=False)),
                         ("static groups, submission order", dict(sort_queue=False, static_groups=True))):
            run_variant(base, weights, suffix_mode=B.SUFFIX_FULL, **kw)
            res = run_variant(base, weights, suffix_mode=B.SUFFIX_FULL, **kw)
            res.update(workload=base.name, block_len=base.block_len, queue=name, suffix="full")
            print(json.dumps(res), flush=True)
            rows.append(res)
    print("\n| L | queue | suffix | committed tokens/s | job s | cycles | steps | packed tokens | mean |A| per step | "
          "share of active rows working |")
    print("|---|---|---|---|---|---|---|---|---|---|")
    for r in rows:
        print(f"| {r['block_len']} | {r['queue']} | {r['suffix']} | {r['tokens_per_s']:.0f} | {r['job_s']:.1f} | "
              f"{r['cycles']} | {r['steps']} | {r['packed_tokens']} | {r['mean_active_per_step']:.1f} | "
              f"{r['rows_working_per_step']:.3f} |")


if __name__ == "__main__":
    main()
