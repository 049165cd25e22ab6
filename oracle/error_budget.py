"""Error budget of the oracle's bf16 mode (TEST INFRASTRUCTURE, CPU only).

For one request of a workload, the logits of the block-start refresh step are
computed in pure fp32 and in the bf16 mode, then with each of the six rounding
points switched off (or on) one at a time.  Printed per variant: the maximum
over masked rows of  max_v |z - z_fp32| / max_v |z_fp32|  (the parity
tolerance's measure) and the same for the confidences.  Calls only the oracle
and the seeded input generators.

    python -m oracle.error_budget --workload 1
    python -m oracle.error_budget --workload 2 --layers 2
    python -m oracle.error_budget --workload 2            # full depth: minutes, ~45 GB of host memory
"""
from __future__ import annotations

import argparse
import dataclasses
import os
import sys
import time

import numpy as np
import torch

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bs_inputs  # noqa: E402
from oracle import blockserve_oracle as O  # noqa: E402


def lazy_model(shape, weights) -> O.Model:
    """Oracle model over bf16 torch weights; a layer is widened to fp32 when it is asked for (not kept)."""
    def f32(t):
        return t.detach().to("cpu", torch.float32).numpy()

    nq, nk = shape.n_q_heads * shape.head_dim, shape.n_kv_heads * shape.head_dim

    def layer(l):
        wqkv = f32(weights["wqkv"][l])
        out = dict(wq=wqkv[:nq], wk=wqkv[nq:nq + nk], wv=wqkv[nq + nk:])
        for name in ("wo", "w_gate", "w_up", "w_down", "norm1", "norm2"):
            out[name] = f32(weights[name][l])
        return out

    return O.Model(shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.d_ffn,
                   shape.vocab, shape.vocab - 1, shape.rms_eps, shape.rope_theta, f32(weights["embed"]),
                   f32(weights["lm_head"]), f32(weights["final_norm"]), layer)


def refresh_logits(model: O.Model, req, L: int):
    r = O.new_request(model, req.req_id, req.prompt, req.g, req.alpha, L, req.start_block, req.gen_prefix)
    O.start_block_state(r, L)
    rec = O.denoise_step(model, r, L, tau=2.0, keep_logits=True)      # tau > 1: the commit plays no role here
    return rec.logits, rec.conf


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", type=int, default=1)
    ap.add_argument("--layers", type=int, default=0, help="shallow replica with this many layers (0: full depth)")
    ap.add_argument("--requests", type=int, nargs="*", help="request ids (default: the shortest row)")
    args = ap.parse_args()
    wl = bs_inputs.workload(args.workload, n_layers=args.layers or None)
    weights = bs_inputs.make_weights(wl.shape, wl.weight_seed)
    base = lazy_model(wl.shape, weights)
    ids = args.requests or [min(wl.requests, key=lambda q: q.p + q.g).req_id]
    variants = [("pure fp32", False, frozenset()), ("all six points (bf16 mode)", True, frozenset(O.ROUNDING_POINTS))]
    variants += [(f"all but '{p}'", True, frozenset(O.ROUNDING_POINTS) - {p}) for p in O.ROUNDING_POINTS]
    variants += [(f"only '{p}'", True, frozenset({p})) for p in O.ROUNDING_POINTS]
    for rid in ids:
        req = wl.requests[rid]
        print(f"# {wl.name}, {wl.shape.n_layers} layers, request {rid}: p={req.p} g={req.g} alpha={req.alpha:.3g} "
              f"start block {req.start_block}")
        ref = None
        for name, on, pts in variants:
            t0 = time.perf_counter()
            z, c = refresh_logits(dataclasses.replace(base, bf16_activations=on, bf16_points=pts), req, wl.block_len)
            if ref is None:
                ref = (z, c)
                print(f"{name:34s} reference  max|z| {np.abs(z).max():.3f}  ({time.perf_counter() - t0:.1f} s)")
                continue
            zerr = float((np.abs(z - ref[0]).max(-1) / np.abs(ref[0]).max(-1)).max())
            cerr = float((np.abs(c - ref[1]) / ref[1]).max())
            print(f"{name:34s} logit err {zerr:.3e}  conf err {cerr:.3e}  ({time.perf_counter() - t0:.1f} s)", flush=True)


if __name__ == "__main__":
    main()
