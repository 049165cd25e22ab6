"""Seeded synthetic inputs for the mixed-state block-denoising iteration.

This module only *draws* inputs: model shapes, random-init weights, request
streams (prompt ids, lengths, logit scales, start blocks) and scheduler
parameters.  It holds none of the method's arithmetic, so that both the CPU
oracle and the CUDA path can be fed from it without sharing anything else.

Workloads stand in for the paper's benchmark runs (Section 3.1, Table 1):
prompt-length ranges, generation limits, block length L=32 and batch sizes
follow the shapes reported there; convergence heterogeneity is imitated by a
per-request logit scale alpha_i because random weights carry no text
statistics.  No dataset item is reproduced anywhere.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional

import numpy as np
import torch


@dataclasses.dataclass(frozen=True)
class ModelShape:
    name: str
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    init_std: float
    rms_eps: float = 1e-6
    rope_theta: float = 10000.0

    @property
    def mask_id(self) -> int:
        return self.vocab - 1

    @property
    def qkv_rows(self) -> int:
        return (self.n_q_heads + 2 * self.n_kv_heads) * self.head_dim

    def with_layers(self, n_layers: int) -> "ModelShape":
        return dataclasses.replace(self, n_layers=n_layers, name=f"{self.name}-{n_layers}L")

    def weight_bytes_bf16(self) -> int:
        per_layer = (self.qkv_rows * self.d_model + self.d_model * self.n_q_heads * self.head_dim
                     + 3 * self.d_ffn * self.d_model + 2 * self.d_model)
        return 2 * (self.n_layers * per_layer + 2 * self.vocab * self.d_model + self.d_model)


TINY = ModelShape("tiny", 2, 256, 4, 4, 64, 704, 1024, init_std=0.1)
DREAM_7B = ModelShape("dream7b", 28, 3584, 28, 4, 128, 18944, 152064, init_std=0.02)
LLADA_8B = ModelShape("llada8b", 32, 4096, 32, 32, 128, 12288, 126464, init_std=0.02)
# A narrow GQA shape used by small tests (several tiles, ragged tails, head_dim 128).
MINI_GQA = ModelShape("mini-gqa", 2, 384, 6, 2, 128, 1000, 2000, init_std=0.06)


@dataclasses.dataclass
class Request:
    req_id: int
    prompt: np.ndarray          # int32 [p]
    g: int                      # generation length
    alpha: float                # logit scale
    start_block: int = 0
    gen_prefix: Optional[np.ndarray] = None   # int32 [start_block * L] or None
    phase: int = 0              # 0: submitted before the first fill, 1: queued after it

    @property
    def p(self) -> int:
        return int(self.prompt.shape[0])


@dataclasses.dataclass
class Workload:
    name: str
    shape: ModelShape
    block_len: int
    tau: float
    token_budget: int           # beta of Eq. 1; <= 0 means unlimited
    max_batch: int
    requests: List[Request]
    weight_seed: int = 1000

    @property
    def max_row_tokens(self) -> int:
        return max(r.p + r.g for r in self.requests)

    def committed_target(self) -> int:
        """Tokens the engine itself has to commit (pre-committed start blocks excluded)."""
        return sum(r.g - r.start_block * self.block_len for r in self.requests)


def _ids(rng: np.random.Generator, n: int, vocab: int) -> np.ndarray:
    # uniform over every id except the mask id (= vocab - 1)
    return rng.integers(0, vocab - 1, size=n, dtype=np.int64).astype(np.int32)


def _finish(rng, shape, L, ps, gs, alphas, starts, phases=None) -> List[Request]:
    reqs = []
    for i, (p, g, a, k) in enumerate(zip(ps, gs, alphas, starts)):
        prompt = _ids(rng, int(p), shape.vocab)
        prefix = _ids(rng, int(k) * L, shape.vocab) if k > 0 else None
        reqs.append(Request(i, prompt, int(g), float(a), int(k), prefix,
                            0 if phases is None else int(phases[i])))
    return reqs


def workload(cfg: int, seed: int = 0, n_layers: Optional[int] = None,
             n_requests: Optional[int] = None) -> Workload:
    """The five benchmark-shaped workloads (1-based ``cfg``).

    Draw order per workload: prompt lengths, generation lengths, alpha, start
    blocks, then per request prompt ids followed by pre-committed block ids.
    ``n_layers`` builds a shallow replica of the same shape; ``n_requests``
    truncates the stream (the draws of the kept requests do not change).
    """
    rng = np.random.default_rng(seed)
    L = 32
    if cfg == 1:
        shape = TINY
        ps = [17, 40, 63, 9, 17, 40, 63, 9]
        al = [0.5, 2.0, 8.0, 32.0] * 2
        st = [0, 1, 2, 0, 0, 0, 0, 0]
        ph = [0, 0, 0, 0, 1, 1, 1, 1]
        reqs = _finish(rng, shape, L, ps, [96] * 8, al, st, ph)
        # the queued four draw their ids from seed + 1
        rng2 = np.random.default_rng(seed + 1)
        for r in reqs[4:]:
            r.prompt = _ids(rng2, r.p, shape.vocab)
        wl = Workload("cfg1-tiny", shape, L, 0.9, 0, 4, reqs)
    elif cfg == 2:
        shape = DREAM_7B
        n = 16
        ps = rng.integers(64, 513, size=n)
        al = rng.lognormal(1.5, 1.0, size=n)
        st = rng.integers(0, 8, size=n)
        wl = Workload("cfg2-dream-batch16", shape, L, 0.9, 0, 16,
                      _finish(rng, shape, L, ps, [256] * n, al, st))
    elif cfg == 3:
        shape = LLADA_8B
        n = 256
        mean, sd = 220.0, 90.0
        sigma2 = math.log(1.0 + (sd / mean) ** 2)
        mu = math.log(mean) - 0.5 * sigma2
        ps = np.clip(np.rint(rng.lognormal(mu, math.sqrt(sigma2), size=n)), 32, 1024).astype(np.int64)
        al = rng.lognormal(1.5, 1.0, size=n)
        wl = Workload("cfg3-llada-stream256", shape, L, 0.9, 16384, 1024,
                      _finish(rng, shape, L, ps, [256] * n, al, [0] * n))
    elif cfg == 4:
        shape = DREAM_7B
        n = 128
        ps = rng.integers(1024, 2049, size=n)
        al = rng.lognormal(1.0, 1.2, size=n)
        wl = Workload("cfg4-dream-long128", shape, L, 0.95, 65536, 1024,
                      _finish(rng, shape, L, ps, [512] * n, al, [0] * n))
    elif cfg == 5:
        shape = LLADA_8B
        n = 1024
        ps = rng.integers(64, 769, size=n)
        gs = rng.choice(np.array([128, 256, 512]), size=n)
        al = np.where(rng.random(size=n) < 0.8, 16.0, 0.7)
        wl = Workload("cfg5-llada-stragglers1024", shape, L, 0.9, 32768, 1024,
                      _finish(rng, shape, L, ps, gs, al, [0] * n))
    else:
        raise ValueError(f"unknown workload {cfg}")
    if n_layers is not None:
        wl.shape = wl.shape.with_layers(n_layers)
    if n_requests is not None:
        wl.requests = wl.requests[:n_requests]
    if wl.token_budget > 0:
        # a budget of beta admits at most beta / (smallest width) rows
        wl.max_batch = min(wl.max_batch, wl.token_budget // (min(r.p for r in wl.requests) + L))
    return wl


def custom_workload(shape: ModelShape, ps, gs, alphas, starts=None, *, L=32, tau=0.9,
                    token_budget=0, max_batch=None, seed=0, phases=None, name="custom") -> Workload:
    rng = np.random.default_rng(seed)
    n = len(ps)
    starts = [0] * n if starts is None else starts
    reqs = _finish(rng, shape, L, ps, gs, alphas, starts, phases)
    return Workload(name, shape, L, tau, token_budget, max_batch or n, reqs)


WEIGHT_NAMES = ("wqkv", "wo", "w_gate", "w_up", "w_down", "norm1", "norm2")


def make_weights(shape: ModelShape, seed: int = 1000, device: str = "cpu") -> Dict[str, object]:
    """Random-init weights, every value rounded to bf16 (so that a bf16 and an
    fp32 consumer see identical numbers).

    Returns ``embed [V,d]``, ``lm_head [V,d]``, ``final_norm [d]`` and per-layer
    lists ``wqkv [(Hq+2Hkv)*dh, d]`` (rows: all q heads, then k heads, then v
    heads), ``wo [d, Hq*dh]``, ``w_gate [ffn,d]``, ``w_up [ffn,d]``,
    ``w_down [d,ffn]``, ``norm1 [d]``, ``norm2 [d]`` as torch bf16 tensors on
    ``device``.  Matrices are N(0, init_std^2); norm gains are 1 + 0.1 N(0,1).
    The generator is torch's for the given device, so CPU and CUDA draws differ:
    a consumer that needs the same numbers elsewhere copies the tensors.
    """
    gen = torch.Generator(device=device)
    counter = [0]

    def mat(rows: int, cols: int) -> torch.Tensor:
        gen.manual_seed(seed + counter[0])
        counter[0] += 1
        w = torch.empty(rows, cols, dtype=torch.bfloat16, device=device)
        step = max(1, (1 << 26) // cols)
        for r0 in range(0, rows, step):       # chunked: bounded fp32 scratch
            r1 = min(rows, r0 + step)
            w[r0:r1] = (torch.randn(r1 - r0, cols, generator=gen, device=device, dtype=torch.float32)
                        * shape.init_std).to(torch.bfloat16)
        return w

    def gain(n: int) -> torch.Tensor:
        # gains jittered around 1 so that a misplaced or dropped gain shows up in parity
        gen.manual_seed(seed + counter[0])
        counter[0] += 1
        return (1.0 + 0.1 * torch.randn(n, generator=gen, device=device, dtype=torch.float32)
                ).to(torch.bfloat16)

    d, hd = shape.d_model, shape.n_q_heads * shape.head_dim
    out: Dict[str, object] = {
        "embed": mat(shape.vocab, d),
        "lm_head": mat(shape.vocab, d),
        "final_norm": gain(d),
    }
    for name in WEIGHT_NAMES:
        out[name] = []
    for _ in range(shape.n_layers):
        out["wqkv"].append(mat(shape.qkv_rows, d))
        out["wo"].append(mat(d, hd))
        out["w_gate"].append(mat(shape.d_ffn, d))
        out["w_up"].append(mat(shape.d_ffn, d))
        out["w_down"].append(mat(d, shape.d_ffn))
        out["norm1"].append(gain(d))
        out["norm2"].append(gain(d))
    return out


def weights_to_numpy_f32(weights: Dict[str, object]) -> Dict[str, object]:
    """Widen a weight dict to fp32 numpy arrays on the host (small models only)."""
    def cv(t):
        return t.detach().to("cpu", torch.float32).numpy()
    out = {}
    for k, v in weights.items():
        out[k] = [cv(t) for t in v] if isinstance(v, list) else cv(v)
    return out
