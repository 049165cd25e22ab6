"""CPU oracle for the mixed-state block-denoising iteration (TEST INFRASTRUCTURE).

A plain, slow, fp32 numpy implementation of what the serving loop computes,
written from the paper's method section and taken step by step in its order:
request state (Section 2.1), the scheduling loop (Algorithm 1), the
bounding-box admission cost (Eq. 1, Section 2.4), explicit position ids and
gather / scatter execution with a dual KV cache (Section 2.5), confidence
thresholded parallel unmasking (related-work description of the dual cache and
parallel decoding), and the effective compute ratio (Eq. 2).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It shares no code with the CUDA path: no kernels, headers,
tables or helpers.  There is no blocking, fusion or reordering beyond what the
definitions state; numpy's matmul, exp, sort and argmax serve as primitives.

Precision: the paper runs its models in bfloat16 (Section 3.1).  Arithmetic
here is fp32 (weights hold bf16-representable values).  Two modes:
  * ``bf16_activations=False``: pure fp32, nothing is rounded.  This is the
    oracle the parity tolerance (2e-2 on logits and confidences) is worded for.
  * ``bf16_activations=True`` (the default of ``Model``): six activation
    tensors per layer are rounded to bf16 (nearest even) where a bf16 pipeline
    stores them between operators - ROUNDING_POINTS below: the normed hidden
    states, q / k / v, the rotated q / k, the attention output, the SwiGLU
    product and the final normed state.  The residual stream, attention
    scores and probabilities, gate and up separately, accumulations, logits
    and confidences stay fp32.  This rounding map is that of the CUDA path's
    HBM tensors, not a statement of the paper: it was adopted together with
    the first kernels so that trajectories of the two sides stay comparable
    (it removes the systematic part of their difference; rounding is
    discontinuous, so the two still drift apart by a fraction of a bf16 ulp
    per operator).  Parity tests report against both modes.
``Model.bf16_points`` selects a subset of the points (error budgets).

Readings taken where the paper is silent (each is listed in the design notes):
  * the model is a pre-norm bidirectional transformer (RMSNorm, rotate-half
    RoPE, GQA, SwiGLU, no biases), logits = alpha_i * norm_f(x) @ W_lm^T;
  * the cache of a request is rebuilt by a full-row forward at the first step
    of every block; later steps of the block forward only the block's tokens,
    rewrite their K/V in place and attend over the cached prefix and suffix
    (``refresh_at_admission_only`` is an ablation variant: only the first step
    after admission is such a forward, the other "frozen prefix" reading);
  * commit rule: strictly conf > tau, plus always the masked position of
    highest confidence (lowest position on ties); argmax over the vocabulary
    takes the lowest id on ties and never the mask id;
  * block-cycles are batch-synchronous as in Algorithm 1.  ``async_advance``
    relaxes exactly that (the straggler effect of Section 2.3: a row whose
    block is done idles until the slowest row of the cycle is): after every
    denoise step each row whose block is complete moves to its next block on
    its own (or leaves), survivors keep their order, and the head of P is
    admitted under the same Eq. 1 rule; a row's own sequence of steps - refresh
    at the first step of each block, cached steps after it - does not change,
    so its tokens are those of the synchronous policy bit for bit.

Whole-trajectory token values for n_layers >= 2 are "parity unpinned" (the
paper prints no worked numeric example); every component and every special
case is pinned by tests/test_oracle_pins.py.
"""
from __future__ import annotations

import dataclasses
from typing import Callable, Dict, List, Optional, Sequence

import numpy as np

F32 = np.float32
# where the bf16 mode rounds an activation tensor (see the module docstring)
ROUNDING_POINTS = ("normed", "qkv", "rope", "attn", "swiglu", "final")
SUFFIX_FULL = 0     # row = prompt + all g positions; future blocks visible as mask tokens
SUFFIX_NONE = 1     # row ends with the current block (Section 2.4's row width)


# --------------------------------------------------------------------------- #
# model pieces
# --------------------------------------------------------------------------- #

@dataclasses.dataclass
class Model:
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    mask_id: int
    rms_eps: float
    rope_theta: float
    embed: np.ndarray            # [V, d]
    lm_head: np.ndarray          # [V, d]
    final_norm: np.ndarray       # [d]
    layer: Callable[[int], Dict[str, np.ndarray]]   # l -> wq wk wv wo w_gate w_up w_down norm1 norm2
    bf16_activations: bool = True
    bf16_points: frozenset = frozenset(ROUNDING_POINTS)

    def act(self, x: np.ndarray, point: str) -> np.ndarray:
        """Storage precision of the activation tensor at a named rounding point."""
        assert point in ROUNDING_POINTS
        if self.bf16_activations and point in self.bf16_points:
            return round_bf16(x)
        return np.asarray(x, dtype=F32)


def round_bf16(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bfloat16 (ties to even), returned as fp32."""
    a = np.ascontiguousarray(x, dtype=F32)
    u = a.view(np.uint32).astype(np.uint64)
    r = ((u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000).astype(np.uint32)
    out = r.view(F32).reshape(a.shape)
    bad = ~np.isfinite(a)
    if bad.any():
        out = np.where(bad, a, out)
    return out


def model_from_weights(shape, w: Dict[str, object], bf16_activations: bool = True) -> Model:
    """Build a Model from fp32 numpy weights laid out as the input generator
    documents (wqkv rows: q heads, k heads, v heads)."""
    nq = shape.n_q_heads * shape.head_dim
    nk = shape.n_kv_heads * shape.head_dim

    def layer(l: int) -> Dict[str, np.ndarray]:
        wqkv = np.asarray(w["wqkv"][l], dtype=F32)
        return dict(wq=wqkv[:nq], wk=wqkv[nq:nq + nk], wv=wqkv[nq + nk:],
                    wo=np.asarray(w["wo"][l], dtype=F32),
                    w_gate=np.asarray(w["w_gate"][l], dtype=F32),
                    w_up=np.asarray(w["w_up"][l], dtype=F32),
                    w_down=np.asarray(w["w_down"][l], dtype=F32),
                    norm1=np.asarray(w["norm1"][l], dtype=F32),
                    norm2=np.asarray(w["norm2"][l], dtype=F32))

    return Model(shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                 shape.d_ffn, shape.vocab, shape.vocab - 1, shape.rms_eps, shape.rope_theta,
                 np.asarray(w["embed"], dtype=F32), np.asarray(w["lm_head"], dtype=F32),
                 np.asarray(w["final_norm"], dtype=F32), layer, bf16_activations)


def rmsnorm(x: np.ndarray, w: np.ndarray, eps: float) -> np.ndarray:
    """y = w * x / sqrt(mean(x^2) + eps), row-wise."""
    x = x.astype(F32)
    ms = np.mean(x * x, axis=-1, keepdims=True, dtype=F32)
    return (x / np.sqrt(ms + F32(eps))).astype(F32) * w.astype(F32)


def silu(x: np.ndarray) -> np.ndarray:
    x = x.astype(F32)
    return x / (F32(1.0) + np.exp(-x))


def rope_cos_sin(pos: np.ndarray, head_dim: int, theta: float):
    """Angles pos * theta^(-2j/head_dim), j = 0..head_dim/2-1, evaluated in
    double and rounded once to fp32 (the relative-distance encoding of
    Section 2.5's logical positional alignment)."""
    j = np.arange(head_dim // 2, dtype=np.float64)
    inv = np.power(float(theta), -2.0 * j / float(head_dim))
    ang = pos.astype(np.float64)[:, None] * inv[None, :]
    return np.cos(ang).astype(F32), np.sin(ang).astype(F32)


def apply_rope(x: np.ndarray, cos: np.ndarray, sin: np.ndarray) -> np.ndarray:
    """Rotate-half pairing: dims (j, j + head_dim/2) are rotated by the angle of j.
    x: [n, H, head_dim]; cos, sin: [n, head_dim/2]."""
    h = x.shape[-1] // 2
    x1, x2 = x[..., :h], x[..., h:]
    c, s = cos[:, None, :], sin[:, None, :]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1).astype(F32)


def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray) -> np.ndarray:
    """Bidirectional softmax attention, no mask.  q: [nq, Hq, dh]; k, v:
    [nk, Hkv, dh]; query head h reads kv head h // (Hq/Hkv).  Returns [nq, Hq, dh]."""
    nq, hq, dh = q.shape
    hkv = k.shape[1]
    group = hq // hkv
    out = np.empty_like(q, dtype=F32)
    scale = F32(1.0 / np.sqrt(float(dh)))
    for h in range(hq):
        kh = h // group
        s = (q[:, h, :] @ k[:, kh, :].T).astype(F32) * scale           # [nq, nk]
        s = s - s.max(axis=-1, keepdims=True)
        e = np.exp(s, dtype=F32)
        pr = e / e.sum(axis=-1, keepdims=True, dtype=F32)
        out[:, h, :] = pr @ v[:, kh, :]
    return out


def confidence(logits: np.ndarray, mask_id: int):
    """Per row of fp32 logits: the mask id can never be produced; token =
    argmax (lowest id on ties); confidence = softmax probability of that token
    = exp(max - logsumexp).  Returns (tok int32 [n], conf fp32 [n])."""
    z = np.array(logits, dtype=F32, copy=True)
    z[:, mask_id] = -np.inf
    tok = np.argmax(z, axis=-1).astype(np.int32)          # first occurrence = lowest id
    m = z.max(axis=-1).astype(F32)
    se = np.sum(np.exp(z - m[:, None], dtype=F32), axis=-1, dtype=F32)
    lse = (m + np.log(se, dtype=F32)).astype(F32)
    conf = np.exp(m - lse, dtype=F32)
    return tok, conf


def transfer_quota(L: int, S: int, s: int) -> int:
    """Per-step transfer quota of Section 2.5: the L masked tokens a block starts
    with are spread uniformly over S diffusion steps, the first L mod S steps
    taking one more.  S = L gives one token per step."""
    if s >= S:
        return 1
    return L // S + (1 if s < L % S else 0)


def commit_set(conf: np.ndarray, tau: float, quota: int = 1) -> np.ndarray:
    """Boolean mask over the still-masked positions of one block (in position
    order): everything strictly above tau, plus the ``quota`` positions of
    highest confidence (lower position first on ties), so that every step
    commits at least its quota (all that is left, if fewer remain)."""
    sel = conf > F32(tau)
    order = np.argsort(-conf, kind="stable")
    sel[order[:max(int(quota), 1)]] = True
    return sel


# --------------------------------------------------------------------------- #
# per-request state and the denoise step
# --------------------------------------------------------------------------- #

@dataclasses.dataclass
class ReqState:
    req_id: int
    p: int
    g: int
    alpha: float
    tokens: np.ndarray                 # int32 [p + g]; masked positions hold mask_id
    b: int                             # current block index
    s: int = 0                         # step inside the block (0 = refresh step)
    mask: int = 0                      # bit j set <=> block position j still masked
    kv_base: int = -1                  # physical first row of the KV slab
    K: Optional[List[np.ndarray]] = None    # per layer [p+g, Hkv, dh]
    V: Optional[List[np.ndarray]] = None
    committed: int = 0                 # tokens committed by the engine
    steps: int = 0
    admit_order: int = 0
    needs_refresh: bool = True         # the block's first step forwards the whole row (rebuilds the cache)
    refreshes: int = 0                 # whole-row forwards this request has had

    def n_blocks(self, L: int) -> int:
        return -(-self.g // L)         # K_i = ceil(g_i / L), Section 2.1

    def block_range(self, L: int):
        lo = self.p + self.b * L
        return lo, min(lo + L, self.p + self.g)

    def vis(self, L: int, suffix_mode: int) -> int:
        return self.p + self.g if suffix_mode == SUFFIX_FULL else self.block_range(L)[1]

    def width(self, L: int) -> int:
        return self.p + (self.b + 1) * L       # row width of Eq. 1


def new_request(model: Model, req_id: int, prompt: Sequence[int], g: int, alpha: float, L: int,
                start_block: int = 0, gen_prefix: Optional[Sequence[int]] = None) -> ReqState:
    p = len(prompt)
    tokens = np.full(p + g, model.mask_id, dtype=np.int32)
    tokens[:p] = np.asarray(prompt, dtype=np.int32)
    if start_block > 0:
        tokens[p:p + start_block * L] = np.asarray(gen_prefix, dtype=np.int32)[:start_block * L]
    return ReqState(req_id, p, g, float(alpha), tokens, start_block)


def start_block_state(r: ReqState, L: int) -> None:
    lo, hi = r.block_range(L)
    r.s = 0
    r.mask = (1 << (hi - lo)) - 1      # every block starts fully masked (Section 2.5)


def _alloc_cache(model: Model, r: ReqState) -> None:
    n = r.p + r.g
    r.K = [np.zeros((n, model.n_kv_heads, model.head_dim), dtype=F32) for _ in range(model.n_layers)]
    r.V = [np.zeros((n, model.n_kv_heads, model.head_dim), dtype=F32) for _ in range(model.n_layers)]


def forward_queries(model: Model, r: ReqState, qpos: np.ndarray, vis: int) -> np.ndarray:
    """Forward the tokens at positions ``qpos`` of request r.  At each layer the
    fresh K/V of the query positions are first written into the cache in place
    (only those rows), then every query attends over cache rows [0, vis).
    Position id of a token = its index in the request's own row (first prompt
    token is position 0).  Returns the final residual stream [len(qpos), d]."""
    if r.K is None:
        _alloc_cache(model, r)
    x = model.embed[r.tokens[qpos]].astype(F32)
    cos, sin = rope_cos_sin(qpos, model.head_dim, model.rope_theta)
    n = len(qpos)
    for l in range(model.n_layers):
        w = model.layer(l)
        h = model.act(rmsnorm(x, w["norm1"], model.rms_eps), "normed")
        q = model.act(h @ w["wq"].T, "qkv").reshape(n, model.n_q_heads, model.head_dim)
        k = model.act(h @ w["wk"].T, "qkv").reshape(n, model.n_kv_heads, model.head_dim)
        v = model.act(h @ w["wv"].T, "qkv").reshape(n, model.n_kv_heads, model.head_dim)
        q = model.act(apply_rope(q, cos, sin), "rope")
        k = model.act(apply_rope(k, cos, sin), "rope")
        r.K[l][qpos] = k
        r.V[l][qpos] = v
        a = model.act(attention(q, r.K[l][:vis], r.V[l][:vis]), "attn").reshape(n, -1)
        x = x + (a @ w["wo"].T).astype(F32)
        h2 = model.act(rmsnorm(x, w["norm2"], model.rms_eps), "normed")
        act = model.act(silu(h2 @ w["w_gate"].T) * (h2 @ w["w_up"].T).astype(F32), "swiglu")
        x = x + (act @ w["w_down"].T).astype(F32)
    return x


def full_forward_logits(model: Model, tokens: np.ndarray, alpha: float) -> np.ndarray:
    """Cache-less forward of a whole row (used by pins): logits [n, V]."""
    tmp = ReqState(-1, len(tokens), 0, alpha, np.asarray(tokens, dtype=np.int32), 0)
    x = forward_queries(model, tmp, np.arange(len(tokens)), len(tokens))
    return lm_logits(model, x, alpha)


def lm_logits(model: Model, x: np.ndarray, alpha: float) -> np.ndarray:
    hf = model.act(rmsnorm(x, model.final_norm, model.rms_eps), "final")
    return (F32(alpha) * (hf @ model.lm_head.T).astype(F32)).astype(F32)


@dataclasses.dataclass
class StepRecord:
    req_id: int
    block: int
    step: int
    positions: np.ndarray      # absolute positions of the still-masked block slots (ascending)
    logits: Optional[np.ndarray]   # [n_masked, V] fp32 (kept only when asked)
    tok: np.ndarray            # int32 [n_masked]
    conf: np.ndarray           # fp32 [n_masked]
    committed: np.ndarray      # bool [n_masked]
    top2_gap: np.ndarray       # fp32 [n_masked]: best minus runner-up logit


def denoise_step(model: Model, r: ReqState, L: int, tau: float, suffix_mode: int = SUFFIX_FULL,
                 keep_logits: bool = False, override_commit: Optional[np.ndarray] = None,
                 override_tok: Optional[np.ndarray] = None, steps_per_block: Optional[int] = None) -> StepRecord:
    """One denoise step of one active request whose block is not done.

    ``override_commit`` / ``override_tok`` let a lockstep comparison make the
    oracle adopt another implementation's decision at excluded near-tie
    positions; they never change what the oracle *computes* and reports."""
    lo, hi = r.block_range(L)
    vis = r.vis(L, suffix_mode)
    refresh = r.s == 0 and r.needs_refresh
    r.refreshes += int(refresh)
    qpos = np.arange(0, vis) if refresh else np.arange(lo, hi)
    x = forward_queries(model, r, qpos, vis)
    slots = np.array([j for j in range(hi - lo) if (r.mask >> j) & 1], dtype=np.int64)
    positions = lo + slots
    rows = positions if refresh else slots
    logits = lm_logits(model, x[rows], r.alpha)
    tok, conf = confidence(logits, model.mask_id)
    z = np.array(logits, copy=True)
    z[:, model.mask_id] = -np.inf
    part = np.partition(z, -2, axis=-1)
    gap = (part[:, -1] - part[:, -2]).astype(F32)
    S = L if not steps_per_block else int(steps_per_block)
    sel = commit_set(conf.copy(), tau, transfer_quota(L, S, r.s))
    rec = StepRecord(r.req_id, r.b, r.s, positions, logits if keep_logits else None,
                     tok.copy(), conf.copy(), sel.copy(), gap)
    use_sel = sel if override_commit is None else np.asarray(override_commit, dtype=bool)
    use_tok = tok if override_tok is None else np.asarray(override_tok, dtype=np.int32)
    for i, j in enumerate(slots):
        if use_sel[i]:
            r.tokens[lo + j] = use_tok[i]
            r.mask &= ~(1 << int(j))
            r.committed += 1
    r.s += 1
    r.steps += 1
    return rec


# --------------------------------------------------------------------------- #
# scheduler: Algorithm 1, Eq. 1, sorted queue, compaction, KV slabs
# --------------------------------------------------------------------------- #

def batch_cost(widths: Sequence[int]) -> int:
    """Eq. 1: |A| * max_i (p_i + (b_i + 1) L)."""
    return 0 if len(widths) == 0 else len(widths) * max(widths)


def first_fit(slabs: Sequence[tuple], need: int, capacity: int) -> int:
    """Lowest row at which ``need`` contiguous rows are free, or -1."""
    start = 0
    for base, n in sorted(slabs):
        if base - start >= need:
            break
        start = max(start, base + n)
    return start if start + need <= capacity else -1


@dataclasses.dataclass
class CycleTrace:
    n_active: int
    width: int
    cost: int
    evicted: List[int]
    admitted: List[int]
    row_ids: List[int]


class Scheduler:
    """Integer-only serving state: pending queue P (ascending prompt length,
    ties by submission order), active rows A, the admission rule and the
    block-boundary advance / evict / stable compaction / refill."""

    def __init__(self, L: int, token_budget: int, max_batch: int, kv_capacity: int,
                 sort_queue: bool = True, eos_id: Optional[int] = None, static_groups: bool = False,
                 async_advance: bool = False, refresh_at_admission_only: bool = False):
        self.L, self.beta, self.max_batch, self.kv_capacity = L, token_budget, max_batch, kv_capacity
        # ablation variant: the cache is rebuilt once, by the first step after admission; later blocks begin with a
        # cached block step (prefix and suffix K/V stay as earlier steps left them)
        self.refresh_at_admission_only = bool(refresh_at_admission_only)
        self.sort_queue = sort_queue
        self.static_groups = bool(static_groups)     # comparison policy of Section 3.1: fixed groups, no refill
        self.async_advance = bool(async_advance)     # per-row block advance after every step (Section 2.3 relaxed)
        assert not (self.static_groups and self.async_advance)
        self.row_steps = 0                           # sum over denoise steps of the rows that ran a forward
        self.eos_id = None if eos_id is None or eos_id < 0 else int(eos_id)
        self.pending: List[ReqState] = []
        self.active: List[ReqState] = []
        self.finished: List[ReqState] = []
        self.trace: List[CycleTrace] = []
        self._n_submitted = 0

    def fits_alone(self, p: int, start_block: int) -> bool:
        return self.beta <= 0 or p + (start_block + 1) * self.L <= self.beta

    def submit(self, r: ReqState) -> None:
        if not self.fits_alone(r.p, r.b):
            raise ValueError("request wider than the token budget")
        if r.p + r.g > self.kv_capacity:
            raise ValueError("request longer than the KV arena")
        r.admit_order = self._n_submitted
        self._n_submitted += 1
        self.pending.append(r)
        if self.sort_queue:
            self.pending.sort(key=lambda q: (q.p, q.admit_order))

    def evict_refill(self, first: bool = False, only_done: bool = False):
        """Block boundary: b_i += 1 for every active row (not on the very first
        fill of a row), evict rows with b_i >= K_i or CheckEOS(r_i) (Algorithm 1:
        an end-of-sequence token among the blocks generated so far; off when
        no eos_id is configured), keep survivors in order,
        then admit the head of P while Eq. 1 stays within the budget, the batch
        cap holds and the KV arena has a hole; admitted rows are appended.

        ``only_done`` (the per-row advance of ``async_advance``, called after
        every denoise step): rows whose block is not complete stay as they are -
        same block, same step counter, same mask word - and only rows with an
        empty mask word advance; everything else is the same rule."""
        L = self.L
        evicted, survivors = [], []
        started = []                      # rows that begin a block now
        for r in self.active:
            if only_done and r.mask != 0:
                survivors.append(r)
                continue
            r.b += 1
            done_upto = min(r.p + r.b * L, r.p + r.g)
            has_eos = self.eos_id is not None and bool((r.tokens[r.p:done_upto] == self.eos_id).any())
            if r.b >= r.n_blocks(L) or has_eos:
                evicted.append(r.req_id)
                r.kv_base = -1
                self.finished.append(r)
            else:
                survivors.append(r)
                started.append(r)
                r.needs_refresh = not self.refresh_at_admission_only
        self.active = survivors
        admitted = []
        # static groups: the next group starts only when every request of the current one has finished
        refill = not (self.static_groups and self.active)
        while refill and self.pending and len(self.active) < self.max_batch:
            c = self.pending[0]
            widths = [r.width(L) for r in self.active] + [c.width(L)]
            if self.beta > 0 and batch_cost(widths) > self.beta:
                break
            base = first_fit([(r.kv_base, r.p + r.g) for r in self.active], c.p + c.g, self.kv_capacity)
            if base < 0:
                break
            c.kv_base = base
            self.pending.pop(0)
            self.active.append(c)
            started.append(c)
            c.needs_refresh = True
            admitted.append(c.req_id)
        for r in started:
            start_block_state(r, L)
        widths = [r.width(L) for r in self.active]
        self.trace.append(CycleTrace(len(self.active), max(widths) if widths else 0, batch_cost(widths),
                                     evicted, admitted, [r.req_id for r in self.active]))
        return evicted, admitted

    def advance_finished(self):
        """async_advance: the step boundary.  Rows whose block is complete advance or leave, the queue refills."""
        return self.evict_refill(only_done=True)

    def effective_compute_ratio(self, nominal_batch: int) -> float:
        """Eq. 2: R = (1 / (T B)) * sum_t a_t over the cycles that ran."""
        a = [t.n_active for t in self.trace if t.n_active > 0]
        return float(sum(a)) / (len(a) * nominal_batch) if a else 0.0


def build_indices(active: Sequence[ReqState], L: int, suffix_mode: int = SUFFIX_FULL):
    """Gather / scatter index arrays of one step, for the rows of A in order.

    cu_q[i]..cu_q[i+1] is row i's span in the packed token list (whole visible
    row on a refresh step, the active block otherwise, nothing if the block is
    done); tok_row / tok_pos / tok_kv give, per packed token, its row, its
    logical position id and its physical KV row; lm_tok lists the packed
    indices of still-masked block positions (row order, then position order)
    with lm_row and lm_slot (bit index inside the block)."""
    cu_q = [0]
    tok_row, tok_pos, tok_kv, lm_tok, lm_row, lm_slot = [], [], [], [], [], []
    for i, r in enumerate(active):
        lo, hi = r.block_range(L)
        if r.mask == 0:
            qpos = range(0)
        elif r.s == 0 and r.needs_refresh:
            qpos = range(0, r.vis(L, suffix_mode))
        else:
            qpos = range(lo, hi)
        base = cu_q[-1]
        for pos in qpos:
            tok_row.append(i)
            tok_pos.append(pos)
            tok_kv.append(r.kv_base + pos)
        if r.mask != 0:
            for j in range(hi - lo):
                if (r.mask >> j) & 1:
                    lm_tok.append(base + (lo + j - qpos[0]))
                    lm_row.append(i)
                    lm_slot.append(j)
        cu_q.append(base + len(qpos))
    i32 = lambda a: np.asarray(a, dtype=np.int32)
    return dict(cu_q=i32(cu_q), tok_row=i32(tok_row), tok_pos=i32(tok_pos), tok_kv=i32(tok_kv),
                lm_tok=i32(lm_tok), lm_row=i32(lm_row), lm_slot=i32(lm_slot))


# --------------------------------------------------------------------------- #
# the engine: scheduler + model, driven like the C-ABI
# --------------------------------------------------------------------------- #

class Engine:
    def __init__(self, model: Model, L: int, tau: float, token_budget: int, max_batch: int,
                 kv_capacity: int, suffix_mode: int = SUFFIX_FULL, sort_queue: bool = True,
                 steps_per_block: Optional[int] = None, eos_id: Optional[int] = None, static_groups: bool = False,
                 async_advance: bool = False, refresh_at_admission_only: bool = False):
        self.model, self.L, self.tau, self.suffix_mode = model, L, tau, suffix_mode
        self.steps_per_block = steps_per_block
        self.async_advance = bool(async_advance)
        self.sched = Scheduler(L, token_budget, max_batch, kv_capacity, sort_queue, eos_id, static_groups,
                               async_advance, refresh_at_admission_only)
        self.by_id: Dict[int, ReqState] = {}
        self.total_committed = 0
        self.total_steps = 0

    def admit(self, req_id, prompt, g, alpha, start_block=0, gen_prefix=None) -> None:
        r = new_request(self.model, req_id, prompt, g, alpha, self.L, start_block, gen_prefix)
        self.sched.submit(r)
        self.by_id[req_id] = r

    def evict_refill(self):
        ev, ad = self.sched.evict_refill()
        for rid in ev:                      # an evicted request keeps its tokens, drops its cache
            self.by_id[rid].K = self.by_id[rid].V = None
        return ev, ad, len(self.sched.active)

    def step_boundary(self):
        """async_advance: after a denoise step, finished rows advance or leave and the queue refills."""
        ev, ad = self.sched.advance_finished()
        for rid in ev:
            self.by_id[rid].K = self.by_id[rid].V = None
        return ev, ad, len(self.sched.active)

    def denoise_step(self, keep_logits: bool = False) -> List[StepRecord]:
        recs = []
        self.sched.row_steps += sum(1 for r in self.sched.active if r.mask != 0)
        for r in self.sched.active:
            if r.mask != 0:
                rec = denoise_step(self.model, r, self.L, self.tau, self.suffix_mode, keep_logits,
                                   steps_per_block=self.steps_per_block)
                self.total_committed += int(rec.committed.sum())
                recs.append(rec)
        self.total_steps += 1
        return recs

    def block_done(self) -> bool:
        return all(r.mask == 0 for r in self.sched.active)

    def run(self, max_cycles: int = 1 << 30) -> int:
        """Algorithm 1 until P and A are empty; returns the number of block-cycles.  With async_advance a "cycle"
        ends only when the active set has run empty (normally once, at the end of the stream)."""
        cycles = 0
        while cycles < max_cycles:
            _, _, n = self.evict_refill()
            if n == 0:
                break
            while not self.block_done():
                self.denoise_step()
                if self.async_advance:
                    self.step_boundary()
            cycles += 1
        return cycles

    def tokens(self, req_id: int) -> np.ndarray:
        return self.by_id[req_id].tokens
