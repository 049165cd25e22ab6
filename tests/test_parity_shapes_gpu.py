"""Parity at the shapes the long-context and straggler workloads bring, in later block cycles, and over whole
request streams (needs a B200; the full-depth cases also ~60 GB of host memory).

* rows of 1.5-2.5 k keys with 512 generated tokens on a two-layer replica of the Dream-7B shape: the tensor-core
  attention walks 30-40 key tiles per row, block steps run against 2.5 k-key rows;
* one refresh step with more than 16384 packed tokens (the MLP runs in token chunks), the tracked row straddling
  the chunk boundary;
* the benchmark workload and the LLaDA-shaped stream at full depth: integer lockstep from the start, and at later
  block boundaries - after evictions, compaction and (for the stream) a refill - a snapshot is taken and the oracle
  follows one sampled request through the cycle that starts there;
* model-free replay of the whole request stream of each of the five workloads on a one-layer toy model with the
  workload's own geometry: admissions, evictions, row order, KV slabs and every index array of every step, with
  rows that finish early and partial mask words.
"""
import numpy as np
import pytest
import torch

import bs_inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2607_08930_b200 import build
    build.build()
    from paper_2607_08930_b200 import binding
    return binding


def _cycle(ls, max_steps=1 << 30, until=None):
    """Runs one block cycle (or its first max_steps steps) in lockstep; returns the number of steps."""
    steps = 0
    while True:
        ls.step()
        steps += 1
        done = ls.eng.block_done()
        assert done == ls.ora.block_done()
        if done or steps >= max_steps or (until is not None and until(steps)):
            return steps


def test_long_context_rows_two_layers_two_cycles(B):
    """Workload 4's geometry (prompts of 1-2 k tokens, g = 512, tau = 0.95, mixed alpha) on a two-layer Dream-shaped
    replica, three requests in full lockstep for two block cycles."""
    from lockstep import Lockstep, lazy_oracle_model
    shape = bs_inputs.DREAM_7B.with_layers(2)
    wl = bs_inputs.custom_workload(shape, [1024, 1531, 2048], [512, 512, 512], [2.5, 9.0, 30.0], seed=41, tau=0.95,
                                   token_budget=65536, max_batch=3)
    w = bs_inputs.make_weights(shape, 4242, device="cuda")
    ls = Lockstep(wl, w, None, model=lazy_oracle_model(shape, w))
    ls.admit(wl.requests)
    for _ in range(2):
        _, _, n = ls.evict_refill()
        assert n == 3
        _cycle(ls)
    print("long-context 2L:", ls.summary())
    ls.assert_caps()
    assert ls.stats["bf16"].max_logit_err < 2e-2


def test_refresh_step_across_the_mlp_token_chunk(B):
    """Eight rows of 2304 tokens: the refresh step packs 18432 tokens, more than one MLP chunk of 16384; the tracked
    row (the last one) holds packed tokens 16128 .. 18431 and so lies on both sides of the chunk boundary."""
    from lockstep import Lockstep, lazy_oracle_model
    shape = bs_inputs.DREAM_7B.with_layers(2)
    n = 8
    wl = bs_inputs.custom_workload(shape, [1792] * n, [512] * n, [6.0] * n, seed=43, tau=0.95, token_budget=65536,
                                   max_batch=n)
    w = bs_inputs.make_weights(shape, 4242, device="cuda")
    ls = Lockstep(wl, w, None, track=[n - 1], model=lazy_oracle_model(shape, w))
    ls.admit(wl.requests)
    _, _, active = ls.evict_refill()
    assert active == n
    hdr = ls.eng.debug(B.DBG_HEADER)
    assert hdr[1] == n * 2304 > 16384
    assert ls.eng.debug(B.DBG_CU_Q).tolist()[n - 1] < 16384 < ls.eng.debug(B.DBG_CU_Q).tolist()[n]
    _cycle(ls, max_steps=3)
    print("MLP chunk boundary:", ls.summary())
    assert ls.rows_checked >= 32 and ls.stats["bf16"].max_logit_err < 2e-2


def _sampled_cycles(B, wl, kv_capacity, boundaries, pick, max_steps):
    """Integer lockstep over the whole batch from the start; at each cycle index in `boundaries` a snapshot is taken
    at the block boundary, the oracle attaches to the request `pick(ls)` names (taking its token row from the engine,
    which is what the snapshot holds) and follows it through that cycle; the engine is then rewound to the snapshot
    and must reproduce the cycle bit for bit before the run goes on untracked."""
    from lockstep import Lockstep, lazy_oracle_model
    w = bs_inputs.make_weights(wl.shape, wl.weight_seed, device="cuda")
    ls = Lockstep(wl, w, None, track=set(), kv_capacity=kv_capacity, model=lazy_oracle_model(wl.shape, w))
    ls.admit(wl.requests)
    cycle, seen = 0, []
    while cycle <= max(boundaries):
        snap = ls.eng.snapshot().copy() if cycle in boundaries else None      # between cycles: tokens + scheduler state
        ev, ad, n = ls.evict_refill()
        assert n > 0
        if cycle in boundaries:
            rid = pick(ls)
            ls.attach([rid])
            r = ls.ora.by_id[rid]
            rows0 = ls.rows_checked
            steps = _cycle(ls, max_steps=max_steps, until=lambda k: r.mask == 0 and k >= 3)
            seen.append(dict(cycle=cycle, request=rid, p=r.p, block=r.b, alpha=r.alpha, active_rows=n, steps=steps,
                             decisions=ls.rows_checked - rows0, evicted_so_far=len(ls.ora.sched.finished)))
            # finish the cycle untracked, remember the tokens, rewind, replay: a snapshot continues bit-identically
            ls.attach([])
            while not ls.eng.block_done():
                ls.step()
            assert ls.ora.block_done()
            want = {q.req_id: ls.eng.read_tokens(q.req_id)[0] for q in ls.ora.sched.active}
            ls.eng.restore(snap)
            assert ls.eng.evict_refill() == (len(ev), len(ad), n)
            while True:
                ls.eng.denoise_step()
                if ls.eng.block_done():
                    break
            for q in ls.ora.sched.active:
                assert (ls.eng.read_tokens(q.req_id)[0] == want[q.req_id]).all()
        else:
            _cycle(ls)
        cycle += 1
    return ls, seen


def test_benchmark_workload_full_depth_later_cycles_from_snapshots(B):
    """Workload 2 at full depth (28 layers, the launch configuration bench.py times).  Requests start at block
    indices 0..7, so rows leave from the first boundary on; the sampled cycles start after evictions and compaction."""
    wl = bs_inputs.workload(2)
    def pick(ls):       # the shortest active row keeps the oracle affordable
        return min(ls.ora.sched.active, key=lambda r: r.p + r.g).req_id
    ls, seen = _sampled_cycles(B, wl, None, boundaries=(1, 3), pick=pick, max_steps=12)
    print("cfg2 full depth, later cycles:", seen, ls.summary())
    assert all(s["evicted_so_far"] > 0 for s in seen) and ls.rows_checked > 0
    ls.assert_caps(noise_cap=0.10)


def test_llada_stream_full_depth_cycle_after_the_first_refill(B):
    """Workload 3 at full depth under its budget: g = 256 means the first rows leave after eight cycles and the queue
    refills the batch; the sampled request is one admitted by that refill, followed through its first cycle."""
    wl = bs_inputs.workload(3)
    state = {}
    def pick(ls):
        tr = ls.ora.sched.trace[-1]
        assert tr.evicted and tr.admitted, "this boundary was meant to evict and refill"
        state["admitted"] = len(tr.admitted)
        return min((ls.ora.by_id[i] for i in tr.admitted), key=lambda r: r.p).req_id
    ls, seen = _sampled_cycles(B, wl, 98304, boundaries=(8,), pick=pick, max_steps=5)
    print("cfg3 full depth, cycle after the first refill:", seen, state, ls.summary())
    assert ls.rows_checked > 0
    ls.assert_caps(noise_cap=0.10)


def test_long_context_stream_full_depth_first_cycle(B):
    """Workload 4 at full depth (28 layers, rows of 1.5-2.5 k tokens under the 65536-token budget, tau = 0.95): the
    whole batch runs in integer lockstep, the oracle follows the shortest admitted row through its refresh step and
    the first block steps of cycle 0."""
    wl = bs_inputs.workload(4)
    def pick(ls):
        return min(ls.ora.sched.active, key=lambda r: r.p + r.g).req_id
    ls, seen = _sampled_cycles(B, wl, 98304, boundaries=(0,), pick=pick, max_steps=4)
    print("cfg4 full depth, cycle 0:", seen, ls.summary())
    assert seen[0]["active_rows"] > 16 and seen[0]["p"] > 1000 and ls.rows_checked > 0
    ls.assert_caps(noise_cap=0.10)


TOY = bs_inputs.ModelShape("toy", 1, 64, 1, 1, 64, 64, 64, init_std=0.1)


@pytest.mark.parametrize("cfg,async_advance", [(1, False), (2, False), (3, False), (4, False), (5, False),
                                               (1, True), (3, True), (5, True)])
def test_whole_stream_model_free_replay(B, cfg, async_advance):
    """The schedule and every index array of a stream depend on the model only through which positions each step
    commits.  Here each workload's whole request stream (same prompt lengths, generation lengths, start blocks,
    alphas, budget and batch cap; token ids redrawn for the toy vocabulary) is served by the engine on a one-layer toy
    model at tau = 0.9, so rows take between one and 32 steps per block; the oracle's scheduler and index builder
    follow with the engine's mask words and must reproduce every admission, eviction, row order, KV slab, header
    count and index array of every step, bit for bit.  With async_advance the boundary runs after every step (rows
    in their refresh step and rows in cached block steps share a step; admissions at any step)."""
    from lockstep import Lockstep
    src = bs_inputs.workload(cfg)
    rng = np.random.default_rng(100 + cfg)
    reqs = []
    for r in src.requests:
        pre = rng.integers(0, 63, size=r.start_block * 32).astype(np.int32) if r.start_block else None
        reqs.append(bs_inputs.Request(r.req_id, rng.integers(0, 63, size=r.p).astype(np.int32), r.g,
                                      float(min(max(r.alpha, 0.5), 40.0)), r.start_block, pre, r.phase))
    wl = bs_inputs.Workload(f"cfg{cfg}-geometry", TOY, 32, 0.9, src.token_budget, src.max_batch, reqs)
    w = bs_inputs.make_weights(TOY, 7, device="cuda")
    cap = None if src.token_budget <= 0 else 98304
    from oracle import blockserve_oracle as O
    model = O.model_from_weights(TOY, bs_inputs.weights_to_numpy_f32({k: ([t.cpu() for t in v] if isinstance(v, list)
                                                                          else v.cpu()) for k, v in w.items()}))
    ls = Lockstep(wl, w, None, track=set(), kv_capacity=cap, model=model, modes=("bf16",), async_advance=async_advance)
    ls.admit([r for r in reqs if r.phase == 0])
    late = [r for r in reqs if r.phase == 1]
    cycles = ls.run(phase1=late or None)
    st = ls.eng.stats()
    assert st.committed == wl.committed_target()
    assert len(ls.ora.sched.finished) == len(reqs)
    print(f"cfg{cfg} geometry, async_advance={async_advance}: {len(reqs)} requests, {cycles} cycles, {st.steps} steps, "
          f"{st.packed_tokens} packed tokens, rows working per step {st.row_steps / max(st.active_row_steps, 1):.3f}")
    if async_advance:
        assert st.row_steps == st.active_row_steps
    else:
        assert cycles == st.cycles == len([t for t in ls.ora.sched.trace if t.n_active])
        assert st.sum_active == sum(t.n_active for t in ls.ora.sched.trace)
        assert 1.0 < st.steps / max(cycles, 1) <= 32.0


def test_async_advance_llada_shape_two_layers(B):
    """Per-row advance at the LLaDA-8B width (two layers, full vocabulary): steps that mix whole-row refreshes with
    cached 32-token block steps go through the tensor-core attention and the refresh-path projections together."""
    from lockstep import Lockstep, lazy_oracle_model
    shape = bs_inputs.LLADA_8B.with_layers(2)
    wl = bs_inputs.custom_workload(shape, [120, 40, 77, 200], [64, 40, 96, 64], [4.0, 25.0, 9.0, 30.0], [0, 0, 1, 0],
                                   seed=12, tau=0.9, max_batch=3, token_budget=900)
    w = bs_inputs.make_weights(shape, 4242, device="cuda")
    ls = Lockstep(wl, w, None, model=lazy_oracle_model(shape, w), async_advance=True)
    ls.admit(wl.requests)
    ls.run()
    st = ls.eng.stats()
    assert st.committed == wl.committed_target() and st.row_steps == st.active_row_steps
    print("llada-2L async:", st.steps, "steps;", ls.summary())
    ls.assert_caps()
    assert ls.stats["bf16"].max_logit_err < 2e-2
