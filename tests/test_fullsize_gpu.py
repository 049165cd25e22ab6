"""Parity at the benchmark's shapes (needs a B200 and ~60 GB of host memory).

* shallow replicas: the Dream-7B- and LLaDA-8B-shaped models cut to 2 layers (every other dimension, the
  vocabulary included, as in the benchmark), a few requests, full lockstep;
* full depth: the benchmark workload itself (16 requests, 28 layers) runs on the engine in the launch
  configuration bench.py times, while the oracle follows ONE sampled request through its block-cycle
  (requests never interact, so the oracle can compute that request alone); every integer check still covers
  the whole batch.
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


def _shallow(B, shape, ps, gs, alphas, starts, seed):
    from lockstep import Lockstep, lazy_oracle_model
    wl = bs_inputs.custom_workload(shape, ps, gs, alphas, starts, seed=seed, tau=0.9, max_batch=len(ps))
    w = bs_inputs.make_weights(shape, 4242, device="cuda")
    ls = Lockstep(wl, w, None, model=lazy_oracle_model(shape, w))
    ls.admit(wl.requests)
    ls.run()
    print("free oracle run:", ls.check_free_run())
    ls.assert_caps()
    assert ls.eng.stats().committed == wl.committed_target()
    return ls


def test_dream_shape_two_layers_full_lockstep(B):
    ls = _shallow(B, bs_inputs.DREAM_7B.with_layers(2), [150, 97, 64], [64, 64, 32], [3.0, 9.0, 30.0], [0, 1, 0], 11)
    print("dream-2L:", ls.summary())
    assert ls.max_logit_err < 2e-2


def test_llada_shape_two_layers_full_lockstep(B):
    ls = _shallow(B, bs_inputs.LLADA_8B.with_layers(2), [120, 40], [64, 40], [4.0, 25.0], [0, 0], 12)
    print("llada-2L:", ls.summary())
    assert ls.max_logit_err < 2e-2


def test_benchmark_workload_full_depth_sampled_request(B):
    from lockstep import Lockstep, lazy_oracle_model
    wl = bs_inputs.workload(2)
    w = bs_inputs.make_weights(wl.shape, wl.weight_seed, device="cuda")
    sample = min(wl.requests, key=lambda r: r.p + r.g)          # the shortest row keeps the oracle affordable
    ls = Lockstep(wl, w, None, track=[sample.req_id], model=lazy_oracle_model(wl.shape, w))
    ls.admit(wl.requests)
    ls.evict_refill()
    steps = 0
    while True:
        ls.step()
        steps += 1
        done = ls.eng.block_done()
        tracked_done = ls.ora.by_id[sample.req_id].mask == 0
        if done or (tracked_done and steps >= 3):
            break
    from lockstep import logit_tol
    print(f"cfg2 full depth, request {sample.req_id} (p={sample.p}, alpha={sample.alpha:.2f}): {ls.summary()} "
          f"(depth-28 tolerance {logit_tol(28):.3f})")
    assert ls.rows_checked > 0 and ls.max_logit_err < logit_tol(wl.shape.n_layers)
    # 28 layers of bf16 rounding put the measured logit deviation D at a few percent of max|z|: the class that D alone
    # explains is the largest here; it is capped on its own, beside the two classes the contract allows
    ls.assert_caps(noise_cap=0.10)


def test_llada_stream_full_depth_first_cycle_sampled_request(B):
    """Workload 3 (LLaDA-8B-shaped stream of 256 under a budget of 16384) at full depth: the first fill admits the
    shortest prompts up to the budget; the whole first block-cycle runs in the benchmark's launch configuration and
    the oracle follows one admitted request."""
    from lockstep import Lockstep, lazy_oracle_model, logit_tol
    wl = bs_inputs.workload(3)
    w = bs_inputs.make_weights(wl.shape, wl.weight_seed, device="cuda")
    first = min(wl.requests, key=lambda r: (r.p, r.req_id))     # head of the sorted queue: admitted for sure
    ls = Lockstep(wl, w, None, track=[first.req_id], kv_capacity=98304, model=lazy_oracle_model(wl.shape, w))
    ls.admit(wl.requests)
    _, admitted, n = ls.evict_refill()
    assert first.req_id in admitted and n > 50
    steps = 0
    while True:
        ls.step()
        steps += 1
        if ls.eng.block_done() or (ls.ora.by_id[first.req_id].mask == 0 and steps >= 3) or steps >= 8:
            break
    print(f"cfg3 full depth, {n} rows active, request {first.req_id} (p={first.p}, alpha={first.alpha:.2f}): "
          f"{ls.summary()}")
    assert ls.rows_checked > 0 and ls.max_logit_err < logit_tol(wl.shape.n_layers)
    ls.assert_caps(noise_cap=0.10)


@pytest.mark.parametrize("shape_name", ["dream", "llada"])
def test_repeated_runs_are_bit_identical_at_benchmark_width(B, shape_name):
    """Sixteen requests on a 4-layer replica of the benchmark shapes, served twice from scratch: every kernel sums in
    a fixed order and every hand-off between roles is fenced, so the committed tokens, the step count and the packed
    token count repeat exactly (a race in a pipeline shows up here as a difference or as BS_E_TIMEOUT)."""
    shape = (bs_inputs.DREAM_7B if shape_name == "dream" else bs_inputs.LLADA_8B).with_layers(4)
    rng = np.random.default_rng(5)
    n = 16
    ps = rng.integers(40, 700, size=n)
    gs = rng.choice([64, 96], size=n)
    al = rng.choice([2.0, 8.0, 30.0], size=n)
    wl = bs_inputs.custom_workload(shape, ps, gs, al, seed=21, tau=0.9, max_batch=n)
    w = bs_inputs.make_weights(shape, 99, device="cuda")
    runs = []
    for _ in range(2):
        eng = B.engine_for_workload(wl, w)
        for r in wl.requests:
            eng.admit(r.req_id, r.prompt, r.g, r.alpha)
        eng.run()
        st = eng.stats()
        assert st.committed == wl.committed_target()
        runs.append(([eng.read_tokens(r.req_id)[0] for r in wl.requests], st.steps, st.packed_tokens))
        eng.close()
    assert runs[0][1:] == runs[1][1:]
    for a, b in zip(runs[0][0], runs[1][0]):
        assert (a == b).all()
