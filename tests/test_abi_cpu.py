"""Host-side checks of the C ABI that need no GPU: the library builds, loads and exports every
symbol the header declares; size queries and argument validation work without a device."""
import ctypes as C
import os
import re

import pytest

import bs_inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2607_08930_b200 import build
    build.build()
    from paper_2607_08930_b200 import binding
    return binding


def test_every_declared_symbol_is_exported(B):
    hdr = open(os.path.join(ROOT, "include", "blockserve.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(bs_[a-z_0-9]+)\s*\(", hdr))
    assert {"bs_init_model", "bs_admit", "bs_denoise_step", "bs_block_done", "bs_evict_refill",
            "bs_read_tokens"} <= declared
    lib = B.lib()
    for name in declared:
        assert hasattr(lib, name), f"{name} declared but not exported"
    assert declared == set(B.EXPORTS)


def test_query_sizes_and_validation(B):
    wl = bs_inputs.workload(1)
    cfg = B.make_config(wl.shape, 32, 0.9, 0, 4, 8, wl.max_row_tokens, 4 * wl.max_row_tokens)
    sz = B.query_sizes(cfg)
    kv = wl.shape.n_layers * 2 * 4 * wl.max_row_tokens * wl.shape.n_kv_heads * wl.shape.head_dim * 2
    assert sz.kv_bytes >= kv and sz.kv_bytes < kv + 256
    assert sz.workspace_bytes > 0 and sz.state_bytes > 8 * wl.max_row_tokens * 4
    # the policy switches do not change any buffer size
    cfg_p = B.make_config(wl.shape, 32, 0.9, 0, 4, 8, wl.max_row_tokens, 4 * wl.max_row_tokens, steps_per_block=8,
                          eos_id=5, static_groups=True)
    sz_p = B.query_sizes(cfg_p)
    assert (sz_p.kv_bytes, sz_p.workspace_bytes, sz_p.state_bytes) == (sz.kv_bytes, sz.workspace_bytes, sz.state_bytes)
    for field, bad in (("head_dim", 48), ("block_len", 65), ("max_batch", 5000), ("vocab", 1023),
                       ("refresh_policy", 2), ("async_advance", 2), ("keep_logits", 3),
                       ("kv_capacity_tokens", 3), ("n_q_heads", 3), ("steps_per_block", 33), ("steps_per_block", -1),
                       ("eos_id", wl.shape.mask_id), ("eos_id", wl.shape.vocab)):
        cfg2 = B.make_config(wl.shape, 32, 0.9, 0, 4, 8, wl.max_row_tokens, 4 * wl.max_row_tokens)
        setattr(cfg2, field, bad)
        if field == "n_q_heads":
            cfg2.n_kv_heads = 2
        with pytest.raises(B.BlockServeError) as ei:
            B.query_sizes(cfg2)
        assert ei.value.code == B.BS_E_ARG


def test_init_fails_loudly_without_a_device(B):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    wl = bs_inputs.workload(1)
    cfg = B.make_config(wl.shape, 32, 0.9, 0, 4, 8, wl.max_row_tokens, 4 * wl.max_row_tokens)
    with pytest.raises(RuntimeError):
        B.Engine(cfg, {})
    # and the C entry point itself refuses (no CPU path behind the ABI)
    n = wl.shape.n_layers
    arr = (C.c_void_p * n)(*([256] * n))
    p = C.cast(arr, C.POINTER(C.c_void_p))
    w = B.BsWeights(256, 256, 256, p, p, p, p, p, p, p)
    h = C.c_void_p()
    rc = B.lib().bs_init_model(C.byref(cfg), C.byref(w), 256, 256, 256, None, C.byref(h))
    assert rc == B.BS_E_CUDA and b"no CUDA device" in B.lib().bs_last_error(None)


def test_bounds_checked_build_exports_the_same_interface():
    """The debugging build compiles from the same sources and must export every declared symbol too."""
    import ctypes
    from paper_2607_08930_b200 import build, binding
    lib = ctypes.CDLL(build.build(debug=True))
    for name in binding.EXPORTS:
        assert hasattr(lib, name), name
    lib.bs_build_flags.argtypes = []
    assert lib.bs_build_flags() == binding.BUILD_BOUNDS_CHECK
    assert binding.lib().bs_build_flags() == (binding.BUILD_BOUNDS_CHECK if binding.DEBUG_LIB else 0)
