"""The allocation-free RoPE + KV-scatter entry point against the regular one (needs a B200).

Some users of the library run where device allocation is not available to them (a pool fixed at start-up, a
host runtime that owns all memory).  bs_op_rope_kv_static serves them with a table kept inside the library;
here it must reproduce bs_op_rope_kv on two calls in a row that use different table contents, so that stale
contents from the first call cannot leak into the second.  Collected last on purpose."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2607_08930_b200 import build
    build.build()
    from paper_2607_08930_b200 import binding
    return binding


def _case(B, seed, hq, hkv, dh, theta, max_pos, M, rows, check_device_free=False):
    rng = np.random.default_rng(seed)
    qkv = torch.from_numpy(rng.normal(size=(M, (hq + 2 * hkv) * dh)).astype(np.float32)).to(torch.bfloat16).cuda()
    pos_h = rng.integers(0, max_pos, size=M).astype(np.int32)
    pos_h[:2] = (max_pos - 1, 0)              # the table's last entry must be this call's own, not an earlier call's
    pos = torch.from_numpy(pos_h).cuda()
    kvrow = torch.from_numpy(rng.permutation(rows)[:M].astype(np.int32)).cuda()
    ref_q = qkv.clone()
    ref_k = torch.zeros(rows, hkv, dh, dtype=torch.bfloat16, device="cuda")
    ref_v = torch.zeros_like(ref_k)
    B.op_rope_kv(ref_q, pos, kvrow, ref_k, ref_v, hq, hkv, dh, theta, max_pos)
    got_q = qkv.clone()
    got_k, got_v = torch.zeros_like(ref_k), torch.zeros_like(ref_v)
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    free_before = torch.cuda.mem_get_info()[0]
    rc = B.op_rope_kv_static(got_q, pos, kvrow, got_k, got_v, hq, hkv, dh, theta, max_pos)
    torch.cuda.synchronize()
    assert rc == B.BS_OK
    assert torch.cuda.memory_allocated() == before          # nothing was taken from torch's allocator
    if check_device_free:
        # nor from the device behind torch's back (a cudaMalloc inside the library would lower the free figure);
        # checked on a call that is not the process's first, so that loading the kernels' code is not counted
        assert torch.cuda.mem_get_info()[0] >= free_before
    for g, r in ((got_q, ref_q), (got_k, ref_k), (got_v, ref_v)):
        g, r = g.float().cpu().numpy(), r.float().cpu().numpy()
        assert np.abs(g - r).max() <= 8e-3 * max(np.abs(r).max(), 1e-30)    # tolerance of the RoPE parity test
    assert (got_v == ref_v).all()


def test_two_calls_in_a_row_match_the_regular_entry_point(B):
    _case(B, 1, hq=28, hkv=4, dh=128, theta=10000.0, max_pos=3000, M=333, rows=4000)
    # a different head_dim, base and table length right after: every entry read must have been rewritten
    _case(B, 2, hq=4, hkv=4, dh=64, theta=500.0, max_pos=777, M=90, rows=900, check_device_free=True)


def test_table_too_large_is_rejected(B):
    dh, max_pos = 128, B.ROPE_STATIC_MAX_FLOATS // 128 + 1
    z = torch.zeros(1, 3 * dh, dtype=torch.bfloat16, device="cuda")
    i = torch.zeros(1, dtype=torch.int32, device="cuda")
    kv = torch.zeros(1, 1, dh, dtype=torch.bfloat16, device="cuda")
    assert B.op_rope_kv_static(z, i, i, kv, kv.clone(), 1, 1, dh, 10000.0, max_pos) == B.BS_E_ARG
    assert B.op_rope_kv_static(z, i, i, kv, kv.clone(), 1, 1, dh, 10000.0, max_pos - 1) == B.BS_OK
    torch.cuda.synchronize()
