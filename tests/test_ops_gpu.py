"""Per-kernel parity against the CPU oracle's functions, through the C ABI (needs a B200)."""
import numpy as np
import pytest
import torch

from oracle import blockserve_oracle as O

pytestmark = pytest.mark.gpu
F32 = np.float32


@pytest.fixture(scope="module")
def B():
    from paper_2607_08930_b200 import build
    build.build()
    from paper_2607_08930_b200 import binding
    return binding


def bf16_round(a):
    return torch.from_numpy(np.asarray(a, dtype=F32)).to(torch.bfloat16)


def rel_err(got, ref):
    return float(np.abs(got - ref).max() / max(np.abs(ref).max(), 1e-30))


GEMM_SHAPES = [  # M, N, K: several tiles, ragged tails in every dimension, one case smaller than a tile
    (1, 128, 64), (33, 200, 72), (128, 256, 128), (130, 1000, 384), (257, 130, 1000), (300, 2000, 256),
    (517, 704, 256), (64, 4608, 512), (1000, 512, 2048), (459, 768, 256), (459, 256, 704), (48, 384, 128),
    (200, 640, 320),
    # more 256-row weight tiles than CTA pairs with a ragged last round: the SwiGLU plan narrows its token tiles
    (1760, 12288, 128),
    # activations beyond the L2 budget: token tiles taken in groups (36 token tiles, groups of 8 or 16, ragged last group)
    (9000, 512, 3584)]


@pytest.mark.parametrize("M,N,K", GEMM_SHAPES)
@pytest.mark.parametrize("mode", [0, 1, 2, 3])
def test_gemm_modes(B, M, N, K, mode):
    rng = np.random.default_rng(M * 7 + N * 3 + K + mode)
    A = bf16_round(rng.normal(size=(M, K)))
    W = bf16_round(rng.normal(size=(N, K)) * 0.1)
    W2 = bf16_round(rng.normal(size=(N, K)) * 0.1)
    a, w, w2 = A.float().numpy(), W.float().numpy(), W2.float().numpy()
    ref = a.astype(np.float64) @ w.T.astype(np.float64)
    Ad, Wd, W2d = A.cuda(), W.cuda(), W2.cuda()
    if mode == 0:
        got = B.op_gemm(Ad, Wd, 0).float().cpu().numpy()
        tol = 6e-3
    elif mode == 1:
        c0 = rng.normal(size=(M, N)).astype(F32)
        Cd = torch.from_numpy(c0).cuda()
        B.op_gemm(Ad, Wd, 1, C_out=Cd)
        got, ref, tol = Cd.cpu().numpy(), ref + c0, 1e-4
    elif mode == 2:
        sc = rng.uniform(0.5, 30.0, size=M).astype(F32)
        got = B.op_gemm(Ad, Wd, 2, row_scale=torch.from_numpy(sc).cuda()).cpu().numpy()
        ref, tol = ref * sc[:, None], 1e-4
    else:
        up = a.astype(np.float64) @ w2.T.astype(np.float64)
        ref = O.silu(ref.astype(F32)).astype(np.float64) * up
        got = B.op_gemm(Ad, Wd, 3, W2=W2d).float().cpu().numpy()
        tol = 8e-3
    assert got.shape == ref.shape
    assert rel_err(got, ref) < tol
    # element-wise too, so that a wrong tile in a corner cannot hide behind the global maximum
    assert np.abs(got - ref).max() <= tol * (np.abs(ref) + np.abs(ref).max() * 0.05).max()


@pytest.mark.parametrize("M,N,K,mode", [(32, 512, 4096, 0), (64, 384, 2048, 1), (100, 256, 8192, 3), (96, 640, 1024, 2),
                                          (256, 1152, 3584, 1), (40, 3584, 18944, 1),
                                          # CTA-pair kernel with a k split (few 256-row tiles, enough tokens)
                                          (400, 512, 4096, 0), (512, 256, 2048, 1), (800, 256, 8192, 1),
                                          (400, 520, 4096, 2)])
def test_gemm_k_split(B, M, N, K, mode):
    """Few output tiles and a long K: the launch splits K across CTAs and sums the partials in a fixed order."""
    rng = np.random.default_rng(M + N + K)
    A = bf16_round(rng.normal(size=(M, K)))
    W = bf16_round(rng.normal(size=(N, K)) * 0.05)
    W2 = bf16_round(rng.normal(size=(N, K)) * 0.05)
    a, w, w2 = A.double().numpy(), W.double().numpy(), W2.double().numpy()
    scratch = torch.empty(16 << 20, dtype=torch.float32, device="cuda")
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    ref = a @ w.T
    kw = dict(scratch=scratch, error_flag=flag)
    if mode == 0:
        got, tol = B.op_gemm(A.cuda(), W.cuda(), 0, **kw).float().cpu().numpy(), 6e-3
    elif mode == 1:
        c0 = rng.normal(size=(M, N)).astype(F32)
        Cd = torch.from_numpy(c0).cuda()
        B.op_gemm(A.cuda(), W.cuda(), 1, C_out=Cd, **kw)
        got, ref, tol = Cd.cpu().numpy(), ref + c0, 1e-4
    elif mode == 2:
        sc = rng.uniform(0.5, 30.0, size=M).astype(F32)
        got = B.op_gemm(A.cuda(), W.cuda(), 2, row_scale=torch.from_numpy(sc).cuda(), **kw).cpu().numpy()
        ref, tol = ref * sc[:, None], 1e-4
    else:
        ref = O.silu(ref.astype(F32)).astype(np.float64) * (a @ w2.T)
        got, tol = B.op_gemm(A.cuda(), W.cuda(), 3, W2=W2.cuda(), **kw).float().cpu().numpy(), 8e-3
    assert int(flag.item()) == 0
    assert rel_err(got, ref) < tol
    # twice the same launch gives the same bits (fixed summation order)
    if mode == 0:
        again = B.op_gemm(A.cuda(), W.cuda(), 0, **kw).float().cpu().numpy()
        assert (again == got).all()


@pytest.mark.parametrize("M,N,K", [(128, 3584, 3584), (200, 4608, 3584), (256, 3584, 2048), (333, 3584, 3584),
                                   (500, 3584, 1024), (512, 3584, 18944), (640, 1024, 4096), (1000, 512, 2048),
                                   (144, 3592, 1024)])
@pytest.mark.parametrize("mode", [0, 1])
def test_gemm_k_split_inside_clusters(B, M, N, K, mode):
    """Direct projections with few output tiles: the pairs of a tile share a cluster and add their partial accumulators
    over distributed shared memory (ragged token tiles, a ragged weight tile, both cluster sizes, both epilogues)."""
    assert B.op_gemm_cluster_splits(M, N, K, mode) in (2, 4), "the shape is meant to take the cluster plan"
    rng = np.random.default_rng(M * 3 + N + K + mode)
    A = bf16_round(rng.normal(size=(M, K)))
    W = bf16_round(rng.normal(size=(N, K)) * 0.05)
    ref = A.double().numpy() @ W.double().numpy().T
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    if mode == 0:
        run = lambda: B.op_gemm(A.cuda(), W.cuda(), 0, error_flag=flag).float().cpu().numpy()
        tol = 6e-3
    else:
        c0 = rng.normal(size=(M, N)).astype(F32)
        ref = ref + c0

        def run():
            Cd = torch.from_numpy(c0).cuda()
            B.op_gemm(A.cuda(), W.cuda(), 1, C_out=Cd, error_flag=flag)
            return Cd.cpu().numpy()
        tol = 1e-4
    got = run()
    assert int(flag.item()) == 0
    assert rel_err(got, ref) < tol
    assert np.abs(got - ref).max() <= tol * (np.abs(ref) + np.abs(ref).max() * 0.05).max()
    assert (run() == got).all()          # split order is fixed: the same bits every time


@pytest.mark.parametrize("M,N,K", [(2200, 1536, 8192), (2048, 1280, 8200), (4100, 1024, 8192),
                                   (5000, 2048, 8192)])      # the last: more items than CTA pairs
@pytest.mark.parametrize("mode", [0, 1, 2])
def test_gemm_wide_pair_items_with_a_long_k(B, M, N, K, mode):
    """Many tokens and a long K (the down projection of a refresh step): work items of 512 weight rows whose two
    accumulators share every token tile, token tiles narrowed to fill the last round; ragged in every dimension
    (a last item with 256 of its 512 weight rows, K beyond the last full k block, a partial token tile)."""
    rng = np.random.default_rng(M + 3 * N + K + mode)
    A = bf16_round(rng.normal(size=(M, K)))
    W = bf16_round(rng.normal(size=(N, K)) * 0.05)
    ref = A.double().numpy() @ W.double().numpy().T
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    if mode == 0:
        got, tol = B.op_gemm(A.cuda(), W.cuda(), 0, error_flag=flag).float().cpu().numpy(), 6e-3
    elif mode == 1:
        c0 = rng.normal(size=(M, N)).astype(F32)
        Cd = torch.from_numpy(c0).cuda()
        B.op_gemm(A.cuda(), W.cuda(), 1, C_out=Cd, error_flag=flag)
        got, ref, tol = Cd.cpu().numpy(), ref + c0, 1e-4
    else:
        sc = rng.uniform(0.5, 30.0, size=M).astype(F32)
        got = B.op_gemm(A.cuda(), W.cuda(), 2, row_scale=torch.from_numpy(sc).cuda(), error_flag=flag).cpu().numpy()
        ref, tol = ref * sc[:, None], 1e-4
    assert int(flag.item()) == 0
    assert rel_err(got, ref) < tol
    assert np.abs(got - ref).max() <= tol * (np.abs(ref) + np.abs(ref).max() * 0.05).max()


def test_gemm_cluster_plan_leaves_other_shapes_alone(B):
    for M, N, K, mode in [(64, 3584, 3584, 0), (2048, 3584, 3584, 1), (256, 3584, 3584, 3), (256, 3584, 3584, 2),
                          (256, 128, 3584, 0), (256, 3584, 256, 0)]:
        assert B.op_gemm_cluster_splits(M, N, K, mode) == 0


def test_gemm_strided_rows_and_empty(B):
    rng = np.random.default_rng(5)
    big = bf16_round(rng.normal(size=(70, 512))).cuda()
    A = big[:, :256]                       # lda 512, K 256
    W = bf16_round(rng.normal(size=(192, 256)) * 0.1).cuda()
    got = B.op_gemm(A, W, 0).float().cpu().numpy()
    ref = A.float().cpu().numpy() @ W.float().cpu().numpy().T
    assert rel_err(got, ref) < 6e-3
    empty = B.op_gemm(big[:0, :256], W, 0)
    assert empty.shape == (0, 192)


@pytest.mark.parametrize("M,d", [(1, 256), (37, 384), (300, 3584)])
def test_rmsnorm(B, M, d):
    rng = np.random.default_rng(d)
    x = (rng.normal(size=(M, d)) * 3).astype(F32)
    w = bf16_round(1 + 0.1 * rng.normal(size=d))
    ref = O.rmsnorm(x, w.float().numpy(), 1e-6)
    got = B.op_rmsnorm(torch.from_numpy(x).cuda(), w.cuda(), 1e-6).float().cpu().numpy()
    assert np.abs(got - ref).max() <= 1e-2 * np.abs(ref).max() and rel_err(got, ref) < 5e-3
    idx = rng.permutation(M)[: max(1, M // 2)].astype(np.int32)
    got = B.op_rmsnorm(torch.from_numpy(x).cuda(), w.cuda(), 1e-6, idx=torch.from_numpy(idx).cuda()).float().cpu().numpy()
    assert rel_err(got, ref[idx]) < 5e-3


@pytest.mark.parametrize("hq,hkv,dh", [(4, 4, 64), (6, 2, 128), (28, 4, 128)])
def test_rope_and_kv_scatter(B, hq, hkv, dh):
    rng = np.random.default_rng(hq)
    M, rows, max_pos = 75, 400, 300
    qkv = bf16_round(rng.normal(size=(M, (hq + 2 * hkv) * dh)))
    pos = rng.integers(0, max_pos, size=M).astype(np.int32)
    kvrow = rng.permutation(rows)[:M].astype(np.int32)
    kc = torch.zeros(rows, hkv, dh, dtype=torch.bfloat16, device="cuda")
    vc = torch.zeros_like(kc)
    qd = qkv.cuda()
    B.op_rope_kv(qd, torch.from_numpy(pos).cuda(), torch.from_numpy(kvrow).cuda(), kc, vc, hq, hkv, dh, 10000.0, max_pos)
    x = qkv.float().numpy()
    q = x[:, :hq * dh].reshape(M, hq, dh)
    k = x[:, hq * dh:(hq + hkv) * dh].reshape(M, hkv, dh)
    v = x[:, (hq + hkv) * dh:].reshape(M, hkv, dh)
    cos, sin = O.rope_cos_sin(pos, dh, 10000.0)
    q_ref, k_ref = O.apply_rope(q, cos, sin), O.apply_rope(k, cos, sin)
    got_q = qd.float().cpu().numpy()[:, :hq * dh].reshape(M, hq, dh)
    assert np.abs(got_q - q_ref).max() < 3e-2 and rel_err(got_q, q_ref) < 8e-3
    kc_h, vc_h = kc.float().cpu().numpy(), vc.float().cpu().numpy()
    assert rel_err(kc_h[kvrow], k_ref) < 8e-3
    assert (vc_h[kvrow] == v).all()                       # v is copied bit for bit
    untouched = np.setdiff1d(np.arange(rows), kvrow)
    assert (kc_h[untouched] == 0).all() and (vc_h[untouched] == 0).all()   # only the query rows are written


ATTN_CASES = [
    # hq, hkv, dh, [(n_q, vis)] per row: block steps (n_q = 32 or a ragged tail), refresh rows (n_q = vis), empty rows
    (4, 4, 64, [(32, 159), (32, 41), (0, 50), (17, 64)]),
    (6, 2, 128, [(32, 200), (8, 8), (130, 130), (0, 9), (32, 65)]),
    (28, 4, 128, [(32, 300), (32, 96), (70, 70)]),
    (32, 32, 128, [(32, 129), (100, 100)]),
    # MHA rows longer than one Q tile (two Q tiles of 128 tokens per work item, several items per row)
    (8, 8, 128, [(300, 300), (32, 517), (129, 129)]),
    # four and eight query heads per kv head (32 and 16 tokens per Q tile)
    (8, 2, 128, [(70, 200), (32, 64), (33, 33)]),
    (16, 2, 128, [(40, 130), (32, 700)]),
    # long-context block steps (GQA 28 / 4): rows of 1-2.5 k keys, whose key tiles are cut into chunks over several
    # CTAs when scratch is given, with a ragged block, an empty row and rows shorter than one chunk beside them
    (28, 4, 128, [(32, 2304)] * 8),
    (28, 4, 128, [(32, 1100), (32, 2560), (17, 1300), (0, 64), (32, 40)]),
    # a refresh row beside cached block steps (steps of the per-row advance mix both)
    (28, 4, 128, [(700, 700), (32, 900), (32, 333)]),
]


@pytest.mark.parametrize("split_keys", [False, True])
@pytest.mark.parametrize("hq,hkv,dh,rows", ATTN_CASES)
def test_ragged_dual_cache_attention(B, hq, hkv, dh, rows, split_keys):
    rng = np.random.default_rng(hq * 100 + dh)
    cap = sum(v for _, v in rows) + 64
    kc = bf16_round(rng.normal(size=(cap, hkv, dh)))
    vc = bf16_round(rng.normal(size=(cap, hkv, dh)))
    M = sum(n for n, _ in rows)
    qkv = bf16_round(rng.normal(size=(M, (hq + 2 * hkv) * dh)) * 1.5)
    # slabs in shuffled physical order with gaps, so that kv_base matters
    order = rng.permutation(len(rows))
    kv_base = np.zeros(len(rows), np.int32)
    at = 7
    for i in order:
        kv_base[i] = at
        at += rows[i][1] + 3
    cu_q = np.zeros(len(rows) + 1, np.int32)
    cu_q[1:] = np.cumsum([n for n, _ in rows])
    vis = np.array([v for _, v in rows], np.int32)
    # with scratch, a launch with few work items splits each row's keys over several CTAs and merges the parts
    scratch = torch.empty(8 << 20, dtype=torch.float32, device="cuda") if split_keys else None
    out = B.op_attention(qkv.cuda(), kc.cuda(), vc.cuda(), torch.from_numpy(cu_q).cuda(),
                         torch.from_numpy(kv_base).cuda(), torch.from_numpy(vis).cuda(), hq, hkv, dh, scratch=scratch)
    got = out.float().cpu().numpy().reshape(M, hq, dh)
    q = qkv.float().numpy()[:, :hq * dh].reshape(M, hq, dh)
    K, V = kc.float().numpy(), vc.float().numpy()
    for i, (n, v) in enumerate(rows):
        if n == 0:
            continue
        ref = O.attention(q[cu_q[i]:cu_q[i + 1]], K[kv_base[i]:kv_base[i] + v], V[kv_base[i]:kv_base[i] + v])
        g = got[cu_q[i]:cu_q[i + 1]]
        assert np.abs(g - ref).max() < 2e-2, f"row {i}: {np.abs(g - ref).max()}"
        assert rel_err(g, ref) < 1e-2


@pytest.mark.parametrize("n,V", [(1, 1024), (37, 2000), (64, 152064), (5, 126464)])
def test_confidence_rows(B, n, V):
    rng = np.random.default_rng(V)
    z = (rng.normal(size=(n, V)) * rng.uniform(0.5, 6.0, size=(n, 1))).astype(F32)
    mask_id = V - 1
    z[0, mask_id] = 1e4                      # the mask id must never win
    if n > 2:
        z[1, :] = 0.25                       # all equal: tok 0, conf 1 / (V - 1)
        z[2, 100] = z[2, 7] = 50.0           # tie: lowest id
    tok_ref, conf_ref = O.confidence(z, mask_id)
    tok, conf = B.op_confidence(torch.from_numpy(z).cuda(), mask_id)
    tok, conf = tok.cpu().numpy(), conf.cpu().numpy()
    assert (tok == tok_ref).all()
    assert (np.abs(conf - conf_ref) / conf_ref).max() < 1e-4


@pytest.mark.parametrize("M,V,K", [(1, 1024, 64), (37, 2000, 72), (130, 1026, 128), (300, 5000, 128),
                                   (64, 152064, 256), (513, 4128, 512)])
def test_lm_head_fused_with_the_confidence_pass(B, M, V, K):
    """The LM-head GEMM reduces its own accumulators to (argmax, confidence) per row; the logits are stored here
    only so that the result can be checked exactly on them: token ids bit for bit (mask id never, lowest id on ties),
    confidences to 1e-4 against the oracle's formula, and both against the stand-alone confidence kernel."""
    rng = np.random.default_rng(M + V + K)
    hf = bf16_round(rng.normal(size=(M, K)))
    W = bf16_round(rng.normal(size=(V, K)) * 0.3)
    mask_id = V - 1
    W[mask_id] = W[5] * 4.0 + 1.0                 # the mask id would win many rows if it took part
    if V > 300:
        W[300] = W[17]                            # identical columns: ties must go to the lower id
    scale = torch.from_numpy(rng.uniform(0.3, 30.0, size=M).astype(F32))
    tok, conf, logits = B.op_lm_head_confidence(hf.cuda(), W.cuda(), scale.cuda(), mask_id, want_logits=True)
    tok, conf, z = tok.cpu().numpy(), conf.cpu().numpy(), logits.cpu().numpy()
    ref = (hf.double().numpy() @ W.double().numpy().T) * scale.double().numpy()[:, None]
    assert rel_err(z, ref) < 1e-4
    tok_ref, conf_ref = O.confidence(z, mask_id)
    assert (tok == tok_ref).all()
    assert (tok != mask_id).all() and (tok != 300).all()
    assert (np.abs(conf - conf_ref) / conf_ref).max() < 1e-4
    tok2, conf2 = B.op_confidence(logits, mask_id)
    assert (tok2.cpu().numpy() == tok).all() and (np.abs(conf2.cpu().numpy() - conf) / conf).max() < 1e-4
    # without the logits store the decisions are the same
    tok3, conf3, none = B.op_lm_head_confidence(hf.cuda(), W.cuda(), scale.cuda(), mask_id)
    assert none is None and (tok3.cpu().numpy() == tok).all() and (conf3.cpu().numpy() == conf).all()
