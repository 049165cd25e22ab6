"""ctypes binding of the C ABI in include/blockserve.h (argument marshalling only).

PyTorch provides device memory and the CUDA stream; every step of the path runs
in the library's kernels.  Importing this module without the built library, or
creating an engine without a CUDA device, raises: there is no CPU path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# BS_DEBUG_LIB=1 selects the bounds-checked build (paper_2607_08930_b200.build.build(debug=True))
DEBUG_LIB = bool(os.environ.get("BS_DEBUG_LIB"))
LIB_PATH = os.path.join(_HERE, "libblockserve_dbg.so" if DEBUG_LIB else "libblockserve.so")
BUILD_BOUNDS_CHECK = 1

BS_OK, BS_E_ARG, BS_E_STATE, BS_E_BUDGET, BS_E_KV_FULL, BS_E_CUDA, BS_E_TIMEOUT, BS_E_UNKNOWN_REQ = (
    0, -1, -2, -3, -4, -5, -6, -7)
SUFFIX_FULL, SUFFIX_NONE = 0, 1
REFRESH_EVERY_BLOCK, REFRESH_AT_ADMISSION = 0, 1
REQ_QUEUED, REQ_ACTIVE, REQ_FINISHED = 0, 1, 2

(DBG_HEADER, DBG_ROW_SLOT, DBG_ROW_MASK, DBG_ROW_S, DBG_ROW_KV_BASE, DBG_CU_Q, DBG_TOK_ROW, DBG_TOK_POS,
 DBG_TOK_KV, DBG_LM_TOK, DBG_LM_ROW, DBG_LM_SLOT, DBG_PREV_LM_ROW, DBG_PREV_LM_SLOT, DBG_PREV_TOK,
 DBG_PREV_CONF, DBG_PREV_COMMIT, DBG_PREV_LOGITS, DBG_REQ_ID_OF_ROW, DBG_KV_ROW) = range(20)


FAMILIES = ("index", "embed_norm", "gemm_qkv", "rope_kv", "attention", "gemm_o", "gemm_gate_up", "gemm_down",
            "gemm_lm_head", "confidence", "attention_refresh")


class BsConfig(C.Structure):
    _fields_ = [("n_layers", C.c_int), ("d_model", C.c_int), ("n_q_heads", C.c_int), ("n_kv_heads", C.c_int),
                ("head_dim", C.c_int), ("d_ffn", C.c_int), ("vocab", C.c_int), ("mask_id", C.c_int),
                ("rms_eps", C.c_float), ("rope_theta", C.c_float), ("block_len", C.c_int), ("tau", C.c_float),
                ("token_budget", C.c_longlong), ("max_batch", C.c_int), ("max_requests", C.c_int),
                ("max_row_tokens", C.c_int), ("kv_capacity_tokens", C.c_longlong), ("suffix_mode", C.c_int),
                ("sort_queue", C.c_int), ("steps_per_block", C.c_int), ("eos_id", C.c_int),
                ("static_groups", C.c_int), ("async_advance", C.c_int), ("refresh_policy", C.c_int),
                ("keep_logits", C.c_int)]


class BsWeights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p),
                ("wqkv", C.POINTER(C.c_void_p)), ("wo", C.POINTER(C.c_void_p)), ("w_gate", C.POINTER(C.c_void_p)),
                ("w_up", C.POINTER(C.c_void_p)), ("w_down", C.POINTER(C.c_void_p)),
                ("norm1", C.POINTER(C.c_void_p)), ("norm2", C.POINTER(C.c_void_p))]


class BsSizes(C.Structure):
    _fields_ = [("kv_bytes", C.c_size_t), ("workspace_bytes", C.c_size_t), ("state_bytes", C.c_size_t)]


class BsStats(C.Structure):
    _fields_ = [("steps", C.c_longlong), ("cycles", C.c_longlong), ("sum_active", C.c_longlong),
                ("committed", C.c_longlong), ("packed_tokens", C.c_longlong), ("lm_rows", C.c_longlong),
                ("kernel_launches", C.c_longlong), ("row_steps", C.c_longlong), ("active_row_steps", C.c_longlong)]


EXPORTS = ["bs_query_sizes", "bs_init_model", "bs_admit", "bs_evict_refill", "bs_denoise_step", "bs_block_done",
           "bs_read_tokens", "bs_get_stats", "bs_set_profiling", "bs_get_profile", "bs_destroy", "bs_last_error", "bs_build_flags", "bs_debug_read", "bs_debug_inject_timeout",
           "bs_debug_force_commit", "bs_debug_snapshot", "bs_debug_restore", "bs_op_gemm", "bs_op_gemm_cluster_splits",
           "bs_op_rmsnorm", "bs_op_rope_kv", "bs_op_rope_kv_static", "bs_op_attention_q_tile", "bs_op_attention", "bs_op_confidence",
           "bs_op_lm_head_confidence", "bs_op_lm_head_confidence_scratch_bytes"]

_lib = None


def lib() -> C.CDLL:
    """Load the CUDA library (built in-tree by paper_2607_08930_b200/build.py)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2607_08930_b200.build` "
                               "(the engine has no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        vp, ip, i, f, ll = C.c_void_p, C.POINTER(C.c_int), C.c_int, C.c_float, C.c_longlong
        L.bs_query_sizes.argtypes = [C.POINTER(BsConfig), C.POINTER(BsSizes)]
        L.bs_init_model.argtypes = [C.POINTER(BsConfig), C.POINTER(BsWeights), vp, vp, vp, vp, C.POINTER(vp)]
        L.bs_admit.argtypes = [vp, ll, ip, i, i, f, i, ip]
        L.bs_evict_refill.argtypes = [vp, ip, ip, ip]
        L.bs_denoise_step.argtypes = [vp, ip]
        L.bs_block_done.argtypes = [vp, ip, C.POINTER(C.c_ubyte)]
        L.bs_read_tokens.argtypes = [vp, ll, ip, i, ip, ip]
        L.bs_get_stats.argtypes = [vp, C.POINTER(BsStats)]
        L.bs_set_profiling.argtypes = [vp, i]
        L.bs_get_profile.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(ll), C.POINTER(C.c_double),
                                     C.POINTER(C.c_double)]
        L.bs_destroy.argtypes = [vp]
        L.bs_destroy.restype = None
        L.bs_last_error.argtypes = [vp]
        L.bs_last_error.restype = C.c_char_p
        L.bs_build_flags.argtypes = []
        L.bs_debug_read.argtypes = [vp, i, i, i, vp, C.c_size_t, C.POINTER(C.c_size_t)]
        L.bs_debug_inject_timeout.argtypes = [vp]
        L.bs_debug_force_commit.argtypes = [vp, i, C.c_ulonglong, vp]
        L.bs_debug_snapshot.argtypes = [vp, vp, C.c_size_t, C.POINTER(C.c_size_t)]
        L.bs_debug_restore.argtypes = [vp, vp, C.c_size_t]
        L.bs_op_gemm.argtypes = [vp, i, vp, vp, vp, i, i, i, i, i, vp, vp, C.c_size_t, vp, vp]
        L.bs_op_gemm_cluster_splits.argtypes = [i, i, i, i]
        L.bs_op_rmsnorm.argtypes = [vp, vp, vp, vp, i, i, f, vp]
        L.bs_op_rope_kv.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, f, i, vp, vp]
        L.bs_op_rope_kv_static.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, f, i, vp]
        L.bs_op_attention_q_tile.argtypes = [i, i, i]
        L.bs_op_attention.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i, i, i, i, i, ll, i, i, i, vp, C.c_size_t, vp, vp]
        L.bs_op_confidence.argtypes = [vp, i, i, i, vp, vp, vp]
        L.bs_op_lm_head_confidence_scratch_bytes.argtypes = [i, i]
        L.bs_op_lm_head_confidence_scratch_bytes.restype = C.c_size_t
        L.bs_op_lm_head_confidence.argtypes = [vp, i, vp, i, i, i, vp, i, vp, C.c_size_t, vp, vp, vp, vp, vp]
        _lib = L
    return _lib


class BlockServeError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"blockserve error {code}: {msg}")
        self.code = code


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check_op(rc: int, name: str) -> None:
    if rc != BS_OK:
        raise BlockServeError(rc, f"{name} failed")


def make_config(shape, block_len: int, tau: float, token_budget: int, max_batch: int, max_requests: int,
                max_row_tokens: int, kv_capacity_tokens: int, suffix_mode: int = SUFFIX_FULL,
                sort_queue: bool = True, steps_per_block: int = 0, eos_id: int = -1,
                static_groups: bool = False, keep_logits: bool = False, async_advance: bool = False,
                refresh_policy: int = 0) -> BsConfig:
    return BsConfig(shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.d_ffn,
                    shape.vocab, shape.mask_id, shape.rms_eps, shape.rope_theta, block_len, tau, token_budget,
                    max_batch, max_requests, max_row_tokens, kv_capacity_tokens, suffix_mode, int(sort_queue),
                    int(steps_per_block), int(eos_id), int(static_groups), int(async_advance), int(refresh_policy),
                    int(keep_logits))


def query_sizes(cfg: BsConfig) -> BsSizes:
    out = BsSizes()
    rc = lib().bs_query_sizes(C.byref(cfg), C.byref(out))
    if rc != BS_OK:
        raise BlockServeError(rc, (lib().bs_last_error(None) or b"").decode())
    return out


class Engine:
    """Owns the torch buffers an engine borrows and forwards calls to the C ABI."""

    def __init__(self, cfg: BsConfig, weights: Dict[str, object], device: str = "cuda:0"):
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: the block-denoising engine has no CPU fallback")
        self.L = lib()
        self.cfg = cfg
        self.device = torch.device(device)
        sz = query_sizes(cfg)
        self.sizes = sz
        with torch.cuda.device(self.device):
            self.kv = torch.empty(sz.kv_bytes, dtype=torch.uint8, device=self.device)
            self.workspace = torch.empty(sz.workspace_bytes, dtype=torch.uint8, device=self.device)
            self.state = torch.empty(sz.state_bytes, dtype=torch.uint8, device=self.device)
            self.weights = weights        # keep the tensors alive
            n = cfg.n_layers
            arrs = {}
            for name in ("wqkv", "wo", "w_gate", "w_up", "w_down", "norm1", "norm2"):
                ts = weights[name]
                assert len(ts) == n and all(t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous() for t in ts)
                arrs[name] = (C.c_void_p * n)(*[t.data_ptr() for t in ts])
            self._arrs = arrs
            w = BsWeights(weights["embed"].data_ptr(), weights["lm_head"].data_ptr(),
                          weights["final_norm"].data_ptr(),
                          *[C.cast(arrs[k], C.POINTER(C.c_void_p)) for k in
                            ("wqkv", "wo", "w_gate", "w_up", "w_down", "norm1", "norm2")])
            h = C.c_void_p()
            rc = self.L.bs_init_model(C.byref(cfg), C.byref(w), self.kv.data_ptr(), self.workspace.data_ptr(),
                                      self.state.data_ptr(), _stream(), C.byref(h))
        if rc != BS_OK:
            raise BlockServeError(rc, (self.L.bs_last_error(None) or b"").decode())
        self.h = h

    def _chk(self, rc: int) -> None:
        if rc != BS_OK:
            raise BlockServeError(rc, (self.L.bs_last_error(self.h) or b"").decode())

    def admit(self, req_id: int, prompt: Sequence[int], g: int, alpha: float, start_block: int = 0,
              gen_prefix: Optional[Sequence[int]] = None) -> None:
        pr = np.ascontiguousarray(prompt, dtype=np.int32)
        gp = None if gen_prefix is None else np.ascontiguousarray(gen_prefix, dtype=np.int32)
        ip = C.POINTER(C.c_int)
        self._chk(self.L.bs_admit(self.h, req_id, pr.ctypes.data_as(ip), len(pr), g, alpha, start_block,
                                  None if gp is None else gp.ctypes.data_as(ip)))

    def evict_refill(self):
        a, b, c = C.c_int(), C.c_int(), C.c_int()
        self._chk(self.L.bs_evict_refill(self.h, C.byref(a), C.byref(b), C.byref(c)))
        return a.value, b.value, c.value

    def denoise_step(self, want_count: bool = False) -> Optional[int]:
        if want_count:
            n = C.c_int()
            self._chk(self.L.bs_denoise_step(self.h, C.byref(n)))
            return n.value
        self._chk(self.L.bs_denoise_step(self.h, None))
        return None

    def block_done(self) -> bool:
        d = C.c_int()
        self._chk(self.L.bs_block_done(self.h, C.byref(d), None))
        return bool(d.value)

    def rows_done(self) -> np.ndarray:
        d = C.c_int()
        buf = (C.c_ubyte * self.cfg.max_batch)()
        self._chk(self.L.bs_block_done(self.h, C.byref(d), buf))
        return np.frombuffer(buf, dtype=np.uint8).copy()

    def read_tokens(self, req_id: int):
        n, st = C.c_int(), C.c_int()
        self._chk(self.L.bs_read_tokens(self.h, req_id, None, 0, C.byref(n), C.byref(st)))
        out = np.empty(n.value, dtype=np.int32)
        self._chk(self.L.bs_read_tokens(self.h, req_id, out.ctypes.data_as(C.POINTER(C.c_int)), n.value,
                                        C.byref(n), C.byref(st)))
        return out, st.value

    def stats(self) -> BsStats:
        s = BsStats()
        self._chk(self.L.bs_get_stats(self.h, C.byref(s)))
        return s

    def inject_timeout(self) -> None:
        self._chk(self.L.bs_debug_inject_timeout(self.h))

    def force_commit(self, row: int, positions: Dict[int, int]) -> None:
        """Commit block position -> token for the given active row (debugging aid)."""
        toks = np.zeros(64, dtype=np.int32)
        bits = 0
        for j, t in positions.items():
            toks[j] = t
            bits |= 1 << j
        self._chk(self.L.bs_debug_force_commit(self.h, row, bits, toks.ctypes.data))

    def snapshot(self) -> np.ndarray:
        """Engine state between block cycles as bytes (token rows + scheduler state; the KV cache is rebuilt)."""
        n = C.c_size_t(0)
        self._chk(self.L.bs_debug_snapshot(self.h, None, 0, C.byref(n)))
        buf = np.empty(n.value, dtype=np.uint8)
        self._chk(self.L.bs_debug_snapshot(self.h, buf.ctypes.data, buf.nbytes, C.byref(n)))
        return buf[:n.value]

    def restore(self, snap: np.ndarray) -> None:
        snap = np.ascontiguousarray(snap, dtype=np.uint8)
        self._chk(self.L.bs_debug_restore(self.h, snap.ctypes.data, snap.nbytes))

    def set_profiling(self, on: bool) -> None:
        self._chk(self.L.bs_set_profiling(self.h, int(on)))

    def profile(self) -> Dict[str, Dict[str, float]]:
        """Per kernel family: device ms, launches, algorithmic flops and bytes since profiling was enabled."""
        n = len(FAMILIES)
        ms, fl, by = (C.c_double * n)(), (C.c_double * n)(), (C.c_double * n)()
        la = (C.c_longlong * n)()
        self._chk(self.L.bs_get_profile(self.h, ms, la, fl, by))
        return {FAMILIES[i]: dict(ms=ms[i], launches=int(la[i]), flops=fl[i], bytes=by[i]) for i in range(n)}

    def debug(self, what: int, dtype=np.int32, arg0: int = 0, arg1: int = 0, cap: int = 1 << 16) -> np.ndarray:
        buf = np.empty(cap, dtype=np.uint8)
        n = C.c_size_t()
        self._chk(self.L.bs_debug_read(self.h, what, arg0, arg1, buf.ctypes.data, cap, C.byref(n)))
        return buf[:n.value].view(dtype).copy()

    def run(self, max_cycles: int = 1 << 30) -> int:
        """Algorithm 1 until the pending queue and the active set are empty."""
        cycles = 0
        while cycles < max_cycles:
            _, _, n = self.evict_refill()
            if n == 0:
                break
            while True:
                self.denoise_step()
                if self.block_done():
                    break
            cycles += 1
        return cycles

    def close(self) -> None:
        if getattr(self, "h", None):
            self.L.bs_destroy(self.h)      # synchronises the engine's stream
            self.h = None
            self.kv = self.workspace = self.state = None    # give the arenas back to the allocator

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def engine_for_workload(wl, weights, *, kv_capacity_tokens: Optional[int] = None, suffix_mode: int = SUFFIX_FULL,
                        sort_queue: bool = True, steps_per_block: int = 0, eos_id: int = -1,
                        static_groups: bool = False, keep_logits: bool = False, async_advance: bool = False,
                        refresh_policy: int = 0, device: str = "cuda:0") -> Engine:
    """Size an engine for a bs_inputs.Workload (the caller still admits the requests)."""
    mrt = wl.max_row_tokens
    if kv_capacity_tokens is None:
        rows = sorted((r.p + r.g for r in wl.requests), reverse=True)[:wl.max_batch]
        kv_capacity_tokens = sum(rows)
        if wl.token_budget > 0:       # Eq. 1 bounds |A| * width; rows are at most width + g long
            kv_capacity_tokens = min(kv_capacity_tokens, wl.token_budget + wl.max_batch * max(r.g for r in wl.requests))
    cfg = make_config(wl.shape, wl.block_len, wl.tau, wl.token_budget, wl.max_batch, len(wl.requests), mrt,
                      max(kv_capacity_tokens, mrt), suffix_mode, sort_queue, steps_per_block, eos_id, static_groups,
                      keep_logits, async_advance, refresh_policy)
    return Engine(cfg, weights, device)


# ---- single operations -------------------------------------------------------------------------------------

def op_gemm(A: torch.Tensor, W: torch.Tensor, mode: int = 0, W2: Optional[torch.Tensor] = None,
            C_out: Optional[torch.Tensor] = None, row_scale: Optional[torch.Tensor] = None,
            scratch: Optional[torch.Tensor] = None, error_flag: Optional[torch.Tensor] = None) -> torch.Tensor:
    M, K = A.shape
    N = W.shape[0]
    if C_out is None:
        C_out = torch.empty(M, N, dtype=torch.bfloat16 if mode in (0, 3) else torch.float32, device=A.device)
    _check_op(lib().bs_op_gemm(A.data_ptr(), A.stride(0), W.data_ptr(), _ptr(W2), C_out.data_ptr(), C_out.stride(0),
                               M, N, K, mode, _ptr(row_scale), _ptr(scratch),
                               0 if scratch is None else scratch.numel() * scratch.element_size(),
                               _ptr(error_flag), _stream()), "bs_op_gemm")
    return C_out


def op_gemm_cluster_splits(M: int, N: int, K: int, mode: int) -> int:
    """CTA pairs that share each output tile's K range inside one cluster for this op_gemm call (0: another plan)."""
    return int(lib().bs_op_gemm_cluster_splits(M, N, K, mode))


def op_rmsnorm(x: torch.Tensor, w: torch.Tensor, eps: float, idx: Optional[torch.Tensor] = None) -> torch.Tensor:
    M = x.shape[0] if idx is None else idx.shape[0]
    y = torch.empty(M, x.shape[1], dtype=torch.bfloat16, device=x.device)
    _check_op(lib().bs_op_rmsnorm(x.data_ptr(), _ptr(idx), w.data_ptr(), y.data_ptr(), M, x.shape[1], eps, _stream()),
              "bs_op_rmsnorm")
    return y


def op_rope_kv(qkv, tok_pos, tok_kv, kcache, vcache, hq, hkv, dh, theta, max_pos) -> None:
    scratch = torch.empty(max_pos * dh, dtype=torch.float32, device=qkv.device)
    _check_op(lib().bs_op_rope_kv(qkv.data_ptr(), tok_pos.data_ptr(), tok_kv.data_ptr(), kcache.data_ptr(),
                                  vcache.data_ptr(), qkv.shape[0], hq, hkv, dh, theta, max_pos, scratch.data_ptr(),
                                  _stream()), "bs_op_rope_kv")
    torch.cuda.current_stream().synchronize()


ROPE_STATIC_MAX_FLOATS = 512 * 1024


def op_rope_kv_static(qkv, tok_pos, tok_kv, kcache, vcache, hq, hkv, dh, theta, max_pos) -> int:
    """bs_op_rope_kv for callers that cannot allocate: the cos/sin table lives inside the library (at most
    ROPE_STATIC_MAX_FLOATS = max_pos * head_dim floats).  Nothing is allocated here either: the wrapper only
    passes the caller's pointers through.  Returns the status code (BS_E_ARG when the table would not fit)."""
    return lib().bs_op_rope_kv_static(qkv.data_ptr(), tok_pos.data_ptr(), tok_kv.data_ptr(), kcache.data_ptr(),
                                      vcache.data_ptr(), qkv.shape[0], hq, hkv, dh, theta, max_pos, _stream())


def attention_plan(cu_q: torch.Tensor, vis: torch.Tensor, hq: int, hkv: int, dh: int = 128):
    """Work-item prefix over rows (q-tiles) and the launch scalars of bs_op_attention; involves a device-to-host
    copy, so callers that launch repeatedly build it once."""
    qt = lib().bs_op_attention_q_tile(hq, hkv, dh)
    cu = cu_q.detach().cpu().numpy().astype(np.int64)
    tiles = np.zeros(len(cu), dtype=np.int32)
    tiles[1:] = np.cumsum((cu[1:] - cu[:-1] + qt - 1) // qt)
    return dict(cu_tile=torch.from_numpy(tiles).to(cu_q.device), n_tiles=int(tiles[-1]),
                max_vis=int(vis.max().item()) if len(vis) else 0,
                max_nq=int((cu[1:] - cu[:-1]).max()) if len(cu) > 1 else 0)


def op_attention(qkv, kcache, vcache, cu_q, kv_base, vis, hq, hkv, dh, scratch: Optional[torch.Tensor] = None,
                 plan=None, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    plan = plan or attention_plan(cu_q, vis, hq, hkv, dh)
    if out is None:
        out = torch.empty(qkv.shape[0], hq * dh, dtype=torch.bfloat16, device=qkv.device)
    _check_op(lib().bs_op_attention(qkv.data_ptr(), kcache.data_ptr(), vcache.data_ptr(), out.data_ptr(),
                                    cu_q.data_ptr(), plan["cu_tile"].data_ptr(), kv_base.data_ptr(), vis.data_ptr(),
                                    len(cu_q) - 1, plan["n_tiles"], qkv.shape[0], plan["max_vis"], plan["max_nq"],
                                    kcache.shape[0], hq, hkv, dh, _ptr(scratch),
                                    0 if scratch is None else scratch.numel() * scratch.element_size(),
                                    None, _stream()), "bs_op_attention")
    return out


def lm_head_confidence_buffers(M: int, V: int, device) -> dict:
    """Buffers of op_lm_head_confidence, for callers that launch repeatedly."""
    nbytes = lib().bs_op_lm_head_confidence_scratch_bytes(M, V)
    return dict(scratch=torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device), nbytes=nbytes,
                tok=torch.empty(M, dtype=torch.int32, device=device),
                conf=torch.empty(M, dtype=torch.float32, device=device),
                flag=torch.zeros(1, dtype=torch.int32, device=device))


def op_lm_head_confidence(hf: torch.Tensor, W: torch.Tensor, row_scale: torch.Tensor, mask_id: int,
                          want_logits: bool = False, buffers: Optional[dict] = None):
    """LM head with the confidence pass in its epilogue: (tok int32 [M], conf fp32 [M], logits fp32 [M, V] or None).
    With `buffers` (from lm_head_confidence_buffers) nothing is allocated and the stream is not synchronised."""
    M, K = hf.shape
    V = W.shape[0]
    b = buffers or lm_head_confidence_buffers(M, V, hf.device)
    logits = torch.empty(M, V, dtype=torch.float32, device=hf.device) if want_logits else None
    _check_op(lib().bs_op_lm_head_confidence(hf.data_ptr(), hf.stride(0), W.data_ptr(), M, V, K, row_scale.data_ptr(),
                                             mask_id, b["scratch"].data_ptr(), b["nbytes"], b["tok"].data_ptr(),
                                             b["conf"].data_ptr(), _ptr(logits), b["flag"].data_ptr(), _stream()),
              "bs_op_lm_head_confidence")
    if buffers is None:
        torch.cuda.current_stream().synchronize()
        if int(b["flag"].item()):
            raise BlockServeError(BS_E_TIMEOUT, "a bounded device-side wait ran out")
    return b["tok"], b["conf"], logits


def op_confidence(logits: torch.Tensor, mask_id: int):
    n, V = logits.shape
    tok = torch.empty(n, dtype=torch.int32, device=logits.device)
    conf = torch.empty(n, dtype=torch.float32, device=logits.device)
    _check_op(lib().bs_op_confidence(logits.data_ptr(), n, V, mask_id, tok.data_ptr(), conf.data_ptr(), _stream()),
              "bs_op_confidence")
    return tok, conf
