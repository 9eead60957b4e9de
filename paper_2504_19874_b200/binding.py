"""ctypes binding of include/tq.h.  Argument marshalling only."""
from __future__ import annotations

import ctypes
import os

import numpy as np
import torch

TQ_MSE, TQ_PROD = 0, 1
TQ_F32, TQ_BF16 = 0, 1
TQ_ORTHOGONAL, TQ_GAUSSIAN = 0, 1
TQ_LAYOUT_CANONICAL, TQ_LAYOUT_NIBBLE = 0, 1
TQ_OP_QUANTIZE, TQ_OP_SCORE, TQ_OP_TOPK, TQ_OP_WSUM, TQ_OP_DEQUANTIZE = 0, 1, 2, 3, 4
TQ_STATIC_SCRATCH_BYTES = 1 << 20

# TQ_LIB_VARIANT=debug loads libtq_debug.so, the build with device-side index checks (build.py --debug)
_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)),
                         "libtq_debug.so" if os.environ.get("TQ_LIB_VARIANT") == "debug" else "libtq.so")
_lib = None

c_void_p, c_int, c_int64, c_size_t, c_u64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_size_t, ctypes.c_uint64
_F = ctypes.POINTER(ctypes.c_float)

_SIGNATURES = {
    "tq_last_error": (ctypes.c_char_p, []),
    "tq_launch_count": (c_u64, []),
    "tq_codebook": (c_int, [c_int, c_int, _F, _F]),
    "tq_rotation": (c_int, [c_int, c_u64, c_int, _F]),
    "tq_idx_row_bytes": (c_size_t, [c_int, c_int]),
    "tq_qjl_row_bytes": (c_size_t, [c_int]),
    "tq_plan_create": (c_int, [c_int, c_int, c_int, _F, _F, _F, ctypes.POINTER(c_void_p)]),
    "tq_plan_destroy": (c_int, [c_void_p]),
    "tq_plan_status": (c_int, [c_void_p]),
    "tq_plan_set_layout": (c_int, [c_void_p, c_int]),
    "tq_plan_layout": (c_int, [c_void_p]),
    "tq_convert_layout": (c_int, [c_void_p, c_int64, c_void_p, c_void_p, c_int, c_int, c_void_p]),
    "tq_workspace_bytes": (c_size_t, [c_void_p, c_int, c_int64, c_int, c_int]),
    "tq_quantize_mse": (c_int, [c_void_p, c_void_p, c_int, c_int64, c_int64, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]),
    "tq_quantize_prod": (c_int, [c_void_p, c_void_p, c_int, c_int64, c_int64, c_void_p, c_void_p, c_void_p, c_void_p,
                                 c_void_p, c_size_t, c_void_p]),
    "tq_dequantize": (c_int, [c_void_p, c_int64, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int64, c_void_p]),
    "tq_score": (c_int, [c_void_p, c_void_p, c_int, c_int, c_int64, c_int64, c_void_p, c_void_p, c_void_p, c_void_p,
                         c_void_p, c_int64, c_void_p, c_size_t, c_void_p]),
    "tq_score_static": (c_int, [c_void_p, c_void_p, c_int, c_int, c_int64, c_int64, c_void_p, c_void_p, c_void_p, c_void_p,
                                c_void_p, c_int64, c_void_p]),
    "tq_score_static_max_queries": (c_int, [c_void_p]),
    "tq_query_bytes": (c_size_t, [c_void_p, c_int]),
    "tq_query_prepare": (c_int, [c_void_p, c_void_p, c_int, c_int, c_int64, c_void_p, c_size_t, c_void_p]),
    "tq_score_prepared": (c_int, [c_void_p, c_void_p, c_int, c_int64, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                  c_int64, c_void_p]),
    "tq_selftest_wait_timeout": (c_int, [c_void_p, ctypes.c_longlong, c_void_p]),
    "tq_entropy_lengths": (c_int, [c_int, c_int, _F, c_void_p]),
    "tq_entropy_workspace_bytes": (c_size_t, [c_int64]),
    "tq_entropy_measure": (c_int, [c_void_p, c_void_p, c_int64, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]),
    "tq_entropy_pack": (c_int, [c_void_p, c_void_p, c_int64, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]),
    "tq_entropy_unpack": (c_int, [c_void_p, c_void_p, c_int64, c_void_p, c_void_p, c_void_p, c_void_p]),
    "tq_topk": (c_int, [c_void_p, c_void_p, c_int, c_int, c_int64, c_int64, c_void_p, c_void_p, c_void_p, c_void_p,
                        c_int, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]),
    "tq_select_topk": (c_int, [c_void_p, c_void_p, c_int, c_int64, c_int64, c_int, c_void_p, c_void_p, c_void_p]),
    "tq_softmax": (c_int, [c_void_p, c_void_p, c_int, c_int64, c_int64, ctypes.c_float, c_void_p, c_int64, c_void_p]),
    "tq_wsum": (c_int, [c_void_p, c_void_p, c_int, c_int64, c_int64, c_void_p, c_void_p, c_void_p, c_void_p,
                        c_void_p, c_int64, c_void_p, c_size_t, c_void_p]),
    "tq_attend_decode_workspace_bytes": (c_size_t, [c_int, c_int, c_int64, c_int]),
    "tq_attend_decode": (c_int, [c_void_p, c_int, c_int, c_int64, c_int64, c_int, c_void_p, c_int, c_int64, ctypes.c_float,
                                 c_void_p, c_int64, c_void_p, c_size_t, c_void_p]),
    "tq_kv_append": (c_int, [c_void_p, c_int, c_int, c_int64, c_int64, c_void_p, c_void_p, c_int, c_int64, c_int64, c_void_p]),
}


class KvGroup(ctypes.Structure):
    """struct tq_kv_group of include/tq.h (one channel group of a compressed KV layer)."""
    _fields_ = [(name, c_void_p) for name in ("plan_k", "plan_v", "k_idx", "k_qjl", "k_gamma", "k_norms", "v_idx", "v_norms",
                                              "k_channels", "v_channels")]


class TqError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__(f"tq error {code}: {message}")
        self.code = code


def lib() -> ctypes.CDLL:
    """Loads libtq.so (built in-tree by paper_2504_19874_b200/build.py).  Raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} is missing: run `python -m paper_2504_19874_b200.build` first "
                               "(there is no fallback path)")
        handle = ctypes.CDLL(_LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype, fn.argtypes = res, args
        _lib = handle
    return _lib


def _check(code: int):
    if code != 0:
        raise TqError(code, lib().tq_last_error().decode())


def _fptr(a: np.ndarray):
    return a.ctypes.data_as(_F)


def _dev(t):
    """Device pointer of a CUDA tensor (None -> NULL)."""
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("expected a CUDA tensor (this library has no CPU path)")
    return t.data_ptr()


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return TQ_F32
    if t.dtype == torch.bfloat16:
        return TQ_BF16
    raise ValueError(f"unsupported dtype {t.dtype}")


def _rows(t: torch.Tensor):
    if t.dim() != 2 or t.stride(1) != 1:
        raise ValueError("expected a 2-D tensor with unit inner stride")
    return t.shape[0], t.stride(0) if t.shape[0] > 1 else max(t.stride(0), t.shape[1])


def _stream():
    return torch.cuda.current_stream().cuda_stream


def tq_launch_count() -> int:
    return lib().tq_launch_count()


def tq_idx_row_bytes(d: int, bits: int) -> int:
    return lib().tq_idx_row_bytes(d, bits)


def tq_qjl_row_bytes(d: int) -> int:
    return lib().tq_qjl_row_bytes(d)


def tq_codebook(d: int, bits: int):
    """(centroids, boundaries) as float32 numpy arrays."""
    levels = 1 << min(max(bits, 0), 8)        # the library rejects bits outside 0..4
    c = np.zeros(levels, dtype=np.float32)
    t = np.zeros(max(levels - 1, 1), dtype=np.float32)
    _check(lib().tq_codebook(d, bits, _fptr(c), _fptr(t)))
    return c, t[:levels - 1]


def tq_rotation(d: int, seed: int, kind: int = TQ_ORTHOGONAL) -> np.ndarray:
    out = np.zeros((d, d), dtype=np.float32)
    _check(lib().tq_rotation(d, seed, kind, _fptr(out)))
    return out


class Plan:
    """Owner of a tq_plan handle (device copies of Pi, S', codebook for one (d, b, mode))."""

    def __init__(self, d: int, bits: int, mode: int, Pi, S, centroids):
        Pi = np.ascontiguousarray(Pi, dtype=np.float32)
        cent = np.ascontiguousarray(centroids, dtype=np.float32)
        Sp = None if S is None else np.ascontiguousarray(S, dtype=np.float32)
        if Pi.shape != (d, d) or (Sp is not None and Sp.shape != (d, d)):
            raise ValueError("Pi and S must be d x d")
        self.d, self.bits, self.mode = d, bits, mode
        self.mse_bits = bits - 1 if mode == TQ_PROD else bits
        if cent.size != (1 << max(self.mse_bits, 0)):
            raise ValueError("centroids must hold 2^b_m values")
        self.idx_row_bytes = tq_idx_row_bytes(d, self.mse_bits)
        self.qjl_row_bytes = tq_qjl_row_bytes(d)
        h = c_void_p()
        _check(lib().tq_plan_create(d, bits, mode, _fptr(Pi), None if Sp is None else _fptr(Sp), _fptr(cent),
                                    ctypes.byref(h)))
        self.handle = h

    def set_layout(self, layout: int) -> None:
        """TQ_LAYOUT_CANONICAL or TQ_LAYOUT_NIBBLE (TQ_PROD with b = 4 only): arrangement of the code rows."""
        _check(lib().tq_plan_set_layout(self.handle, layout))

    @property
    def layout(self) -> int:
        return lib().tq_plan_layout(self.handle)

    def close(self):
        if getattr(self, "handle", None):
            lib().tq_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def tq_plan_status(plan: Plan) -> None:
    """Synchronises and raises TqError(6) if a kernel of this plan gave up a bounded wait."""
    _check(lib().tq_plan_status(plan.handle))


def tq_convert_layout(plan: Plan, n: int, idx, qjl, src: int, dst: int) -> None:
    """Rewrites n rows of (idx, qjl) in place from layout `src` into layout `dst`."""
    _check(lib().tq_convert_layout(plan.handle, n, _dev(idx), _dev(qjl), src, dst, _stream()))


def tq_workspace_bytes(plan: Plan, op: int, n: int, nq: int = 0, k: int = 0) -> int:
    return lib().tq_workspace_bytes(plan.handle, op, n, nq, k)


def _scratch_args(t):
    return (_dev(t), 0 if t is None else t.numel() * t.element_size())


def tq_quantize_mse(plan: Plan, X, idx, norms=None, scratch=None):
    n, ldx = _rows(X)
    _check(lib().tq_quantize_mse(plan.handle, _dev(X), _dtype_code(X), n, ldx, _dev(idx), _dev(norms),
                                 *_scratch_args(scratch), _stream()))


def tq_quantize_prod(plan: Plan, X, idx, qjl, gamma, norms=None, scratch=None):
    n, ldx = _rows(X)
    _check(lib().tq_quantize_prod(plan.handle, _dev(X), _dtype_code(X), n, ldx, _dev(idx), _dev(qjl), _dev(gamma),
                                  _dev(norms), *_scratch_args(scratch), _stream()))


def tq_dequantize(plan: Plan, n: int, idx, qjl, gamma, norms, Xhat):
    _, ld = _rows(Xhat)
    _check(lib().tq_dequantize(plan.handle, n, _dev(idx), _dev(qjl), _dev(gamma), _dev(norms), _dev(Xhat), ld, _stream()))


def tq_score(plan: Plan, Q, n: int, idx, qjl, gamma, norms, scores, workspace):
    nq, ldq = _rows(Q)
    _, lds = _rows(scores)
    _check(lib().tq_score(plan.handle, _dev(Q), _dtype_code(Q), nq, ldq, n, _dev(idx), _dev(qjl), _dev(gamma),
                          _dev(norms), _dev(scores), lds, *_scratch_args(workspace), _stream()))


def tq_score_static(plan: Plan, Q, n: int, idx, qjl, gamma, norms, scores):
    """tq_score for callers that cannot allocate device memory: the rotated-query workspace is an
    array built into the library (TQ_STATIC_SCRATCH_BYTES), shared by every call on the device."""
    nq, ldq = _rows(Q)
    _, lds = _rows(scores)
    _check(lib().tq_score_static(plan.handle, _dev(Q), _dtype_code(Q), nq, ldq, n, _dev(idx), _dev(qjl), _dev(gamma),
                                 _dev(norms), _dev(scores), lds, _stream()))


def tq_score_static_max_queries(plan: Plan) -> int:
    return lib().tq_score_static_max_queries(plan.handle)


def tq_query_bytes(plan: Plan, nq: int) -> int:
    return lib().tq_query_bytes(plan.handle, nq)


def tq_query_prepare(plan: Plan, Q, prepared):
    """Query-side work of tq_score (rotations, scan operand) into `prepared` (>= tq_query_bytes(plan, nq) bytes)."""
    nq, ldq = _rows(Q)
    _check(lib().tq_query_prepare(plan.handle, _dev(Q), _dtype_code(Q), nq, ldq, *_scratch_args(prepared), _stream()))


def tq_score_prepared(plan: Plan, prepared, nq: int, n: int, idx, qjl, gamma, norms, scores):
    _, lds = _rows(scores)
    _check(lib().tq_score_prepared(plan.handle, _dev(prepared), nq, n, _dev(idx), _dev(qjl), _dev(gamma), _dev(norms),
                                   _dev(scores), lds, _stream()))


def tq_selftest_wait_timeout(plan: Plan, limit_cycles: int = 20000) -> None:
    """Enqueues the library's bounded-wait self test; the next tq_plan_status(plan) must raise TqError(6)."""
    _check(lib().tq_selftest_wait_timeout(plan.handle, limit_cycles, _stream()))


def tq_topk(plan: Plan, Q, n: int, idx, qjl, gamma, norms, k: int, top_scores, top_ids, workspace):
    nq, ldq = _rows(Q)
    _check(lib().tq_topk(plan.handle, _dev(Q), _dtype_code(Q), nq, ldq, n, _dev(idx), _dev(qjl), _dev(gamma),
                         _dev(norms), k, _dev(top_scores), _dev(top_ids), *_scratch_args(workspace), _stream()))


def tq_wsum(plan: Plan, W, n: int, idx, qjl, gamma, norms, out, workspace):
    nw, ldo = _rows(out)
    ldw = _rows(W)[1] if W is not None else n
    _check(lib().tq_wsum(plan.handle, _dev(W), nw, ldw, n, _dev(idx), _dev(qjl), _dev(gamma), _dev(norms),
                         _dev(out), ldo, *_scratch_args(workspace), _stream()))


def tq_softmax(s1, s2, scale: float, W):
    nw, lds = _rows(s1)
    _, ldw = _rows(W)
    n = s1.shape[1]
    if s2 is not None and (_rows(s2)[1] != lds or s2.shape != s1.shape):
        raise ValueError("s2 must have the shape and row stride of s1")
    _check(lib().tq_softmax(_dev(s1), _dev(s2), nw, n, lds, scale, _dev(W), ldw, _stream()))


def tq_attend_decode_workspace_bytes(ngroups: int, heads: int, tokens: int, d: int) -> int:
    return lib().tq_attend_decode_workspace_bytes(ngroups, heads, tokens, d)


def _kv_groups(groups):
    arr = (KvGroup * len(groups))()
    for dst, g in zip(arr, groups):
        dst.plan_k, dst.plan_v = g["plan_k"].handle, g["plan_v"].handle
        for name in ("k_idx", "k_qjl", "k_gamma", "k_norms", "v_idx", "v_norms", "k_channels", "v_channels"):
            setattr(dst, name, _dev(g.get(name)))
        for name in ("k_channels", "v_channels"):
            if g[name].dtype != torch.int32 or not g[name].is_contiguous():
                raise ValueError(f"{name} must be a contiguous int32 tensor")
    return arr


def tq_attend_decode(groups, heads: int, tokens: int, q_per_kv: int, Q, scale: float, out, workspace, head_stride=None):
    """groups: sequence of dicts with keys plan_k, plan_v (Plan) and k_idx, k_qjl, k_gamma, k_norms, v_idx,
    v_norms, k_channels, v_channels (CUDA tensors or None); rows of all heads head-major, head_stride rows
    per head (default: tokens)."""
    arr = _kv_groups(groups)
    _, ldq = _rows(Q)
    _, ldo = _rows(out)
    _check(lib().tq_attend_decode(ctypes.cast(arr, c_void_p), len(groups), heads, tokens,
                                  tokens if head_stride is None else head_stride, q_per_kv, _dev(Q), _dtype_code(Q),
                                  ldq, scale, _dev(out), ldo, *_scratch_args(workspace), _stream()))


def tq_kv_append(groups, heads: int, head_stride: int, position: int, K, V):
    """Quantises one new token per KV head (K, V: [heads, head_dim]) into row `position` of every head."""
    arr = _kv_groups(groups)
    _, ldk = _rows(K)
    _, ldv = _rows(V)
    if K.dtype != V.dtype:
        raise ValueError("K and V must have one dtype")
    _check(lib().tq_kv_append(ctypes.cast(arr, c_void_p), len(groups), heads, head_stride, position, _dev(K), _dev(V),
                              _dtype_code(K), ldk, ldv, _stream()))


def tq_entropy_lengths(d: int, bits: int, centroids) -> np.ndarray:
    """Huffman code lengths of the 2^bits index values for the given codebook (uint8 array)."""
    cent = np.ascontiguousarray(centroids, dtype=np.float32)
    out = np.zeros(1 << bits, dtype=np.uint8)
    _check(lib().tq_entropy_lengths(d, bits, _fptr(cent), out.ctypes.data_as(c_void_p)))
    return out


def tq_entropy_pack(plan: Plan, lengths, n: int, idx):
    """(packed uint8 tensor, row_offsets int64 tensor of n + 1 byte offsets): the entropy-coded index rows."""
    ln = np.ascontiguousarray(lengths, dtype=np.uint8)
    lp = ln.ctypes.data_as(c_void_p)
    dev = idx.device
    offsets = torch.empty(n + 1, dtype=torch.int64, device=dev)
    ws = torch.empty(max(lib().tq_entropy_workspace_bytes(n), 256), dtype=torch.uint8, device=dev)
    _check(lib().tq_entropy_measure(plan.handle, lp, n, _dev(idx), _dev(offsets), *_scratch_args(ws), _stream()))
    total = int(offsets[n].item())
    out = torch.empty(max(total, 4), dtype=torch.uint8, device=dev)
    _check(lib().tq_entropy_pack(plan.handle, lp, n, _dev(idx), _dev(offsets), _dev(out), total, _stream()))
    return out[:total], offsets


def tq_entropy_unpack(plan: Plan, lengths, n: int, packed, offsets, idx_out):
    ln = np.ascontiguousarray(lengths, dtype=np.uint8)
    _check(lib().tq_entropy_unpack(plan.handle, ln.ctypes.data_as(c_void_p), n, _dev(packed), _dev(offsets), _dev(idx_out),
                                   _stream()))


def tq_select_topk(cand_scores, cand_ids, k: int, top_scores, top_ids):
    nq, ld = _rows(cand_scores)
    if _rows(cand_ids)[1] != ld or cand_ids.shape != cand_scores.shape:
        raise ValueError("cand_ids must have the shape and row stride of cand_scores")
    _check(lib().tq_select_topk(_dev(cand_scores), _dev(cand_ids), nq, cand_scores.shape[1], ld, k, _dev(top_scores),
                                _dev(top_ids), _stream()))
