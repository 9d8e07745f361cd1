"""Thin ctypes binding over libshareprefill.so (see include/shareprefill.h).

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  torch is used for device memory and streams.  There is no fallback:
if the shared library has not been built, loading raises.

Tensors: q [Hq, N, d] or [1, Hq, N, d] bf16 CUDA; k, v [Hkv, N, d] likewise.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# SHAREPREFILL_LIB: load this library instead of the in-tree release build (e.g. the range-checked debug build,
# paper_2505_19578_b200/libshareprefill_debug.so, made by `python -m paper_2505_19578_b200.build --debug`)
LIB_PATH = os.environ.get("SHAREPREFILL_LIB") or os.path.join(_HERE, "libshareprefill.so")

SP_OK = 0
SP_ERR_INVALID_ARG = -1
SP_ERR_UNSUPPORTED = -2
SP_ERR_WORKSPACE = -3
SP_ERR_CUDA = -4
SP_ERR_TIMEOUT = -5
SP_ERR_SCRATCH_LIMIT = -6
SP_ERR_RANGE = -7
FIXED_SCRATCH_BYTES = 64 << 20

EXPORTS = (
    "sp_ctx_create", "sp_ctx_destroy", "sp_workspace_bytes", "sp_ctx_reserve", "sp_get_status",
    "sp_strerror", "sp_dense_pivot_attn", "sp_block_mask_from_importance", "sp_block_sparse_attn",
    "sp_prefill_attn", "sp_ctx_set_kernel", "sp_ctx_launch_count", "sp_dense_pivot_attn_fixed_scratch",
    "sp_ctx_set_trace", "sp_prefill_attn_host", "sp_pooled_logits", "sp_pattern_from_pooled",
    "sp_determine_pattern", "sp_vertical_slash_pattern", "sp_prefill_attn_auto",
    "sp_dict_create", "sp_dict_destroy", "sp_dict_clear", "sp_dict_count", "sp_prefill_attn_layer",
    "sp_selftest_wait_timeout", "sp_fixed_scratch_status", "sp_workspace_bytes_patterns",
    "sp_internal_pair_work_order",
)


class SpTensor(ctypes.Structure):
    _fields_ = [("data", ctypes.c_void_p), ("shape", ctypes.c_int64 * 4), ("stride", ctypes.c_int64 * 4)]


class SpError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {error_string(code)} ({code})")
        self.code = code


_lib = None


def load() -> ctypes.CDLL:
    """Load the shared library; raises if it is missing (no CPU fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} not found: build it with `python -m paper_2505_19578_b200.build` "
            "(there is no CPU fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    P, I, F = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
    T = ctypes.POINTER(SpTensor)
    IP = ctypes.POINTER(ctypes.c_int32)
    lib.sp_ctx_create.argtypes = [ctypes.POINTER(P), I]
    lib.sp_ctx_destroy.argtypes = [P]
    lib.sp_workspace_bytes.argtypes = [ctypes.c_int64, I, I, I, I, I, ctypes.POINTER(ctypes.c_size_t)]
    lib.sp_workspace_bytes_patterns.argtypes = [ctypes.c_int64, I, I, I, I, I, I, ctypes.POINTER(ctypes.c_size_t),
                                                ctypes.POINTER(ctypes.c_size_t)]
    lib.sp_ctx_reserve.argtypes = [P, ctypes.c_size_t]
    lib.sp_get_status.argtypes = [P, ctypes.POINTER(I), ctypes.POINTER(I)]
    lib.sp_strerror.argtypes = [I]
    lib.sp_strerror.restype = ctypes.c_char_p
    lib.sp_dense_pivot_attn.argtypes = [P, T, T, T, IP, I, I, T, P, P, P]
    lib.sp_dense_pivot_attn_fixed_scratch.argtypes = [I, T, T, T, IP, I, I, T, P, P, P]
    lib.sp_fixed_scratch_status.argtypes = [I, IP, IP]
    lib.sp_block_mask_from_importance.argtypes = [P, P, I, I, F, P, P, P, P]
    lib.sp_block_sparse_attn.argtypes = [P, T, T, T, IP, I, IP, P, P, I, I, T, P]
    lib.sp_prefill_attn.argtypes = [P, T, T, T, IP, IP, I, F, I, T, P, P]
    lib.sp_prefill_attn_host.argtypes = [P, P, P, P, I, I, ctypes.c_int64, I, IP, IP, I, F, I, P, P, P]
    lib.sp_pooled_logits.argtypes = [P, T, T, IP, I, I, P, P]
    lib.sp_pattern_from_pooled.argtypes = [P, P, I, I, F, P, P, P, P, P]
    lib.sp_determine_pattern.argtypes = [P, T, T, IP, I, I, P, IP, F, F, P, P, P]
    lib.sp_vertical_slash_pattern.argtypes = [P, T, T, IP, I, F, I, P, P, P, P, P, P]
    lib.sp_prefill_attn_auto.argtypes = [P, T, T, T, IP, IP, I, F, F, F, I, I, T, P, P, P]
    lib.sp_dict_create.argtypes = [P, I, I, ctypes.c_int64, I, ctypes.POINTER(P)]
    lib.sp_dict_destroy.argtypes = [P]
    lib.sp_dict_clear.argtypes = [P]
    lib.sp_dict_count.argtypes = [P]
    lib.sp_prefill_attn_layer.argtypes = [P, P, T, T, T, IP, F, F, F, I, I, T, P, P, P]
    lib.sp_ctx_set_kernel.argtypes = [P, I]
    lib.sp_selftest_wait_timeout.argtypes = [P, ctypes.c_int64, P]
    lib.sp_ctx_set_trace.argtypes = [P, P, I]
    lib.sp_ctx_launch_count.argtypes = [P]
    lib.sp_ctx_launch_count.restype = ctypes.c_int64
    for name in EXPORTS:
        fn = getattr(lib, name)
        if name not in ("sp_strerror", "sp_ctx_launch_count"):
            fn.restype = I
    _lib = lib
    return lib


def error_string(code: int) -> str:
    return load().sp_strerror(code).decode()


def _check(code: int, what: str):
    if code != SP_OK:
        raise SpError(code, what)


def _view(t: torch.Tensor) -> SpTensor:
    if t.dim() == 3:
        t = t.unsqueeze(0)
    if t.dim() != 4 or t.dtype != torch.bfloat16 or not t.is_cuda:
        raise ValueError("expected a CUDA bf16 tensor [heads, seq, dim] or [1, heads, seq, dim]")
    s = SpTensor()
    s.data = t.data_ptr()
    for x in range(4):
        s.shape[x] = t.shape[x]
        # the stride of a size-1 dimension is never used; report 0 for it
        s.stride[x] = t.stride(x) if (t.shape[x] > 1 or x == 3) else 0
    return s


def _i32(xs):
    xs = list(xs)
    return (ctypes.c_int32 * max(len(xs), 1))(*xs)


def _ptr(t):
    return ctypes.c_void_p(t.data_ptr()) if t is not None else None


def _stream(stream):
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


class Context:
    """Owns one sp_ctx (workspace + status word) on one CUDA device."""

    def __init__(self, device: int | None = None, kernel: str = "tc"):
        self._lib = load()
        self.device = torch.cuda.current_device() if device is None else int(device)
        h = ctypes.c_void_p()
        _check(self._lib.sp_ctx_create(ctypes.byref(h), self.device), "sp_ctx_create")
        self._h = h
        self.set_kernel(kernel)

    def close(self):
        if getattr(self, "_h", None):
            self._lib.sp_ctx_destroy(self._h)
            self._h = None

    __del__ = close

    def set_kernel(self, kernel: str):
        _check(self._lib.sp_ctx_set_kernel(self._h, {"tc": 0, "simt": 1, "tc1": 2, "tc_single_head_items": 3}[kernel]), "sp_ctx_set_kernel")

    def set_trace(self, events, events_per_role: int):
        """events: zeroed CUDA int64 tensor of 5 * events_per_role * 2 entries, or None to switch off."""
        _check(self._lib.sp_ctx_set_trace(self._h, _ptr(events), events_per_role if events is not None else 0),
               "sp_ctx_set_trace")

    def selftest_wait_timeout(self, limit_cycles: int, stream=None):
        """Launch the one-warp kernel whose wait cannot complete (see the header); status() then reports the timeout."""
        _check(self._lib.sp_selftest_wait_timeout(self._h, int(limit_cycles), _stream(stream)), "sp_selftest_wait_timeout")

    def launch_count(self) -> int:
        return int(self._lib.sp_ctx_launch_count(self._h))

    def reserve(self, nbytes: int):
        _check(self._lib.sp_ctx_reserve(self._h, nbytes), "sp_ctx_reserve")

    def status(self):
        """(code, where) of the device status word; call after synchronising."""
        c, w = ctypes.c_int(), ctypes.c_int()
        _check(self._lib.sp_get_status(self._h, ctypes.byref(c), ctypes.byref(w)), "sp_get_status")
        return c.value, w.value

    # ---- the four calls -------------------------------------------------

    def sp_dense_pivot_attn(self, q, k, v, heads, block, out, importance_out=None, lse_out=None, stream=None):
        heads = list(heads)
        _check(self._lib.sp_dense_pivot_attn(self._h, _view(q), _view(k), _view(v), _i32(heads), len(heads), block,
                                             _view(out), _ptr(importance_out), _ptr(lse_out), _stream(stream)),
               "sp_dense_pivot_attn")

    def sp_block_mask_from_importance(self, importance, gamma, mask_out, counts_out, indices_out, stream=None):
        n_maps, nb, nb2 = importance.shape
        assert nb == nb2 and importance.dtype == torch.float32 and importance.is_contiguous()
        _check(self._lib.sp_block_mask_from_importance(self._h, _ptr(importance), n_maps, nb, gamma, _ptr(mask_out),
                                                       _ptr(counts_out), _ptr(indices_out), _stream(stream)),
               "sp_block_mask_from_importance")

    def sp_block_sparse_attn(self, q, k, v, heads, list_of_head, counts, indices, block, out, stream=None):
        heads, list_of_head = list(heads), list(list_of_head)
        assert len(heads) == len(list_of_head)
        n_lists = 0 if counts is None else counts.shape[0]
        _check(self._lib.sp_block_sparse_attn(self._h, _view(q), _view(k), _view(v), _i32(heads), len(heads),
                                              _i32(list_of_head), _ptr(counts), _ptr(indices), n_lists, block,
                                              _view(out), _stream(stream)),
               "sp_block_sparse_attn")

    # ---- paper-literal pattern construction and decision -------------------

    def sp_pooled_logits(self, q, k, heads, block, pooled_out, stream=None):
        heads = list(heads)
        assert pooled_out.dtype == torch.float64 and pooled_out.is_contiguous(), "the pooled map is float64"
        _check(self._lib.sp_pooled_logits(self._h, _view(q), _view(k), _i32(heads), len(heads), block, _ptr(pooled_out),
                                          _stream(stream)), "sp_pooled_logits")

    def sp_pattern_from_pooled(self, pooled, gamma, mask_out, counts_out, indices_out, last_row_out=None, stream=None):
        n_maps, nb, nb2 = pooled.shape
        assert nb == nb2 and pooled.dtype == torch.float64 and pooled.is_contiguous(), "the pooled map is float64"
        _check(self._lib.sp_pattern_from_pooled(self._h, _ptr(pooled), n_maps, nb, gamma, _ptr(mask_out), _ptr(counts_out),
                                                _ptr(indices_out), _ptr(last_row_out), _stream(stream)),
               "sp_pattern_from_pooled")

    def sp_determine_pattern(self, q, k, heads, block, pivot_last_rows, row_of_head, delta, tau, pattern_out,
                             dist_out=None, stream=None):
        heads, row_of_head = list(heads), list(row_of_head)
        assert len(heads) == len(row_of_head)
        _check(self._lib.sp_determine_pattern(self._h, _view(q), _view(k), _i32(heads), len(heads), block,
                                              _ptr(pivot_last_rows), _i32(row_of_head), delta, tau, _ptr(pattern_out),
                                              _ptr(dist_out), _stream(stream)), "sp_determine_pattern")

    def sp_vertical_slash_pattern(self, q, k, heads, gamma, block, mask_out, counts_out, indices_out, sel_v_out=None,
                                  sel_s_out=None, stream=None):
        heads = list(heads)
        _check(self._lib.sp_vertical_slash_pattern(self._h, _view(q), _view(k), _i32(heads), len(heads), gamma, block,
                                                   _ptr(mask_out), _ptr(counts_out), _ptr(indices_out), _ptr(sel_v_out),
                                                   _ptr(sel_s_out), _stream(stream)), "sp_vertical_slash_pattern")

    def sp_prefill_attn_auto(self, q, k, v, cluster_map, pivot_heads, gamma, delta, tau, block, out, pooled_construction=False,
                             mask_out=None, pattern_out=None, stream=None):
        cluster_map, pivot_heads = list(cluster_map), list(pivot_heads)
        _check(self._lib.sp_prefill_attn_auto(self._h, _view(q), _view(k), _view(v), _i32(cluster_map), _i32(pivot_heads),
                                              len(pivot_heads), gamma, delta, tau, block, int(bool(pooled_construction)),
                                              _view(out), _ptr(mask_out), _ptr(pattern_out), _stream(stream)),
               "sp_prefill_attn_auto")

    def sp_prefill_attn_host(self, q, k, v, cluster_map, pivot_heads, gamma, block, out, mask_out=None, stream=None):
        """Host tensors (bf16, contiguous, preferably pinned): q, out [Hq, N, d]; k, v [Hkv, N, d]; mask_out u8 [Hq, Nb, Nb]."""
        cluster_map, pivot_heads = list(cluster_map), list(pivot_heads)
        Hq, N, d = q.shape[-3:]
        Hkv = k.shape[-3]
        if tuple(k.shape[-3:]) != (Hkv, N, d) or v.shape != k.shape or out.shape != q.shape:
            raise ValueError("sp_prefill_attn_host: shapes of q, k, v, out do not match")
        bf = torch.bfloat16
        mp = _host_ptr(mask_out, torch.uint8, "mask_out") if mask_out is not None else None
        _check(self._lib.sp_prefill_attn_host(self._h, _host_ptr(q, bf, "q"), _host_ptr(k, bf, "k"), _host_ptr(v, bf, "v"),
                                              Hq, Hkv, N, d, _i32(cluster_map), _i32(pivot_heads), len(pivot_heads),
                                              gamma, block, _host_ptr(out, bf, "out"), mp, _stream(stream)),
               "sp_prefill_attn_host")

    def sp_prefill_attn(self, q, k, v, cluster_map, pivot_heads, gamma, block, out, mask_out=None, stream=None):
        cluster_map, pivot_heads = list(cluster_map), list(pivot_heads)
        _check(self._lib.sp_prefill_attn(self._h, _view(q), _view(k), _view(v), _i32(cluster_map), _i32(pivot_heads),
                                         len(pivot_heads), gamma, block, _view(out), _ptr(mask_out), _stream(stream)),
               "sp_prefill_attn")


class PatternDict:
    """Cross-layer dictionary of pivotal patterns (cluster id -> mask, lists, representative)."""

    def __init__(self, ctx: "Context", max_clusters: int, n_q_heads: int, seq: int, block: int = 128):
        self._lib, self._ctx = load(), ctx
        h = ctypes.c_void_p()
        _check(self._lib.sp_dict_create(ctx._h, max_clusters, n_q_heads, seq, block, ctypes.byref(h)), "sp_dict_create")
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            self._lib.sp_dict_destroy(self._h)
            self._h = None

    __del__ = close

    def clear(self):
        _check(self._lib.sp_dict_clear(self._h), "sp_dict_clear")

    def count(self) -> int:
        return int(self._lib.sp_dict_count(self._h))

    def prefill_attn_layer(self, q, k, v, cluster_of_head, gamma, delta, tau, block, out, pooled_construction=False,
                           mask_out=None, pattern_out=None, stream=None):
        cluster_of_head = list(cluster_of_head)
        _check(self._lib.sp_prefill_attn_layer(self._ctx._h, self._h, _view(q), _view(k), _view(v), _i32(cluster_of_head),
                                               gamma, delta, tau, block, int(bool(pooled_construction)), _view(out),
                                               _ptr(mask_out), _ptr(pattern_out), _stream(stream)), "sp_prefill_attn_layer")


def _host_ptr(t, dtype, what):
    if t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise ValueError(f"{what}: expected a contiguous host tensor of {dtype}")
    return ctypes.c_void_p(t.data_ptr())


def sp_dense_pivot_attn_fixed_scratch(q, k, v, heads, block, out, importance_out=None, lse_out=None, stream=None,
                                      device=None):
    """Dense pivot attention + block importance without any device allocation.

    For hosts that may not allocate when they need attention (an engine plugin's
    enqueue hook, a server whose pool owns the whole device, a latency-critical
    loop): no context, and the per-tile statistics live in a 64 MiB array inside
    the library image instead of a workspace.  Raises SpError(SP_ERR_SCRATCH_LIMIT)
    when n_heads * Nb * (Nb + 1) / 2 * block * 4 bytes exceed that array.  Calls on
    one device share the array: do not let two of them overlap on the GPU.  The
    first call on a device resolves the array's address; make it outside stream
    capture.
    """
    heads = list(heads)
    dev = q.device.index if device is None else int(device)
    _check(load().sp_dense_pivot_attn_fixed_scratch(dev, _view(q), _view(k), _view(v), _i32(heads), len(heads), block,
                                                    _view(out), _ptr(importance_out), _ptr(lse_out), _stream(stream)),
           "sp_dense_pivot_attn_fixed_scratch")


def workspace_bytes_patterns(seq, n_q_heads, n_kv_heads, head_dim, block, n_pivots, pooled_construction=False):
    """(bytes for sp_prefill_attn_auto, bytes for sp_prefill_attn_layer) at this problem size."""
    a, b = ctypes.c_size_t(), ctypes.c_size_t()
    _check(load().sp_workspace_bytes_patterns(seq, n_q_heads, n_kv_heads, head_dim, block, n_pivots,
                                              int(bool(pooled_construction)), ctypes.byref(a), ctypes.byref(b)),
           "sp_workspace_bytes_patterns")
    return a.value, b.value


def pair_work_order(heads, lists, n_q_heads, n_kv_heads, n_row_blocks, n_sm=148, pair_heads=True):
    """Work order of a paired-kernel launch, computed on the host: (items, n_groups), items[raw] = (slot of tile A,
    row-block of tile A, slot of tile B, row-block of tile B).  Touches no device."""
    heads, lists = list(heads), list(lists)
    n_items = len(heads) * ((n_row_blocks + 1) // 2)
    tiles = (ctypes.c_int32 * (4 * n_items))()
    ng = ctypes.c_int()
    _check(load().sp_internal_pair_work_order(_i32(heads), _i32(lists), len(heads), n_q_heads, n_kv_heads, n_row_blocks,
                                              n_sm, int(bool(pair_heads)), tiles, ctypes.byref(ng)),
           "sp_internal_pair_work_order")
    return [tuple(tiles[4 * r:4 * r + 4]) for r in range(n_items)], ng.value


def fixed_scratch_status(device=0):
    """(code, where) of the allocation-free entry point's status word on `device`; clears it when set.

    Synchronise the stream the call was made on first."""
    code, where = ctypes.c_int(), ctypes.c_int()
    _check(load().sp_fixed_scratch_status(int(device), ctypes.byref(code), ctypes.byref(where)), "sp_fixed_scratch_status")
    return code.value, where.value


def workspace_bytes(seq, n_q_heads, n_kv_heads, head_dim, block, n_pivots) -> int:
    out = ctypes.c_size_t()
    _check(load().sp_workspace_bytes(seq, n_q_heads, n_kv_heads, head_dim, block, n_pivots, ctypes.byref(out)),
           "sp_workspace_bytes")
    return out.value
