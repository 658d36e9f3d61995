"""ctypes binding of the CAST C-ABI library (include/cast.h).

Argument marshalling only: every function here has the name and the argument
order of its C counterpart and passes device pointers of torch tensors plus
sizes.  No step of the method runs in Python.  Loading fails loudly when the
CUDA library has not been built; there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libcast_b200.so")

CAST_OK = 0
STATUS_NAMES = {
    0: "OK", 1: "INVALID_ARG", 2: "SHAPE", 3: "CAPACITY", 4: "DTYPE", 5: "COST_TABLE",
    6: "BAD_TREE", 7: "BAD_PAGE", 8: "NONFINITE", 9: "TIMEOUT", 10: "CUDA",
}
CAST_F32, CAST_BF16 = 0, 1
MAX_DEPTH = 16

EXPORTS = [
    "cast_create", "cast_destroy", "cast_status_string", "cast_set_cost_tables", "cast_state_export",
    "cast_state_import", "cast_step_begin", "cast_tree_expand", "cast_select_nodes", "cast_tree_attention",
    "cast_accept", "cast_compact_kv", "cast_poll_status", "cast_step_info", "cast_accept_static",
    "cast_accept_stochastic", "cast_accept_stochastic_plan", "cast_tree_attention_rows", "cast_reserve_attention",
    "cast_set_attention_early_reads",
]


class CastConfig(C.Structure):
    _fields_ = [
        ("C1", C.c_double), ("C2", C.c_double), ("C3", C.c_double),
        ("max_batch", C.c_int32), ("vocab", C.c_int32), ("top_k", C.c_int32), ("max_depth", C.c_int32),
        ("max_width", C.c_int32), ("max_tree", C.c_int32), ("total_token", C.c_int32),
        ("fifo_len", C.c_int32), ("enable_bp", C.c_int32), ("enable_dp", C.c_int32), ("enable_dr", C.c_int32),
        ("pool_mode", C.c_int32), ("ctx_base_mode", C.c_int32), ("rerank_per_row", C.c_int32),
    ]


class CastError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: CAST_ERR_{STATUS_NAMES.get(code, code)}")


_lib = None


def load_library() -> C.CDLL:
    """Loads libcast_b200.so (built in-tree by paper_2510_26577_b200/build.py)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError(
            f"{_LIB_PATH} is missing: build it with `python paper_2510_26577_b200/build.py` "
            "(there is no CPU or PyTorch fallback for the CAST kernels)")
    lib = C.CDLL(_LIB_PATH)
    vp, i32, i32p = C.c_void_p, C.c_int, C.c_void_p
    lib.cast_status_string.restype = C.c_char_p
    lib.cast_status_string.argtypes = [C.c_int]
    sig = {
        "cast_create": [C.POINTER(CastConfig), C.POINTER(vp)],
        "cast_destroy": [vp],
        "cast_set_cost_tables": [vp, i32, i32, i32, i32, vp, vp],
        "cast_state_export": [vp, vp, C.POINTER(C.c_size_t)],
        "cast_state_import": [vp, vp, C.c_size_t],
        "cast_step_begin": [vp, i32, i32p, i32p, vp],
        "cast_tree_expand": [vp, i32, vp, i32, i32p, i32p, i32p, vp],
        "cast_select_nodes": [vp, i32p, i32p, i32p, vp, i32p, vp, i32p, vp],
        "cast_reserve_attention": [vp, i32, i32, i32, i32, i32, i32, i32],
        "cast_set_attention_early_reads": [vp, i32],
        "cast_tree_attention": [vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32p, i32, i32, i32p, vp, i32p,
                                C.c_float, vp, vp],
        "cast_tree_attention_rows": [vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32p, i32, i32, i32p, vp, i32p,
                                     i32p, C.c_float, vp, vp],
        "cast_accept": [vp, vp, i32, i32, i32p, i32p, i32p, vp, i32p, i32p, i32p, i32p, vp],
        "cast_compact_kv": [vp, vp, vp, i32, i32, i32, C.c_size_t, i32, i32, i32, i32p, i32, i32, i32p, i32p, i32p,
                            vp],
        "cast_accept_static": [vp, i32, i32, i32, i32, i32, i32p, i32p, i32p, i32p, i32p, i32p, vp],
        "cast_accept_stochastic": [vp, vp, vp, i32, i32, C.c_double, i32p, i32p, i32p, vp, vp, i32p, i32p, i32p, vp],
        "cast_accept_stochastic_plan": [vp, i32, C.POINTER(C.c_int), C.POINTER(C.c_int)],
        "cast_poll_status": [vp, vp, C.POINTER(C.c_int), C.POINTER(C.c_int32)],
        "cast_step_info": [vp, vp, C.POINTER(C.c_int32)],
    }
    for name, argtypes in sig.items():
        fn = getattr(lib, name)
        fn.restype = C.c_int
        fn.argtypes = argtypes
    _lib = lib
    return lib


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device-resident contiguous tensor expected"
    return t.data_ptr()


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return CAST_F32
    if t.dtype == torch.bfloat16:
        return CAST_BF16
    raise CastError(4, "dtype")


def _stream(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream


def _check(code: int, where: str):
    if code != CAST_OK:
        raise CastError(code, where)


def cast_accept_static(target_logits, B, n_cap, vocab, max_depth, tokens, parent, n_tree, accept_len, accept_path,
                       bonus_token, stream=None):
    """The acceptance step without a context and without any allocation (see include/cast.h): for callers
    that are handed device pointers but may not allocate.  Needs B * n_cap <= 2048."""
    lib = load_library()
    _check(lib.cast_accept_static(_ptr(target_logits), _dtype_code(target_logits), B, n_cap, vocab, max_depth,
                                  _ptr(tokens), _ptr(parent), _ptr(n_tree), _ptr(accept_len), _ptr(accept_path),
                                  _ptr(bonus_token), _stream(stream)), "cast_accept_static")


class CastContext:
    """Owns one cast_ctx.  Methods mirror the C entry points one to one."""

    def __init__(self, *, max_batch, vocab, top_k, max_depth, total_token, max_width=0, max_tree=128,
                 C1=1.0, C2=1.0, C3=1.0, fifo_len=8, enable_bp=0, enable_dp=0, enable_dr=0, pool_mode=0,
                 ctx_base_mode=0, rerank_per_row=0):
        self.lib = load_library()
        self.cfg = CastConfig(C1, C2, C3, max_batch, vocab, top_k, max_depth, max_width, max_tree, total_token,
                              fifo_len, enable_bp, enable_dp, enable_dr, pool_mode, ctx_base_mode, rerank_per_row)
        self.handle = C.c_void_p()
        _check(self.lib.cast_create(C.byref(self.cfg), C.byref(self.handle)), "cast_create")
        self.width = max_width if max_width > 0 else top_k
        self.words = (max_tree + 31) // 32

    def close(self):
        if getattr(self, "handle", None) and self.handle.value:
            self.lib.cast_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # --- host-side set-up ---------------------------------------------------
    def cast_set_cost_tables(self, B, L, M, Ntab, fT, fD):
        import numpy as np
        fT = np.ascontiguousarray(fT, dtype=np.float64)
        fD = np.ascontiguousarray(fD, dtype=np.float64)
        assert fT.size == M * Ntab and fD.size == M * Ntab
        _check(self.lib.cast_set_cost_tables(self.handle, B, L, M, Ntab, fT.ctypes.data, fD.ctypes.data),
               "cast_set_cost_tables")

    def cast_state_export(self) -> bytes:
        n = C.c_size_t(0)
        _check(self.lib.cast_state_export(self.handle, None, C.byref(n)), "cast_state_export")
        buf = C.create_string_buffer(n.value)
        _check(self.lib.cast_state_export(self.handle, buf, C.byref(n)), "cast_state_export")
        return buf.raw[: n.value]

    def cast_state_import(self, blob: bytes):
        _check(self.lib.cast_state_import(self.handle, blob, len(blob)), "cast_state_import")

    def cast_reserve_attention(self, dtype, B, Hq, Hkv, D, page_size, seq_capacity):
        """Sizes the attention workspace for calls of this shape (set-up time; synchronises)."""
        code = CAST_F32 if dtype == torch.float32 else CAST_BF16
        _check(self.lib.cast_reserve_attention(self.handle, code, B, Hq, Hkv, D, page_size, seq_capacity),
               "cast_reserve_attention")

    def cast_set_attention_early_reads(self, promise: bool):
        """The caller's promise that only q and the tree tokens' cache rows come from the operation right before an
        attention call (see include/cast.h)."""
        _check(self.lib.cast_set_attention_early_reads(self.handle, 1 if promise else 0), "cast_set_attention_early_reads")

    # --- compute calls (enqueue only) ----------------------------------------
    def cast_step_begin(self, B, root_token, kv_len, stream=None):
        _check(self.lib.cast_step_begin(self.handle, B, _ptr(root_token), _ptr(kv_len), _stream(stream)),
               "cast_step_begin")

    def cast_tree_expand(self, layer, draft_logits, next_tokens, next_parent_row, next_count, stream=None):
        _check(self.lib.cast_tree_expand(self.handle, layer, _ptr(draft_logits), _dtype_code(draft_logits),
                                         _ptr(next_tokens), _ptr(next_parent_row), _ptr(next_count),
                                         _stream(stream)), "cast_tree_expand")

    def cast_select_nodes(self, tokens, parent, depth, anc_mask, pool_idx, scores, n_tree, stream=None):
        _check(self.lib.cast_select_nodes(self.handle, _ptr(tokens), _ptr(parent), _ptr(depth), _ptr(anc_mask),
                                          _ptr(pool_idx), _ptr(scores), _ptr(n_tree), _stream(stream)),
               "cast_select_nodes")

    def cast_tree_attention(self, q, k_cache, v_cache, B, Hq, Hkv, D, page_size, page_table, seq_capacity,
                            num_pages, kv_len, anc_mask, n_tree, scale, out, stream=None):
        _check(self.lib.cast_tree_attention(self.handle, _ptr(q), _ptr(k_cache), _ptr(v_cache), _dtype_code(q), B, Hq,
                                            Hkv, D, page_size, _ptr(page_table), seq_capacity, num_pages,
                                            _ptr(kv_len), _ptr(anc_mask), _ptr(n_tree), float(scale), _ptr(out),
                                            _stream(stream)), "cast_tree_attention")

    def cast_tree_attention_rows(self, q, k_cache, v_cache, B, Hq, Hkv, D, page_size, page_table, seq_capacity,
                                 num_pages, kv_len, anc_mask, n_tree, first_row, scale, out, stream=None):
        _check(self.lib.cast_tree_attention_rows(self.handle, _ptr(q), _ptr(k_cache), _ptr(v_cache), _dtype_code(q), B,
                                                 Hq, Hkv, D, page_size, _ptr(page_table), seq_capacity, num_pages,
                                                 _ptr(kv_len), _ptr(anc_mask), _ptr(n_tree), _ptr(first_row),
                                                 float(scale), _ptr(out), _stream(stream)), "cast_tree_attention_rows")

    def cast_accept(self, target_logits, B, tokens, parent, depth, anc_mask, n_tree, accept_len, accept_path,
                    bonus_token, stream=None):
        _check(self.lib.cast_accept(self.handle, _ptr(target_logits), _dtype_code(target_logits), B, _ptr(tokens),
                                    _ptr(parent), _ptr(depth), _ptr(anc_mask), _ptr(n_tree), _ptr(accept_len),
                                    _ptr(accept_path), _ptr(bonus_token), _stream(stream)), "cast_accept")

    def cast_accept_stochastic(self, target_logits, draft_logits, B, temperature, tokens, parent, n_tree, u_accept,
                               u_bonus, accept_len, accept_path, bonus_token, stream=None):
        assert draft_logits.dtype == target_logits.dtype and u_accept.dtype == torch.float64 and \
            u_bonus.dtype == torch.float64
        _check(self.lib.cast_accept_stochastic(self.handle, _ptr(target_logits), _ptr(draft_logits),
                                               _dtype_code(target_logits), B, float(temperature), _ptr(tokens),
                                               _ptr(parent), _ptr(n_tree), _ptr(u_accept), _ptr(u_bonus),
                                               _ptr(accept_len), _ptr(accept_path), _ptr(bonus_token),
                                               _stream(stream)), "cast_accept_stochastic")

    def cast_accept_stochastic_plan(self, dtype):
        """(cluster size, slices cached in shared memory?) for logits of torch dtype `dtype`."""
        cs, cached = C.c_int(0), C.c_int(0)
        code = CAST_F32 if dtype == torch.float32 else CAST_BF16
        _check(self.lib.cast_accept_stochastic_plan(self.handle, code, C.byref(cs), C.byref(cached)),
               "cast_accept_stochastic_plan")
        return cs.value, bool(cached.value)

    def cast_compact_kv(self, k_cache, v_cache, B, n_layers, layer_stride_bytes, Hkv, D, page_size, page_table,
                        seq_capacity, num_pages, accept_path, accept_len, kv_len, stream=None):
        _check(self.lib.cast_compact_kv(self.handle, _ptr(k_cache), _ptr(v_cache), _dtype_code(k_cache), B, n_layers,
                                        layer_stride_bytes, Hkv, D, page_size, _ptr(page_table), seq_capacity,
                                        num_pages, _ptr(accept_path), _ptr(accept_len), _ptr(kv_len),
                                        _stream(stream)), "cast_compact_kv")

    # --- synchronising queries ------------------------------------------------
    def cast_poll_status(self, stream=None):
        st, detail = C.c_int(0), C.c_int32(0)
        _check(self.lib.cast_poll_status(self.handle, _stream(stream), C.byref(st), C.byref(detail)),
               "cast_poll_status")
        return st.value, detail.value

    def cast_step_info(self, stream=None):
        H = self.cfg.max_depth
        arr = (C.c_int32 * (4 + MAX_DEPTH))()
        _check(self.lib.cast_step_info(self.handle, _stream(stream), arr), "cast_step_info")
        return {"layers": arr[0], "pool_size": arr[1], "n0": arr[2], "n_tree": arr[3],
                "n_hist": [arr[4 + i] for i in range(H)]}
