"""Thin ctypes binding of libflashloop.so: argument marshalling only, same names as the C ABI.

Every step of the path runs inside the library's CUDA kernels.  PyTorch appears here only as the
owner of device memory and streams: tensor arguments are turned into raw device pointers.
There is no fallback: if the shared library is missing or does not load, importing fails loudly.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("FLASHLOOP_LIB", os.path.join(_PKG, "libflashloop.so"))  # override: a custom build

FL_OK = 0
FL_ERR_INVALID_ARG = -1
FL_ERR_UNSUPPORTED = -2
FL_ERR_WORKSPACE = -3
FL_ERR_CUDA = -4
FL_ERR_TIMEOUT = -5
FL_BF16 = 0
FL_F32 = 1
FL_MAX_LOOPS = 32


class FlKvBaseQ(C.Structure):
    _fields_ = [("k_codes", C.c_void_p), ("k_scale", C.c_void_p), ("k_zero", C.c_void_p),
                ("v_codes", C.c_void_p), ("v_scale", C.c_void_p), ("v_zero", C.c_void_p),
                ("k_tail", C.c_void_p), ("v_tail", C.c_void_p), ("group", C.c_int32), ("tail", C.c_int32)]


class FlShape(C.Structure):
    _fields_ = [("L", C.c_int32), ("n_heads", C.c_int32), ("head_dim", C.c_int32), ("dtype", C.c_int32),
                ("q_block", C.c_int32), ("bits", C.c_int32), ("group", C.c_int32),
                ("eps", C.c_float), ("sm_scale", C.c_float)]


class FlKvStream(C.Structure):
    _fields_ = [("codes", C.c_void_p), ("scale", C.c_void_p), ("zero", C.c_void_p),
                ("slot_of_pos", C.c_void_p), ("rows_prev", C.c_void_p), ("rows_cur", C.c_void_p),
                ("n_rows", C.c_int32), ("reserved_", C.c_int32)]


class FlKvStore(C.Structure):
    _fields_ = [("k_base", C.c_void_p), ("v_base", C.c_void_p),
                ("k_res", FlKvStream * FL_MAX_LOOPS), ("v_res", FlKvStream * FL_MAX_LOOPS),
                ("n_streams", C.c_int32), ("reserved_", C.c_int32)]


class FlAttnCarry(C.Structure):
    _fields_ = [("bg_store", C.c_void_p), ("mass", C.c_void_p), ("reuse", C.c_int32), ("reserved_", C.c_int32)]


class FlashLoopError(RuntimeError):
    def __init__(self, call: str, status: int):
        self.status = status
        super().__init__(f"{call} failed: {status} ({status_string(status)})")


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build the CUDA library first "
            "(python -m paper_2609_29812_b200.build); there is no CPU fallback")
    lib = C.CDLL(LIB_PATH)
    p, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
    sig = {
        "fl_create": [C.POINTER(C.c_void_p), C.c_int],
        "fl_destroy": [p],
        "fl_version": [],
        "fl_debug_bounds_enabled": [],
        "fl_select_tokens": [p, C.POINTER(FlShape), C.c_int, p, p, p, i32, i32, p, p, p, p, p],
        "fl_gather_rows": [p, p, p, i32, i64, p, p],
        "fl_scatter_update": [p, p, p, i32, i64, p, p],
        "fl_project_rows": [p, p, i64, p, i32, i32, p, i32, p, i64, p, i32, p, p],
        "fl_project_qkv_quant": [p, C.POINTER(FlShape), C.c_int, p, i64, p, i32, p, p, p, C.POINTER(FlKvStore), p, p],
        "fl_quant_kv_residual": [p, C.POINTER(FlShape), C.c_int, p, p, p, i32, C.POINTER(FlKvStore), p, p],
        "fl_dense_loop_attention": [p, C.POINTER(FlShape), p, p, p, p, p, p, p, p],
        "fl_select_columns": [p, C.POINTER(FlShape), p, p, p, i32, i32, p, p, p, p],
        "fl_loop_attention": [p, C.POINTER(FlShape), C.c_int, p, p, p, i32, C.POINTER(FlKvStore), p, p, i32,
                              p, p, p, p, p, p, p],
        "fl_loop_attention_indexed": [p, C.POINTER(FlShape), C.c_int, p, p, p, p, i32, C.POINTER(FlKvStore), p, p,
                                      i32, p, p, p, p, p, p, p],
        "fl_loop_attention_indexed_carry": [p, C.POINTER(FlShape), C.c_int, p, p, p, p, i32, C.POINTER(FlKvStore), p, p,
                                            i32, p, p, p, p, C.POINTER(FlAttnCarry), p, p, p],
        "fl_loop_attention_indexed_static": [p, C.POINTER(FlShape), C.c_int, p, p, p, p, i32, C.POINTER(FlKvStore),
                                             p, p, i32, p, p, p, p, p, p, p],
        "fl_decode_attention": [p, C.POINTER(FlShape), C.c_int, p, p, i32, C.POINTER(FlKvStore), p, p, i32, p, p, p, p, p,
                                p, p],
        "fl_quant_kv_base": [p, C.POINTER(FlShape), p, p, C.POINTER(FlKvBaseQ), p, p],
        "fl_dequant_kv_base": [p, C.POINTER(FlShape), C.POINTER(FlKvBaseQ), p, p, p, p, p],
        "fl_mark_base_rows": [p, C.POINTER(FlShape), p, p, i32, p, i32, p, p, p],
        "fl_kv_base_q_bytes": [C.POINTER(FlShape), i32, i32, C.POINTER(i64)],
        "fl_kv_store_bytes": [C.POINTER(FlShape), C.POINTER(FlKvStore), C.c_int, C.c_int,
                              C.POINTER(i64), C.POINTER(i64)],
        "fl_loop_attention_workspace_bytes": [p, C.POINTER(FlShape), C.POINTER(i64)],
        "fl_set_workspace": [p, p, i64, p],
    }
    for name, args in sig.items():
        fn = getattr(lib, name)
        fn.argtypes = args
        fn.restype = C.c_int
    lib.fl_status_string.argtypes = [C.c_int]
    lib.fl_status_string.restype = C.c_char_p
    return lib


lib = _load()


def status_string(status: int) -> str:
    return lib.fl_status_string(int(status)).decode()


def _ptr(x) -> Optional[int]:
    """Device (or host) address of a tensor-like, an int address, or None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    return int(x.data_ptr())


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return int(torch.cuda.current_stream().cuda_stream) or None
    if isinstance(stream, int):
        return stream or None
    return int(stream.cuda_stream) or None


def _check(call: str, rc: int, check: bool) -> int:
    if check and rc != FL_OK:
        raise FlashLoopError(call, rc)
    return rc


def make_shape(L, n_heads, head_dim, dtype, q_block, bits, group, eps, sm_scale) -> FlShape:
    return FlShape(int(L), int(n_heads), int(head_dim), int(dtype), int(q_block), int(bits), int(group),
                   float(eps), float(sm_scale))


def make_store(k_base, v_base, k_streams: Sequence[dict] = (), v_streams: Sequence[dict] = ()) -> FlKvStore:
    """Builds the host-side store struct.  Each stream is a dict with codes, scale, zero, slot_of_pos
    (tensors or addresses), n_rows and optionally rows_prev / rows_cur (the transient workspace for the loop's
    materialized rows).  The caller keeps the tensors alive."""
    st = FlKvStore()
    st.k_base, st.v_base = _ptr(k_base), _ptr(v_base)
    assert len(k_streams) == len(v_streams) <= FL_MAX_LOOPS
    for dst, src in ((st.k_res, k_streams), (st.v_res, v_streams)):
        for i, s in enumerate(src):
            dst[i].codes = _ptr(s.get("codes"))
            dst[i].scale = _ptr(s.get("scale"))
            dst[i].zero = _ptr(s.get("zero"))
            dst[i].slot_of_pos = _ptr(s.get("slot_of_pos"))
            dst[i].rows_prev = _ptr(s.get("rows_prev"))
            dst[i].rows_cur = _ptr(s.get("rows_cur"))
            dst[i].n_rows = int(s["n_rows"])
    st.n_streams = len(k_streams)
    return st


class Context:
    """Owns an fl_ctx.  Use as a context manager or call close()."""

    def __init__(self, device: int = 0):
        h = C.c_void_p()
        _check("fl_create", lib.fl_create(C.byref(h), int(device)), True)
        self.handle = h

    def close(self):
        if self.handle:
            lib.fl_destroy(self.handle)
            self.handle = C.c_void_p()

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def _h(ctx):
    return ctx.handle if isinstance(ctx, Context) else ctx


def fl_select_tokens(ctx, shape, loop_r, h_prev, h_cur, cand, n_cand, k, scores, active_idx, slot_of_pos,
                     status=None, stream=None, check=True) -> int:
    rc = lib.fl_select_tokens(_h(ctx), C.byref(shape), int(loop_r), _ptr(h_prev), _ptr(h_cur), _ptr(cand),
                              int(n_cand), int(k), _ptr(scores), _ptr(active_idx), _ptr(slot_of_pos),
                              _ptr(status), _stream(stream))
    return _check("fl_select_tokens", rc, check)


def fl_loop_attention_workspace_bytes(ctx, shape) -> int:
    out = C.c_int64(0)
    _check("fl_loop_attention_workspace_bytes", lib.fl_loop_attention_workspace_bytes(_h(ctx), C.byref(shape),
                                                                                      C.byref(out)), True)
    return int(out.value)


def fl_set_workspace(ctx, workspace, nbytes, stream=None, check=True) -> int:
    rc = lib.fl_set_workspace(_h(ctx), _ptr(workspace), int(nbytes), _stream(stream))
    return _check("fl_set_workspace", rc, check)


def fl_gather_rows(ctx, src, idx, n, row_bytes, dst, stream=None, check=True) -> int:
    rc = lib.fl_gather_rows(_h(ctx), _ptr(src), _ptr(idx), int(n), int(row_bytes), _ptr(dst), _stream(stream))
    return _check("fl_gather_rows", rc, check)


def fl_scatter_update(ctx, src, idx, n, row_bytes, dst, stream=None, check=True) -> int:
    rc = lib.fl_scatter_update(_h(ctx), _ptr(src), _ptr(idx), int(n), int(row_bytes), _ptr(dst), _stream(stream))
    return _check("fl_scatter_update", rc, check)


def fl_project_rows(ctx, x, x_rows, src_idx, n, d_in, w, d_out, y, y_rows, dst_idx, accumulate, status=None,
                    stream=None, check=True) -> int:
    rc = lib.fl_project_rows(_h(ctx), _ptr(x), int(x_rows), _ptr(src_idx), int(n), int(d_in), _ptr(w), int(d_out),
                             _ptr(y), int(y_rows), _ptr(dst_idx), int(accumulate), _ptr(status), _stream(stream))
    return _check("fl_project_rows", rc, check)


def fl_project_qkv_quant(ctx, shape, loop_r, x, x_rows, active_idx, n_active, w_qkv, q_out, kv_out, store, status=None,
                         stream=None, check=True) -> int:
    rc = lib.fl_project_qkv_quant(_h(ctx), C.byref(shape), int(loop_r), _ptr(x), int(x_rows), _ptr(active_idx),
                                  int(n_active), _ptr(w_qkv), _ptr(q_out), _ptr(kv_out),
                                  C.byref(store) if store is not None else None, _ptr(status), _stream(stream))
    return _check("fl_project_qkv_quant", rc, check)


def make_base_q(k_codes, k_scale, k_zero, v_codes, v_scale, v_zero, k_tail, v_tail, group, tail) -> FlKvBaseQ:
    """Host struct of a quantized base; the tensors (or raw addresses) must outlive every call that uses it."""
    q = FlKvBaseQ()
    for name, t in (("k_codes", k_codes), ("k_scale", k_scale), ("k_zero", k_zero), ("v_codes", v_codes),
                    ("v_scale", v_scale), ("v_zero", v_zero), ("k_tail", k_tail), ("v_tail", v_tail)):
        setattr(q, name, _ptr(t))
    q.group, q.tail = int(group), int(tail)
    return q


def fl_quant_kv_base(ctx, shape, k, v, base, status=None, stream=None, check=True) -> int:
    rc = lib.fl_quant_kv_base(_h(ctx), C.byref(shape), _ptr(k), _ptr(v), C.byref(base) if base is not None else None,
                              _ptr(status), _stream(stream))
    return _check("fl_quant_kv_base", rc, check)


def fl_dequant_kv_base(ctx, shape, base, k_out, v_out, row_mask=None, status=None, stream=None, check=True) -> int:
    rc = lib.fl_dequant_kv_base(_h(ctx), C.byref(shape), C.byref(base) if base is not None else None, _ptr(row_mask),
                                _ptr(k_out), _ptr(v_out), _ptr(status), _stream(stream))
    return _check("fl_dequant_kv_base", rc, check)


def fl_mark_base_rows(ctx, shape, col_idx, col_cnt, c, active_idx, n_active, row_mask, status=None, stream=None,
                      check=True) -> int:
    rc = lib.fl_mark_base_rows(_h(ctx), C.byref(shape), _ptr(col_idx), _ptr(col_cnt), int(c), _ptr(active_idx),
                               int(n_active), _ptr(row_mask), _ptr(status), _stream(stream))
    return _check("fl_mark_base_rows", rc, check)


def fl_kv_base_q_bytes(shape, group, tail) -> int:
    out = C.c_int64()
    _check("fl_kv_base_q_bytes", lib.fl_kv_base_q_bytes(C.byref(shape), int(group), int(tail), C.byref(out)), True)
    return out.value


def fl_quant_kv_residual(ctx, shape, loop_r, k_new, v_new, active_idx, n_active, store, status=None, stream=None,
                         check=True) -> int:
    rc = lib.fl_quant_kv_residual(_h(ctx), C.byref(shape), int(loop_r), _ptr(k_new), _ptr(v_new), _ptr(active_idx),
                                  int(n_active), C.byref(store) if store is not None else None, _ptr(status),
                                  _stream(stream))
    return _check("fl_quant_kv_residual", rc, check)


def fl_dense_loop_attention(ctx, shape, q, k, v, o, lse, col_scores, status=None, stream=None, check=True) -> int:
    rc = lib.fl_dense_loop_attention(_h(ctx), C.byref(shape), _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse),
                                     _ptr(col_scores), _ptr(status), _stream(stream))
    return _check("fl_dense_loop_attention", rc, check)


def fl_select_columns(ctx, shape, col_scores, cand_cols, cand_cnt, n_cand, c, col_idx, col_cnt, status=None,
                      stream=None, check=True) -> int:
    rc = lib.fl_select_columns(_h(ctx), C.byref(shape), _ptr(col_scores), _ptr(cand_cols), _ptr(cand_cnt),
                               int(n_cand), int(c), _ptr(col_idx), _ptr(col_cnt), _ptr(status), _stream(stream))
    return _check("fl_select_columns", rc, check)


def fl_loop_attention(ctx, shape, loop_r, q_new, q_old, active_idx, n_active, store, col_idx, col_cnt, c,
                      lse_prev, lse_out, o_prev, o_out, col_scores_next=None, status=None, stream=None,
                      check=True) -> int:
    rc = lib.fl_loop_attention(_h(ctx), C.byref(shape), int(loop_r), _ptr(q_new), _ptr(q_old), _ptr(active_idx),
                               int(n_active), C.byref(store) if store is not None else None, _ptr(col_idx),
                               _ptr(col_cnt), int(c), _ptr(lse_prev), _ptr(lse_out), _ptr(o_prev), _ptr(o_out),
                               _ptr(col_scores_next), _ptr(status), _stream(stream))
    return _check("fl_loop_attention", rc, check)


def fl_loop_attention_indexed(ctx, shape, loop_r, q_new, q_store_in, q_store_out, active_idx, n_active, store,
                              col_idx, col_cnt, c, lse_in, lse_out, o_store_in, o_store_out, col_scores_next=None,
                              status=None, stream=None, check=True) -> int:
    rc = lib.fl_loop_attention_indexed(_h(ctx), C.byref(shape), int(loop_r), _ptr(q_new), _ptr(q_store_in),
                                       _ptr(q_store_out), _ptr(active_idx), int(n_active),
                                       C.byref(store) if store is not None else None, _ptr(col_idx), _ptr(col_cnt),
                                       int(c), _ptr(lse_in), _ptr(lse_out), _ptr(o_store_in), _ptr(o_store_out),
                                       _ptr(col_scores_next), _ptr(status), _stream(stream))
    return _check("fl_loop_attention_indexed", rc, check)


def make_carry(bg_store, mass, reuse: bool) -> FlAttnCarry:
    """Host struct of the old-term economy: background rows [L, H, dh], mass [H, L], and whether the call reuses
    them (True) or recomputes the old term and writes them (False).  The caller keeps the tensors alive."""
    return FlAttnCarry(_ptr(bg_store), _ptr(mass), 1 if reuse else 0, 0)


def fl_loop_attention_indexed_carry(ctx, shape, loop_r, q_new, q_store_in, q_store_out, active_idx, n_active, store,
                                    col_idx, col_cnt, c, lse_in, lse_out, o_store_in, o_store_out, carry,
                                    col_scores_next=None, status=None, stream=None, check=True) -> int:
    rc = lib.fl_loop_attention_indexed_carry(_h(ctx), C.byref(shape), int(loop_r), _ptr(q_new), _ptr(q_store_in),
                                             _ptr(q_store_out), _ptr(active_idx), int(n_active),
                                             C.byref(store) if store is not None else None, _ptr(col_idx),
                                             _ptr(col_cnt), int(c), _ptr(lse_in), _ptr(lse_out), _ptr(o_store_in),
                                             _ptr(o_store_out), C.byref(carry) if carry is not None else None,
                                             _ptr(col_scores_next), _ptr(status), _stream(stream))
    return _check("fl_loop_attention_indexed_carry", rc, check)


def fl_loop_attention_indexed_static(ctx, shape, loop_r, q_new, q_store_in, q_store_out, active_idx, n_active, store,
                                     col_idx, col_cnt, c, lse_in, lse_out, o_store_in, o_store_out,
                                     col_scores_next=None, status=None, stream=None, check=True) -> int:
    rc = lib.fl_loop_attention_indexed_static(_h(ctx), C.byref(shape), int(loop_r), _ptr(q_new), _ptr(q_store_in),
                                              _ptr(q_store_out), _ptr(active_idx), int(n_active),
                                              C.byref(store) if store is not None else None, _ptr(col_idx),
                                              _ptr(col_cnt), int(c), _ptr(lse_in), _ptr(lse_out), _ptr(o_store_in),
                                              _ptr(o_store_out), _ptr(col_scores_next), _ptr(status), _stream(stream))
    return _check("fl_loop_attention_indexed_static", rc, check)


def fl_decode_attention(ctx, shape, loop_r, q_new, q_old, n_queries, store, col_idx, col_cnt, c, lse_prev, lse_out,
                        o_prev, o_out, p_new_out=None, status=None, stream=None, check=True) -> int:
    rc = lib.fl_decode_attention(_h(ctx), C.byref(shape), int(loop_r), _ptr(q_new), _ptr(q_old), int(n_queries),
                                 C.byref(store) if store is not None else None, _ptr(col_idx), _ptr(col_cnt), int(c),
                                 _ptr(lse_prev), _ptr(lse_out), _ptr(o_prev), _ptr(o_out), _ptr(p_new_out),
                                 _ptr(status), _stream(stream))
    return _check("fl_decode_attention", rc, check)


def fl_kv_store_bytes(shape, store, n_loops, share_layers=1, check=True):
    a, b = C.c_int64(), C.c_int64()
    rc = lib.fl_kv_store_bytes(C.byref(shape), C.byref(store), int(n_loops), int(share_layers), C.byref(a), C.byref(b))
    _check("fl_kv_store_bytes", rc, check)
    return int(a.value), int(b.value)
