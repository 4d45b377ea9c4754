"""Call-order harness for one layer: allocates device buffers with PyTorch and calls the C-ABI
entry points in the order of the hot path.  No arithmetic of the method lives here; every step
runs inside libflashloop's kernels.

Per-layer state carried across loops (all caller-owned device tensors):
  k_base, v_base [L,H,dh]      loop-1 K/V (storage type)
  streams[r-2]                 residual payloads of loop r: codes, scale, zero (K and V)
  q_store, o_store [L,H,dh]    latest Q and attention output of every position
  lse [H,L]                    latest log-normaliser of every (head, position), updated in place
  col_idx [H,nb,c], col_cnt    selected columns per (head, query block)
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional

import torch

from . import binding as B
from .workloads import Workload


def torch_dtype(w: Workload):
    return torch.float32 if w.dtype == "f32" else torch.bfloat16


def fl_dtype(w: Workload) -> int:
    return B.FL_F32 if w.dtype == "f32" else B.FL_BF16


def shape_of(w: Workload, bits: Optional[int] = None, q_block: Optional[int] = None):
    return B.make_shape(w.L, w.n_heads, w.head_dim, fl_dtype(w), q_block or w.q_block, bits or w.bits, w.group,
                        w.eps, w.sm_scale)


@dataclass
class TokenSelection:
    active_idx: torch.Tensor     # int32 [n]
    slot_of_pos: torch.Tensor    # int32 [L]
    scores: torch.Tensor         # f32 [n_cand]
    n: int


def select_tokens(ctx, shape, loop_r, g_prev, g_cur, cand: Optional[torch.Tensor], k: int) -> TokenSelection:
    L = shape.L
    dev = g_cur.device
    n_cand = L if cand is None else int(cand.numel())
    n = min(k, n_cand)
    scores = torch.empty(n_cand, dtype=torch.float32, device=dev)
    active = torch.empty(max(n, 1), dtype=torch.int32, device=dev)
    slot = torch.empty(L, dtype=torch.int32, device=dev)
    B.fl_select_tokens(ctx, shape, loop_r, g_prev, g_cur, cand, n_cand, k, scores, active, slot)
    return TokenSelection(active[:n], slot, scores, n)


_ROWS_WS: dict = {}


def rows_workspace(dev, n: int, d: int):
    """Transient bf16 buffers [n, d] for the materialized rows of one loop: ((K before, K after), (V before,
    V after)).  One set per device, grown on demand and reused by every layer and loop: a loop's rows are dead once
    its attention call has been issued on the stream."""
    key = (str(dev), d)
    ws = _ROWS_WS.get(key)
    if ws is None or ws[0][0].shape[0] < n:
        ws = tuple(tuple(torch.empty(n, d, dtype=torch.bfloat16, device=dev) for _ in range(2)) for _ in range(2))
        _ROWS_WS[key] = ws
    return ws


def lend_workspace(ctx, shape, dev) -> int:
    """Hands the context the workspace with which the attention launch splits the problems of its last, partly empty
    wave over two CTAs each (a scheduling aid; 0 bytes when the shape cannot profit).  The tensor stays referenced
    by the Context object.  Returns the bytes lent."""
    need = B.fl_loop_attention_workspace_bytes(ctx, shape)
    if need > 0:
        ws = getattr(ctx, "_workspace", None)
        if ws is None or ws.numel() < need:
            ws = torch.empty(need, dtype=torch.uint8, device=dev)
        B.fl_set_workspace(ctx, ws, ws.numel())
        ctx._workspace = ws
    return need


class LayerState:
    """Buffers of one layer and the calls that advance it by one loop."""

    def __init__(self, ctx, w: Workload, device="cuda:0", bits: Optional[int] = None, q_block: Optional[int] = None,
                 c: Optional[int] = None, split: bool = True):
        self.ctx, self.w, self.dev = ctx, w, torch.device(device)
        self.shape = shape_of(w, bits, q_block)
        self.bits = self.shape.bits
        self.c = c or w.col_budget
        self.nb = (w.L + self.shape.q_block - 1) // self.shape.q_block
        self.dt = torch_dtype(w)
        if self.dt == torch.bfloat16:
            if split:
                lend_workspace(ctx, self.shape, self.dev)
            else:   # the context's attention launches go back to one CTA per problem
                B.fl_set_workspace(ctx, None, 0)
                ctx._workspace = None
        self.k_streams: List[dict] = []
        self.v_streams: List[dict] = []
        self.col_idx = None
        self.col_cnt = None
        self.col_scores = None
        self.lse = None
        self.store = None
        self.status = torch.zeros(1, dtype=torch.int32, device=self.dev)   # asynchronous device-side errors

    # ---- loop 1 -------------------------------------------------------------------------------
    def dense_loop(self, q, k, v, want_col_scores=True):
        w = self.w
        self.k_base, self.v_base = k, v
        self.q_store = q.clone()
        self.o_store = torch.empty_like(q)
        self.lse = torch.empty(w.n_heads, w.L, dtype=torch.float32, device=self.dev)
        if want_col_scores:
            self.col_scores = torch.empty(w.n_heads, self.nb, w.L, dtype=torch.float32, device=self.dev)
        B.fl_dense_loop_attention(self.ctx, self.shape, q, k, v, self.o_store, self.lse, self.col_scores)
        self._rebuild_store()

    def select_columns_dense(self, c: Optional[int] = None, col_scores=None):
        w = self.w
        c = c or self.c
        self.c = c
        self.col_idx = torch.empty(w.n_heads, self.nb, c, dtype=torch.int32, device=self.dev)
        self.col_cnt = torch.empty(w.n_heads, self.nb, dtype=torch.int32, device=self.dev)
        B.fl_select_columns(self.ctx, self.shape, self.col_scores if col_scores is None else col_scores, None, None,
                            w.L, c, self.col_idx, self.col_cnt)

    def prune_columns(self, col_scores_next, c_next: int):
        """Sparse source loop: keep the c_next best of the current set (Eq. 6, nested selection)."""
        w = self.w
        new_idx = torch.empty(w.n_heads, self.nb, c_next, dtype=torch.int32, device=self.dev)
        new_cnt = torch.empty(w.n_heads, self.nb, dtype=torch.int32, device=self.dev)
        B.fl_select_columns(self.ctx, self.shape, col_scores_next, self.col_idx, self.col_cnt, self.c, c_next,
                            new_idx, new_cnt)
        self.col_idx, self.col_cnt, self.c = new_idx, new_cnt, c_next

    # ---- packed loop-1 base (Appendix E) ------------------------------------------------------
    def pack_base(self, k, v, group: int = 64, tail: int = 64):
        """Packs the loop-1 K and V of the layer (keys per channel over `group` positions, values per token over
        `group` channels, the last `tail` positions unquantized) and keeps only the packed form; returns its bytes."""
        w, L, d = self.w, self.w.L, self.w.d
        Lq = max(0, L - tail)
        n_tg = (Lq + group - 1) // group
        u8 = lambda *s_: torch.empty(s_, dtype=torch.uint8, device=self.dev)
        f16 = lambda *s_: torch.empty(s_, dtype=torch.float16, device=self.dev)
        self.base_tensors = [u8(max(Lq, 1), d * self.bits // 8), f16(max(n_tg, 1), d), f16(max(n_tg, 1), d),
                             u8(max(Lq, 1), d * self.bits // 8), f16(max(Lq, 1), d // group), f16(max(Lq, 1), d // group),
                             torch.empty(max(L - Lq, 1), d, dtype=self.dt, device=self.dev),
                             torch.empty(max(L - Lq, 1), d, dtype=self.dt, device=self.dev)]
        self.base_q = B.make_base_q(*self.base_tensors, group, tail)
        B.fl_quant_kv_base(self.ctx, self.shape, k, v, self.base_q)
        return B.fl_kv_base_q_bytes(self.shape, group, tail)

    def rebuild_base(self, k_out, v_out, sel: Optional["TokenSelection"] = None):
        """Rebuilds the packed base into k_out, v_out ([L, H, dh], e.g. a buffer shared by all layers) and makes them
        the layer's base.  With a token selection (and the layer's column lists) only the rows the sparse loops read."""
        mask = None
        if sel is not None and self.col_idx is not None:
            words = (self.w.L + 31) // 32
            if getattr(self, "row_mask", None) is None:
                self.row_mask = torch.empty(self.w.n_heads, words, dtype=torch.int32, device=self.dev)
            B.fl_mark_base_rows(self.ctx, self.shape, self.col_idx, self.col_cnt, self.c, sel.active_idx, sel.n,
                                self.row_mask)
            mask = self.row_mask
        B.fl_dequant_kv_base(self.ctx, self.shape, self.base_q, k_out, v_out, row_mask=mask)
        self.k_base, self.v_base = k_out, v_out
        self._rebuild_store()

    # ---- loop r >= 2 --------------------------------------------------------------------------
    def _rebuild_store(self):
        self.store = B.make_store(self.k_base, self.v_base, self.k_streams, self.v_streams)

    def alloc_stream(self, sel: TokenSelection, rows: bool = True):
        """Adds the residual stream of the next loop.  rows: also lend it the transient workspace for the loop's
        materialized rows (bf16 storage only), which the quantization kernel fills and the attention kernel of the
        same loop gathers from; the workspace is shared by every LayerState of the device.  rows="cur": only the
        rows after the loop's residual (all a call that reuses the carried old term reads)."""
        w, n = self.w, sel.n
        d = w.d
        ws = rows_workspace(self.dev, n, d) if rows and self.dt == torch.bfloat16 and n > 0 else None

        def one(side):
            st = {"slot_of_pos": sel.slot_of_pos, "n_rows": n}
            if ws is not None:
                st["rows_cur"] = ws[side][1][:n]
                if rows != "cur":    # rows="cur": a loop that reuses the carried old term reads nothing else
                    st["rows_prev"] = ws[side][0][:n]
            if self.bits == 16:
                st.update(codes=torch.empty(max(n, 1), d, dtype=self.dt, device=self.dev), scale=None, zero=None)
            else:
                st.update(codes=torch.empty(max(n, 1), d * self.bits // 8, dtype=torch.uint8, device=self.dev),
                          scale=torch.empty(max(n, 1), d // w.group, dtype=torch.float16, device=self.dev),
                          zero=torch.empty(max(n, 1), d // w.group, dtype=torch.float16, device=self.dev))
            return st
        # every stream of the device points at the same workspace: its content belongs to whichever loop was
        # quantized last, and only that loop's attention call reads it
        self.k_streams.append(one(0))
        self.v_streams.append(one(1))
        self._rebuild_store()

    def quantize(self, loop_r, k_new, v_new, sel: TokenSelection):
        B.fl_quant_kv_residual(self.ctx, self.shape, loop_r, k_new, v_new, sel.active_idx, sel.n, self.store)

    def gather(self, full, sel: TokenSelection, out=None):
        row_bytes = full.shape[1] * full.shape[2] * full.element_size() if full.dim() == 3 else \
            full.shape[1] * full.element_size()
        if out is None:
            out = torch.empty((max(sel.n, 1),) + tuple(full.shape[1:]), dtype=full.dtype, device=self.dev)
        B.fl_gather_rows(self.ctx, full, sel.active_idx, sel.n, row_bytes, out)
        return out

    def scatter(self, rows, sel: TokenSelection, full):
        row_bytes = full.shape[1] * full.shape[2] * full.element_size() if full.dim() == 3 else \
            full.shape[1] * full.element_size()
        B.fl_scatter_update(self.ctx, rows, sel.active_idx, sel.n, row_bytes, full)

    def attention(self, loop_r, q_new, q_old, o_prev, o_out, sel: TokenSelection, col_scores_next=None):
        B.fl_loop_attention(self.ctx, self.shape, loop_r, q_new, q_old, sel.active_idx, sel.n, self.store,
                            self.col_idx, self.col_cnt, self.c, self.lse, self.lse, o_prev, o_out,
                            col_scores_next, status=self.status)   # lse updated in place (active rows only)

    def carry_buffers(self):
        """Buffers of the old-term economy, allocated on first use: background rows [L, H, dh] and mass [H, L]."""
        if getattr(self, "bg_store", None) is None:
            self.bg_store = torch.zeros_like(self.o_store)
            self.mass = torch.zeros(self.w.n_heads, self.w.L, dtype=torch.float32, device=self.dev)
        return self.bg_store, self.mass

    def attention_indexed(self, loop_r, q_new, sel: TokenSelection, col_scores_next=None, check=True,
                          carry: Optional[str] = None) -> int:
        """Same step on the position-indexed Q / O stores, updated in place (no gathers or scatters around it);
        returns the status code, FL_ERR_UNSUPPORTED when the shape is outside the tensor path.
        carry: None (plain call), "write" (recompute the old term and leave background rows and masses for later
        loops) or "reuse" (take the old term from them: valid while the column sets are unchanged and the token sets
        nested)."""
        if carry is None:
            return B.fl_loop_attention_indexed(self.ctx, self.shape, loop_r, q_new, self.q_store, self.q_store,
                                               sel.active_idx, sel.n, self.store, self.col_idx, self.col_cnt, self.c,
                                               self.lse, self.lse, self.o_store, self.o_store, col_scores_next,
                                               status=self.status, check=check)
        bg, mass = self.carry_buffers()
        cs = B.make_carry(bg, mass, carry == "reuse")
        return B.fl_loop_attention_indexed_carry(self.ctx, self.shape, loop_r, q_new, self.q_store, self.q_store,
                                                 sel.active_idx, sel.n, self.store, self.col_idx, self.col_cnt,
                                                 self.c, self.lse, self.lse, self.o_store, self.o_store, cs,
                                                 col_scores_next, status=self.status, check=check)

    def check_status(self):
        """Synchronises and raises if a kernel reported an asynchronous error (e.g. a bounded wait ran out)."""
        code = int(self.status.item())
        if code != 0:
            raise B.FlashLoopError("device status", code)

    def sparse_loop(self, loop_r, q_new, k_new, v_new, sel: TokenSelection, want_col_scores_next=False,
                    indexed=False, carry: Optional[str] = None, rows: bool = True):
        """One loop r >= 2 for this layer: store residuals, gather the carried rows, attend, scatter back
        (indexed=True: one call on the stores instead).  q_new, k_new, v_new: [n, H, dh] rows of the active tokens.
        Returns (o_rows, col_scores_next)."""
        self.alloc_stream(sel, rows=rows)
        self.quantize(loop_r, k_new, v_new, sel)
        if indexed:
            csn = None
            if want_col_scores_next:
                csn = torch.zeros(self.w.n_heads, self.nb, self.c, dtype=torch.float32, device=self.dev)
            self.attention_indexed(loop_r, q_new, sel, csn, carry=carry)
            return self.gather(self.o_store, sel), csn
        q_old = self.gather(self.q_store, sel)
        o_prev = self.gather(self.o_store, sel)
        o_out = torch.empty_like(o_prev)
        csn = None
        if want_col_scores_next:
            csn = torch.zeros(self.w.n_heads, self.nb, self.c, dtype=torch.float32, device=self.dev)
        self.attention(loop_r, q_new, q_old, o_prev, o_out, sel, csn)
        self.scatter(o_out, sel, self.o_store)
        self.scatter(q_new, sel, self.q_store)
        return o_out, csn
