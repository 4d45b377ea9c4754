"""Budget calibration (Appendix E, "Hyperparameter"): the smallest retention whose relative reconstruction error of
the attention outputs stays below a tolerance (5% in the paper), found once on calibration inputs and then fixed.

Everything here runs through the CUDA library: the candidate budgets are tried with the library's own calls and the
reference they are compared with is the library's dense loop (fl_dense_loop_attention) on the same loop's K/V.  The
calibration inputs are the caller's (the paper samples 128 sequences of a public corpus; here they are the seeded
synthetic workloads)."""
from __future__ import annotations

from typing import Dict, Sequence

import torch

from . import binding as B
from . import pipeline as P
from .workloads import Workload


def _rel_err(a: torch.Tensor, b: torch.Tensor) -> float:
    a, b = a.float(), b.float()
    return float((a - b).norm() / b.norm().clamp_min(1e-30))


def _loop2_outputs(ctx, w: Workload, qkv1, qkv2, g1, g2, k_tokens: int, c: int):
    """O^(2) of the active rows under budgets (k_tokens, c), and the dense attention of loop 2 over the K/V the
    token-sparse update leaves (active rows take their loop-2 K/V, the others keep loop 1's), codec off."""
    w16 = w if w.bits == 16 else Workload(**{**w.__dict__, "bits": 16})
    st = P.LayerState(ctx, w16, qkv1[0].device, c=c)
    st.dense_loop(*qkv1)
    st.select_columns_dense(c)
    sel = P.select_tokens(ctx, st.shape, 2, g1, g2, None, k_tokens)
    idx = sel.active_idx.long()
    o_rows, _ = st.sparse_loop(2, qkv2[0][idx].contiguous(), qkv2[1][idx].contiguous(), qkv2[2][idx].contiguous(), sel)
    st.check_status()
    k_mix, v_mix = qkv1[1].clone(), qkv1[2].clone()
    k_mix[idx], v_mix[idx] = qkv2[1][idx], qkv2[2][idx]
    ref = P.LayerState(ctx, w16, qkv1[0].device)
    ref.dense_loop(qkv2[0], k_mix, v_mix, want_col_scores=False)
    return o_rows, ref.o_store[idx], sel


def calibrate_column_budget(ctx, w: Workload, qkv1, qkv2, g1, g2, k_tokens: int, candidates: Sequence[int],
                            tol: float = 0.05) -> Dict:
    """Smallest column budget of `candidates` whose loop-2 outputs stay within `tol` (relative L2) of dense attention
    over the same K/V.  qkv1 / qkv2: (Q, K, V) of all rows for loops 1 and 2, [L, H, dh] device tensors in storage
    type; g1 / g2: hidden states [L, d].  Returns the chosen budget and the error of every candidate tried."""
    errs = {}
    chosen = None
    for c in sorted(candidates):
        got, want, _ = _loop2_outputs(ctx, w, qkv1, qkv2, g1, g2, k_tokens, c)
        errs[c] = _rel_err(got, want)
        if errs[c] <= tol:
            chosen = c
            break
    return {"budget": chosen, "errors": errs, "tol": tol}


def calibrate_token_budget(ctx, w: Workload, qkv1, qkv2, g1, g2, c: int, candidates: Sequence[int],
                           tol: float = 0.05) -> Dict:
    """Smallest token budget of `candidates` for which the layer's attention output after loop 2, over ALL rows
    (active rows recomputed, the others reused from loop 1), stays within `tol` of recomputing every row."""
    L = w.L
    full, _, _ = _loop2_outputs(ctx, w, qkv1, qkv2, g1, g2, L, c)          # every row active: rows come back in order
    errs = {}
    chosen = None
    for k in sorted(candidates):
        w16 = w if w.bits == 16 else Workload(**{**w.__dict__, "bits": 16})
        st = P.LayerState(ctx, w16, qkv1[0].device, c=c)
        st.dense_loop(*qkv1)
        st.select_columns_dense(c)
        sel = P.select_tokens(ctx, st.shape, 2, g1, g2, None, k)
        idx = sel.active_idx.long()
        st.sparse_loop(2, qkv2[0][idx].contiguous(), qkv2[1][idx].contiguous(), qkv2[2][idx].contiguous(), sel)
        st.check_status()
        errs[k] = _rel_err(st.o_store, full)
        if errs[k] <= tol:
            chosen = k
            break
    return {"budget": chosen, "errors": errs, "tol": tol}
