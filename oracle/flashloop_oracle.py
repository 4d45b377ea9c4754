"""Plain CPU oracle for the FlashLoop loop-r (r > 1) prefill step.

TEST INFRASTRUCTURE ONLY.  This module is the slow, obviously-correct statement of
what the CUDA library must compute.  It shares no code with the CUDA path, imports
nothing from it, and may only be used by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The product path never calls it.

Everything is numpy.  Floating point is fp64, except the residual codec (Eq. 4 of
Section 4.3 and the masked form in Appendix D.3), which is carried out in strict
binary32 with fp16 metadata so that the integer codes have one right answer.

Notation (the paper's, with G^(r) = the hidden state that ENTERS loop r, i.e. the
paper's H^(r-1)):
  L tokens, H heads, dh head dimension, A^(r) active-token set of loop r,
  S[h,b] selected key columns of head h and query block b (a block is q_block
  consecutive token positions), T_i = {j in S[h, block(i)] : j <= i}.

Functions and the passage each one follows:
  token_scores, select_tokens      Appendix D.1 (token selection equation)
  topk_ascending                   the TopK of Appendix D.1 / D.2 with a total order
  dense_loop_attention             Section 3.2 (attention equation) + Appendix D.2 (the
                                   dense-source case: every causal key is a candidate and
                                   the cached mass is one)
  select_columns                   Appendix D.2 (column selection equation)
  sparse_loop_attention            Appendix D.2 (attention replacement equation)
  decode_sparse_attention          Appendix D.2 as written, for decode positions (per-position sets)
  quantize_groups, dequantize_groups, pack_codes, unpack_codes
                                   Appendix E "Quantization Setting" (asymmetric,
                                   group-wise, scale and offset from min / max)
  residual_update                  Section 4.3 / Appendix D.3 (masked residual codec)
  quantize_base, base_q_bytes      Appendix E "Quantization Setting" (the loop-1 base: keys per channel,
                                   values per token, the most recent tokens kept unquantized)
  base_rows_needed                 Appendix D.2 / D.3 (which base rows a layer's sparse loops read)
  project_rows                     Section 4.4 / Appendix G (only the selected token rows pass through
                                   the projections; results return to their positions)
  kv_bytes_per_token_layer         Section 1 (48 GiB example) and Section 4.3 accounting
  LayerOracle                      the steps above in the order of Appendix D

Parity pins live in tests/test_oracle_*.py.  Unpinned: nothing in this file claims
to reproduce the paper's accuracy / perplexity tables (they need trained weights).
"""
from __future__ import annotations

import numpy as np

F64 = np.float64
F32 = np.float32


# --------------------------------------------------------------------------------------
# TopK with a total order (score descending, index ascending), result sorted ascending.
# --------------------------------------------------------------------------------------
def topk_ascending(values: np.ndarray, k: int) -> np.ndarray:
    """Positions (into `values`) of the min(k, n) largest entries.

    Ties go to the lowest position; the result is sorted by ascending position.
    """
    values = np.asarray(values)
    n = values.shape[0]
    k_eff = min(int(k), n)
    if k_eff <= 0:
        return np.zeros(0, dtype=np.int64)
    # lexsort: last key is primary.  Primary = value descending, secondary = position ascending.
    order = np.lexsort((np.arange(n), -values.astype(F64)))
    return np.sort(order[:k_eff]).astype(np.int64)


# --------------------------------------------------------------------------------------
# Appendix D.1: token scores and nested active sets.
# --------------------------------------------------------------------------------------
def token_scores(g_prev: np.ndarray, g_cur: np.ndarray, cand: np.ndarray, eps: float) -> np.ndarray:
    """s_i = ||G_i^(r) - G_i^(r-1)||_2 / (||G_i^(r)||_2 + eps) for i in cand (fp64)."""
    a = np.asarray(g_cur)[cand].astype(F64)
    b = np.asarray(g_prev)[cand].astype(F64)
    num = np.sqrt(np.sum((a - b) ** 2, axis=1))
    den = np.sqrt(np.sum(a ** 2, axis=1)) + F64(eps)
    return num / den


def select_tokens(g_prev, g_cur, cand, k, eps):
    """A^(r) = TopK_k { s_i : i in A^(r-1) }.  Returns (scores[n_cand], active positions ascending)."""
    cand = np.asarray(cand, dtype=np.int64)
    s = token_scores(g_prev, g_cur, cand, eps)
    sel = topk_ascending(s, k)
    return s, cand[sel]


def slot_map(active: np.ndarray, L: int) -> np.ndarray:
    """slot[i] = rank of position i inside the ascending active list, or -1."""
    slot = np.full(L, -1, dtype=np.int32)
    slot[np.asarray(active, dtype=np.int64)] = np.arange(len(active), dtype=np.int32)
    return slot


# --------------------------------------------------------------------------------------
# Section 3.2 attention equation, dense and causal, plus the statistics of a dense
# source loop (Appendix D.2 with m_C = 1).
# --------------------------------------------------------------------------------------
def n_blocks(L: int, q_block: int) -> int:
    return (L + q_block - 1) // q_block


def dense_loop_attention(q, k, v, sm_scale, q_block, rows_to_cache=None, head_list=None, block_list=None):
    """Causal softmax attention of one loop over all L rows, head by head.

    q, k, v: [L, H, dh].  Returns a dict with
      O          [L, H, dh] fp64
      lse        [H, L]     fp64, log of the causal softmax denominator
      col_scores [H, nb, L] fp64, col_scores[h,b,j] = sum_{i in block b, i >= j} p_ij
                 (zero for j beyond the block's last row)
      probs      {(h,b): (rows, P)} only if rows_to_cache is given: P[t, j] = p_{rows[t], j}
                 for the rows of rows_to_cache that fall in block b, all j <= block end.
    head_list / block_list restrict the work to some heads / query blocks (the rest stays zero).
    """
    q = np.asarray(q); k = np.asarray(k); v = np.asarray(v)
    L, H, dh = q.shape
    nb = n_blocks(L, q_block)
    O = np.zeros((L, H, dh), dtype=F64)
    lse = np.zeros((H, L), dtype=F64)
    col_scores = np.zeros((H, nb, L), dtype=F64)
    probs = {}
    heads = range(H) if head_list is None else head_list
    if rows_to_cache is not None:
        rows_to_cache = np.asarray(rows_to_cache, dtype=np.int64)
    for h in heads:
        kh = k[:, h, :].astype(F64)
        vh = v[:, h, :].astype(F64)
        for b in (range(nb) if block_list is None else block_list):
            i0, i1 = b * q_block, min(L, (b + 1) * q_block)
            qi = q[i0:i1, h, :].astype(F64)
            logits = (qi @ kh[:i1].T) * F64(sm_scale)              # [rows, i1]
            causal = np.arange(i1)[None, :] <= np.arange(i0, i1)[:, None]
            logits = np.where(causal, logits, -np.inf)
            mx = logits.max(axis=1, keepdims=True)
            e = np.exp(logits - mx)
            den = e.sum(axis=1, keepdims=True)
            p = e / den
            O[i0:i1, h, :] = p @ vh[:i1]
            lse[h, i0:i1] = (mx + np.log(den))[:, 0]
            col_scores[h, b, :i1] = p.sum(axis=0)
            if rows_to_cache is not None:
                rows = rows_to_cache[(rows_to_cache >= i0) & (rows_to_cache < i1)]
                probs[(h, b)] = (rows, p[rows - i0, :].copy())
    return {"O": O, "lse": lse, "col_scores": col_scores, "probs": probs}


def dense_attention_rows(q, k, v, sm_scale, rows, head):
    """Textbook causal attention for a few query rows of one head (for sampled checks)."""
    q = np.asarray(q); k = np.asarray(k); v = np.asarray(v)
    out = np.zeros((len(rows), q.shape[2]), dtype=F64)
    for t, i in enumerate(rows):
        logit = (k[: i + 1, head, :].astype(F64) @ q[i, head, :].astype(F64)) * F64(sm_scale)
        e = np.exp(logit - logit.max())
        out[t] = (e / e.sum()) @ v[: i + 1, head, :].astype(F64)
    return out


# --------------------------------------------------------------------------------------
# Appendix D.2: column selection.
# --------------------------------------------------------------------------------------
def select_columns(scores: np.ndarray, cand_cols: np.ndarray, c: int) -> np.ndarray:
    """S = TopK_c over the candidate columns; `scores[t]` belongs to column cand_cols[t].

    Returns the selected column ids, ascending.  (1 <= c; c is clipped to |cand|.)
    """
    cand_cols = np.asarray(cand_cols, dtype=np.int64)
    sel = topk_ascending(np.asarray(scores), c)
    return cand_cols[sel]


# --------------------------------------------------------------------------------------
# Appendix E quantizer: asymmetric, group-wise, scale and offset from the group's
# minimum and maximum.  Strict binary32; fp16 metadata.
# --------------------------------------------------------------------------------------
def _half_round_down(x32: np.ndarray) -> np.ndarray:
    """Largest fp16 value <= x (x finite, |x| <= 65504)."""
    h = x32.astype(np.float16)                       # round to nearest even
    up = h.astype(F32) > x32
    h = np.where(up, np.nextafter(h, np.float16(-np.inf)), h)
    return h.astype(np.float16)


def _half_round_up(x32: np.ndarray) -> np.ndarray:
    """Smallest fp16 value >= x (x finite, |x| <= 65504)."""
    h = x32.astype(np.float16)
    dn = h.astype(F32) < x32
    h = np.where(dn, np.nextafter(h, np.float16(np.inf)), h)
    return h.astype(np.float16)


def quantize_groups(delta: np.ndarray, bits: int, group: int):
    """Q of Appendix E on the last axis, split into groups of `group` consecutive elements.

    delta: float32 [..., dh].  Returns (codes uint8 [..., dh], scale fp16 [..., dh/group],
    zero fp16 [..., dh/group]).  The offset is the group minimum rounded DOWN to fp16,
    the scale is (max - offset) / (2^bits - 1) rounded UP to fp16, so the representable
    interval always covers the group and the error is at most half a step.
    """
    assert delta.dtype == F32
    dh = delta.shape[-1]
    assert dh % group == 0
    qmax = F32(2 ** bits - 1)
    d = delta.reshape(delta.shape[:-1] + (dh // group, group))
    mn = d.min(axis=-1)
    mx = d.max(axis=-1)
    zero = _half_round_down(mn)
    zf = zero.astype(F32)
    rng = (mx - zf).astype(F32)                       # binary32 subtraction, >= 0
    ratio = (rng / qmax).astype(F32)                  # binary32 division
    scale = np.where(rng == 0, np.float16(0), _half_round_up(ratio)).astype(np.float16)
    sf = scale.astype(F32)
    safe = np.where(sf == 0, F32(1), sf)
    t = ((d - zf[..., None]).astype(F32) / safe[..., None]).astype(F32)
    code = np.clip(np.rint(t), F32(0), qmax)          # rint = round half to even
    code = np.where(sf[..., None] == 0, F32(0), code)
    codes = code.astype(np.uint8).reshape(delta.shape)
    return codes, scale, zero


def dequantize_groups(codes: np.ndarray, scale: np.ndarray, zero: np.ndarray, group: int) -> np.ndarray:
    """D: code * scale + offset with a single binary32 rounding (code*scale is exact)."""
    dh = codes.shape[-1]
    c = codes.reshape(codes.shape[:-1] + (dh // group, group)).astype(F64)
    val = c * scale.astype(F64)[..., None] + zero.astype(F64)[..., None]   # exact in fp64
    return val.astype(F32).reshape(codes.shape)


def pack_codes(codes: np.ndarray, bits: int) -> np.ndarray:
    """Little-endian packing inside a byte: element (8/bits)*t + u sits at bits [u*bits, (u+1)*bits)."""
    if bits == 8:
        return codes.astype(np.uint8).copy()
    per = 8 // bits
    c = codes.reshape(codes.shape[:-1] + (codes.shape[-1] // per, per)).astype(np.uint16)
    out = np.zeros(c.shape[:-1], dtype=np.uint16)
    for u in range(per):
        out |= c[..., u] << (u * bits)
    return out.astype(np.uint8)


def unpack_codes(packed: np.ndarray, bits: int) -> np.ndarray:
    if bits == 8:
        return packed.astype(np.uint8).copy()
    per = 8 // bits
    mask = (1 << bits) - 1
    out = np.zeros(packed.shape + (per,), dtype=np.uint8)
    for u in range(per):
        out[..., u] = (packed >> (u * bits)) & mask
    return out.reshape(packed.shape[:-1] + (packed.shape[-1] * per,))


def residual_update(x_new_rows, xhat_prev, active, bits, group):
    """Masked residual codec of Appendix D.3 for X in {K, V}.

    x_new_rows: [n, H, dh] the loop-r states of the active rows (storage precision, any float dtype)
    xhat_prev : [L, H, dh] float32, reconstructed state of loop r-1
    active    : [n] ascending positions
    Returns (xhat_new [L,H,dh] float32, payload dict).  Inactive rows are copied unchanged.
    bits == 16 means the codec is off: the new row itself is stored.
    """
    active = np.asarray(active, dtype=np.int64)
    xhat_new = xhat_prev.copy()
    x_new_rows = np.asarray(x_new_rows).astype(F32)
    if bits == 16:
        xhat_new[active] = x_new_rows
        return xhat_new, {"raw": x_new_rows.copy()}
    delta = (x_new_rows - xhat_prev[active]).astype(F32)          # binary32 subtraction
    codes, scale, zero = quantize_groups(delta, bits, group)
    deq = dequantize_groups(codes, scale, zero, group)
    xhat_new[active] = (xhat_prev[active] + deq).astype(F32)      # binary32 addition
    return xhat_new, {"codes": codes, "packed": pack_codes(codes, bits), "scale": scale, "zero": zero}


# --------------------------------------------------------------------------------------
# Appendix E "Quantization Setting", the base states: the same asymmetric min/max quantizer, with the keys
# grouped per channel (a group = `group` consecutive tokens of ONE channel) and the values per token (a group =
# `group` consecutive channels of ONE token); the most recent `tail` tokens stay in the storage type.
# --------------------------------------------------------------------------------------
def quantize_base(k, v, bits, group, tail, storage_round=None):
    """Quantizes the loop-1 K and V of one layer and returns what every later reader sees in their place.

    k, v: [L, H, dh] (or [L, d]) storage-precision values.  Positions [0, Lq), Lq = max(0, L - tail), are
    quantized; the last `tail` positions are kept as they are.  K: for every channel, groups of `group`
    consecutive positions (the last group of the quantized range may be shorter).  V: for every position, groups
    of `group` consecutive channels.  The dequantized value code * scale + offset is formed with one binary32
    rounding and then rounded to the storage type by `storage_round` (None: binary32 storage).
    Returns a dict: khat, vhat [L, d] float32 (the base as read back), k_codes, v_codes uint8 [Lq, d],
    k_scale, k_zero fp16 [ceil(Lq / group), d], v_scale, v_zero fp16 [Lq, d / group], k_tail, v_tail [min(tail, L), d].
    """
    L = k.shape[0]
    k2 = np.asarray(k).reshape(L, -1).astype(F32)
    v2 = np.asarray(v).reshape(L, -1).astype(F32)
    d = k2.shape[1]
    Lq = max(0, L - tail)
    n_tg = (Lq + group - 1) // group
    rnd = storage_round if storage_round is not None else (lambda a: a)
    khat, vhat = k2.copy(), v2.copy()
    k_codes = np.zeros((Lq, d), dtype=np.uint8)
    k_scale = np.zeros((n_tg, d), dtype=np.float16)
    k_zero = np.zeros((n_tg, d), dtype=np.float16)
    for g in range(n_tg):                                   # keys: one group = one channel over up to `group` tokens
        lo, hi = g * group, min(Lq, (g + 1) * group)
        chan_major = np.ascontiguousarray(k2[lo:hi].T)      # [d, tokens of the group]
        c, s, z = quantize_groups(chan_major, bits, hi - lo)
        k_codes[lo:hi] = c.T
        k_scale[g], k_zero[g] = s[:, 0], z[:, 0]
        khat[lo:hi] = rnd(dequantize_groups(c, s, z, hi - lo).T)
    v_codes = np.zeros((Lq, d), dtype=np.uint8)
    v_scale = np.zeros((Lq, d // group), dtype=np.float16)
    v_zero = np.zeros((Lq, d // group), dtype=np.float16)
    if Lq > 0:                                              # values: one group = one token over `group` channels
        v_codes, v_scale, v_zero = quantize_groups(np.ascontiguousarray(v2[:Lq]), bits, group)
        vhat[:Lq] = rnd(dequantize_groups(v_codes, v_scale, v_zero, group))
    return {"khat": khat, "vhat": vhat, "k_codes": k_codes, "k_scale": k_scale, "k_zero": k_zero,
            "v_codes": v_codes, "v_scale": v_scale, "v_zero": v_zero, "k_tail": k2[Lq:].copy(), "v_tail": v2[Lq:].copy()}


def base_rows_needed(col_sets, active, H, L):
    """[H, L] booleans: the base rows of head h that a layer's sparse loops read.  The attention of Appendix D.2
    touches, for head h, only the columns of its blocks' selected sets; the residual codec of Appendix D.3 starts the
    chain of every active position from its base row (all heads)."""
    need = np.zeros((H, L), dtype=bool)
    for (h, _b), S in col_sets.items():
        for j in S:
            need[h, int(j)] = True
    for i in active:
        need[:, int(i)] = True
    return need


def base_q_bytes(L, d, bits, group, tail, elem_bytes=2):
    """Bytes of one layer's quantized base, K and V together: packed codes of the quantized positions, fp16 scale
    and offset per group (keys: per channel and token group; values: per token and channel group), the tail rows."""
    Lq = max(0, L - tail)
    n_tg = (Lq + group - 1) // group
    codes = 2 * Lq * (d * bits // 8)
    meta = 2 * 2 * (n_tg * d) + 2 * 2 * (Lq * (d // group))
    return codes + meta + 2 * (L - Lq) * d * elem_bytes


# --------------------------------------------------------------------------------------
# Appendix D.2: attention replacement for a sparse loop, with literally cached
# previous-loop probabilities.
# --------------------------------------------------------------------------------------
def round_bf16(x: np.ndarray) -> np.ndarray:
    """Nearest bf16 (ties to even) of binary32 values, returned as binary32."""
    x = np.ascontiguousarray(x, dtype=F32)
    u = x.view(np.uint32).astype(np.uint64)
    r = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16) << 16
    return r.astype(np.uint32).view(F32).reshape(x.shape)


def sparse_loop_attention(q_new, khat_new, vhat_new, vhat_old, o_prev, active, col_sets, p_old_cache,
                          sm_scale, q_block, head_list=None, block_list=None, kv_round=None):
    """One sparse loop of Appendix D.2 for every (head, block).

    q_new     : [n, H, dh] queries of the active rows (ascending positions `active`)
    khat_new, vhat_new : [L, H, dh] reconstructed K, V of loop r
    vhat_old  : [L, H, dh] reconstructed V of loop r-1
    o_prev    : [n, H, dh] fp64 previous-loop outputs of the active rows
    col_sets  : {(h,b): ascending column ids S[h,b]}
    p_old_cache : {(h,b): (rows, P)} with P[t, u] = p^(r-1) of query rows[t], column S[h,b][u]
                  (zero where the column is not causal); rows must contain the block's active rows.
    kv_round  : optional rounding applied to the reconstructed K/V rows when attention consumes them.
                The chain Xhat itself stays binary32 (the codec needs it exact); with bf16 storage the
                reconstructed cache that attention reads is a BF16 KV cache (Appendix G, the items on the
                activation type and on the kernels that consume the packed streams without first writing a
                full-precision cache), so its rows are bf16 values: kv_round = round_bf16. None for binary32
                storage.
    Returns dict: O [n,H,dh] fp64, mass {(h,b): m_i per active row}, probs {(h,b): (rows, P_new)},
                  col_scores {(h,b): sum over rows of P_new, per column of S},
                  lse [H, n] fp64: the one-number summary of each row's cached probabilities,
                  p_new_ij = exp(logit_ij - lse_i), i.e. logsumexp_{T_i}(logits) - log m_i (NaN where
                  T_i is empty).  The oracle itself never reads it; tests use it to feed a GPU stage.
    """
    q_new = np.asarray(q_new)
    active = np.asarray(active, dtype=np.int64)
    n, H, dh = q_new.shape
    L = khat_new.shape[0]
    nb = n_blocks(L, q_block)
    O = np.array(o_prev, dtype=F64, copy=True)
    mass, probs, scores = {}, {}, {}
    lse = np.full((H, n), np.nan, dtype=F64)
    heads = range(H) if head_list is None else head_list
    blk = active // q_block
    rd = (lambda x: x) if kv_round is None else kv_round
    for h in heads:
        for b in (range(nb) if block_list is None else block_list):
            t_idx = np.nonzero(blk == b)[0]                      # slots of this block's active rows
            rows = active[t_idx]
            S = np.asarray(col_sets[(h, b)], dtype=np.int64)
            c_rows, P_old_all = p_old_cache[(h, b)]
            if len(rows) == 0 or len(S) == 0:
                mass[(h, b)] = np.zeros(len(rows)); probs[(h, b)] = (rows, np.zeros((len(rows), len(S))))
                scores[(h, b)] = np.zeros(len(S))
                continue
            pos = np.searchsorted(c_rows, rows)
            assert np.all(c_rows[pos] == rows), "cached probabilities must cover the active rows"
            P_old = P_old_all[pos, :]
            assert P_old.shape[1] == len(S)
            causal = S[None, :] <= rows[:, None]                 # T_i membership
            P_old = np.where(causal, P_old, 0.0)
            m = P_old.sum(axis=1)                                # cached global mass, per query
            logits = (q_new[t_idx, h, :].astype(F64) @ rd(khat_new[S, h, :]).astype(F64).T) * F64(sm_scale)
            logits = np.where(causal, logits, -np.inf)
            has = causal.any(axis=1)
            mx = np.where(has, logits.max(axis=1, initial=-np.inf), 0.0)
            e = np.where(causal, np.exp(logits - mx[:, None]), 0.0)
            den = e.sum(axis=1)
            P_new = np.where(has[:, None], m[:, None] * e / np.where(den > 0, den, 1.0)[:, None], 0.0)
            upd = (-P_old @ rd(vhat_old[S, h, :]).astype(F64)) + (P_new @ rd(vhat_new[S, h, :]).astype(F64))
            O[t_idx, h, :] = O[t_idx, h, :] + np.where(has[:, None], upd, 0.0)
            mass[(h, b)] = m
            probs[(h, b)] = (rows, P_new)
            scores[(h, b)] = P_new.sum(axis=0)
            with np.errstate(divide="ignore", invalid="ignore"):
                lse[h, t_idx] = np.where(has, mx + np.log(np.where(den > 0, den, 1.0)) - np.log(m), np.nan)
    return {"O": O, "mass": mass, "probs": probs, "col_scores": scores, "lse": lse}


def decode_sparse_attention(q_new, khat_new, vhat_new, vhat_old, o_prev, col_sets, p_old, sm_scale, kv_round=None):
    """Appendix D.2 literally: one decode position per query, its own selected subset S and cached probabilities.

    q_new  : [B, H, dh] current queries of loop r (decode positions follow every cached key: no causal cut)
    khat_new, vhat_new : [L, H, dh] reconstructed K, V of loop r;  vhat_old : [L, H, dh] reconstructed V of loop r-1
    o_prev : [B, H, dh] fp64 outputs of loop r-1
    col_sets : {(t, h): ascending column ids S};  p_old : {(t, h): cached loop r-1 probabilities over S}
    Returns dict O [B,H,dh] fp64, p_new {(t,h): probabilities over S}, mass [B,H], lse [B,H] with
    p_new_j = exp(logit_j - lse) (NaN for an empty S, whose output row is o_prev unchanged).
    """
    q_new = np.asarray(q_new)
    Bq, H, dh = q_new.shape
    rd = (lambda x: x) if kv_round is None else kv_round
    O = np.array(o_prev, dtype=F64, copy=True)
    mass = np.zeros((Bq, H))
    lse = np.full((Bq, H), np.nan)
    p_out = {}
    for t in range(Bq):
        for h in range(H):
            S = np.asarray(col_sets[(t, h)], dtype=np.int64)
            po = np.asarray(p_old[(t, h)], dtype=F64)
            if len(S) == 0:
                p_out[(t, h)] = np.zeros(0)
                continue
            m = po.sum()                                           # cached global mass of the subset
            logits = (rd(khat_new[S, h, :]).astype(F64) @ q_new[t, h, :].astype(F64)) * F64(sm_scale)
            mx = logits.max()
            e = np.exp(logits - mx)
            pn = m * e / e.sum()                                   # m * softmax over S
            O[t, h, :] = O[t, h, :] - po @ rd(vhat_old[S, h, :]).astype(F64) + pn @ rd(vhat_new[S, h, :]).astype(F64)
            mass[t, h] = m
            with np.errstate(divide="ignore"):
                lse[t, h] = mx + np.log(e.sum()) - np.log(m)
            p_out[(t, h)] = pn
    return {"O": O, "p_new": p_out, "mass": mass, "lse": lse}


def old_term_local_softmax(q_old, khat_old, vhat_old, rows, S, m, sm_scale, head):
    """Section 3.2, sparse-attention-delta equation: m * softmax_S(q^(r-1) K_S^(r-1)T) V_S^(r-1),
    the other way of writing the cached old term (used to cross-check the cache)."""
    S = np.asarray(S, dtype=np.int64)
    out = np.zeros((len(rows), khat_old.shape[2]), dtype=F64)
    for t, i in enumerate(rows):
        T = S[S <= i]
        if len(T) == 0:
            continue
        logit = (khat_old[T, head, :].astype(F64) @ q_old[t].astype(F64)) * F64(sm_scale)
        e = np.exp(logit - logit.max())
        out[t] = m[t] * (e / e.sum()) @ vhat_old[T, head, :].astype(F64)
    return out


# --------------------------------------------------------------------------------------
# Section 4.4 / Appendix G: projections of the active rows only.
# --------------------------------------------------------------------------------------
def project_rows(x, src_idx, w, y, dst_idx, accumulate):
    """y[dst(t), :] (+)= x[src(t), :] @ w.T for t = 0..n-1, in fp64; other rows of y are left as they are.

    src(t) = src_idx[t] (or t when src_idx is None), dst(t) = dst_idx[t] (or t).  w is [d_out, d_in] (the layout
    of a linear layer's weight).  With accumulate the product is added to the row that is there (the residual
    add of the output projection); without, it replaces it.  Returns the new y (fp64); the caller applies the
    storage rounding.
    """
    x = np.asarray(x, dtype=F64)
    w = np.asarray(w, dtype=F64)
    out = np.array(y, dtype=F64, copy=True)
    n = len(src_idx) if src_idx is not None else (len(dst_idx) if dst_idx is not None else x.shape[0])
    for t in range(n):
        s = int(src_idx[t]) if src_idx is not None else t
        d = int(dst_idx[t]) if dst_idx is not None else t
        row = w @ x[s]
        out[d] = out[d] + row if accumulate else row
    return out


# --------------------------------------------------------------------------------------
# KV-cache accounting.
# --------------------------------------------------------------------------------------
def payload_bytes_per_row(d: int, bits: int, group: int, elem_bytes: int = 2) -> int:
    """Bytes one active row adds to one loop's residual stream, K and V together."""
    if bits == 16:
        return 2 * d * elem_bytes
    return 2 * (d * bits // 8 + 2 * 2 * (d // group))           # codes + fp16 scale + fp16 offset


def kv_bytes_per_token_layer(L, d, n_active_per_loop, bits, group, n_layers, elem_bytes=2):
    """(flashloop, dense) KV bytes per token per layer.

    Dense looped cache: one K and one V row per token and per loop (Section 3, first paragraph:
    every loop keeps its own keys and values).  FlashLoop here: bf16 loop-1 base, per-loop payloads for active
    rows only, plus each loop's int32 slot map [L] and index list [n_r], shared by all layers.
    n_active_per_loop lists n_r for r = 2..R.
    """
    R = 1 + len(n_active_per_loop)
    dense = R * 2 * d * elem_bytes
    pay = payload_bytes_per_row(d, bits, group, elem_bytes)
    fl = 2.0 * d * elem_bytes
    for n_r in n_active_per_loop:
        fl += (n_r / L) * pay + 4.0 * (1.0 + n_r / L) / n_layers
    return fl, float(dense)


# --------------------------------------------------------------------------------------
# One layer through all loops, in the order of Appendix D.
# --------------------------------------------------------------------------------------
class LayerOracle:
    """Runs loop 1 densely and loops 2..R with FlashLoop's three mechanisms, for one layer.

    Inputs (all float arrays holding the storage-precision values the GPU also sees):
      G[r-1] : hidden state entering loop r, [L, d]           (token selection only)
      Q[r-1], K[r-1], V[r-1] : per-loop projections of ALL rows, [L, H, dh]; loops r >= 2 read
                               only the rows of A^(r)
    Budgets: k_tokens[r-2], c_cols[r-2] for r = 2..R.
    """

    def __init__(self, L, H, dh, q_block, bits, group, eps, sm_scale, head_list=None, storage="f32"):
        assert storage in ("f32", "bf16")
        self.kv_round = round_bf16 if storage == "bf16" else None
        self.L, self.H, self.dh = L, H, dh
        self.q_block, self.bits, self.group = q_block, bits, group
        self.eps, self.sm_scale = eps, sm_scale
        self.nb = n_blocks(L, q_block)
        self.head_list = list(range(H)) if head_list is None else list(head_list)

    def token_sets(self, G, k_tokens):
        """All A^(r), r = 2..R (they depend on the hidden states only)."""
        cand = np.arange(self.L, dtype=np.int64)
        sets, scores = [], []
        for r in range(2, len(G) + 1):
            s, cand = select_tokens(G[r - 2], G[r - 1], cand, k_tokens[r - 2], self.eps)
            sets.append(cand); scores.append(s)
        return sets, scores

    def run(self, G, Q, K, V, k_tokens, c_cols):
        R = len(Q)
        L, H, nb = self.L, self.H, self.nb
        active_sets, tok_scores = self.token_sets(G, k_tokens)
        out = {"active": active_sets, "token_scores": tok_scores, "loops": []}

        # ---- loop 1: dense source --------------------------------------------------------
        d1 = dense_loop_attention(Q[0], K[0], V[0], self.sm_scale, self.q_block,
                                  rows_to_cache=active_sets[0] if R > 1 else None,
                                  head_list=self.head_list)
        out["dense"] = d1
        if R == 1:
            return out
        col_sets, cache = {}, {}
        for h in self.head_list:
            for b in range(nb):
                end = min(L, (b + 1) * self.q_block)
                S = select_columns(d1["col_scores"][h, b, :end], np.arange(end), c_cols[0])
                rows, P = d1["probs"][(h, b)]
                col_sets[(h, b)] = S
                cache[(h, b)] = (rows, P[:, S])
        khat = np.asarray(K[0]).astype(F32)                      # bf16 base: X^(1) stored as is
        vhat = np.asarray(V[0]).astype(F32)
        o_full = d1["O"]                                         # FlashLoop's running output, all rows

        # ---- loops 2..R -------------------------------------------------------------------
        for r in range(2, R + 1):
            act = active_sets[r - 2]
            khat_new, k_pay = residual_update(np.asarray(K[r - 1])[act], khat, act, self.bits, self.group)
            vhat_new, v_pay = residual_update(np.asarray(V[r - 1])[act], vhat, act, self.bits, self.group)
            o_prev_rows = o_full[act]
            res = sparse_loop_attention(np.asarray(Q[r - 1])[act], khat_new, vhat_new, vhat, o_prev_rows,
                                        act, col_sets, cache, self.sm_scale, self.q_block,
                                        head_list=self.head_list, kv_round=self.kv_round)
            o_full = o_full.copy()
            o_full[act] = res["O"]
            rec = {"r": r, "active": act, "col_sets": dict(col_sets), "k_payload": k_pay, "v_payload": v_pay,
                   "khat": khat_new, "vhat": vhat_new, "khat_old": khat, "vhat_old": vhat,
                   "O_rows": res["O"], "O_full": o_full, "O_prev_rows": o_prev_rows, "lse_rows": res["lse"],
                   "mass": res["mass"], "p_old": cache,
                   "p_new": res["probs"], "col_scores_next": res["col_scores"]}
            out["loops"].append(rec)
            # prepare loop r+1: prune within S with the next budget, keep the matching probabilities
            if r < R:
                nxt_rows = active_sets[r - 1]
                new_sets, new_cache = {}, {}
                for h in self.head_list:
                    for b in range(nb):
                        S = col_sets[(h, b)]
                        rows, P_new = res["probs"][(h, b)]
                        S_next = select_columns(res["col_scores"][(h, b)], S, c_cols[r - 1]) if len(S) else S
                        keep_c = np.searchsorted(S, S_next)
                        keep_r = np.isin(rows, nxt_rows)
                        new_sets[(h, b)] = S_next
                        new_cache[(h, b)] = (rows[keep_r], P_new[np.ix_(keep_r, keep_c)] if len(S) else P_new[keep_r])
                col_sets, cache = new_sets, new_cache
            khat, vhat = khat_new, vhat_new
        return out
