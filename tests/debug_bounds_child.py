"""Child process of test_gpu_debug_bounds.py: runs loop 2 of one small layer through the library named by FLASHLOOP_LIB.

  run      prints a digest of every output (the parent compares the normal and the checked build)
  corrupt  checked build only: hands each call a damaged index array and expects FL_ERR_INVALID_ARG, the code in the
           status word, and untouched outputs.  Refuses to run unless the loaded library says it validates indices:
           the normal build would follow the damaged indices.
"""
import hashlib
import os
import sys

import numpy as np
import torch

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
from paper_2609_29812_b200 import binding as B, pipeline as P, workloads   # noqa: E402
from helpers import to_dev                                                  # noqa: E402
from test_gpu_parity import small_bf16                                      # noqa: E402


def layer(ctx, w, seed):
    x = workloads.make_layer_inputs(w, seed=seed)
    st = P.LayerState(ctx, w)
    st.dense_loop(to_dev(x.Q[0], w), to_dev(x.K[0], w), to_dev(x.V[0], w))
    st.select_columns_dense()
    sel = P.select_tokens(ctx, st.shape, 2, to_dev(x.G[0], w), to_dev(x.G[1], w), None, w.k_tokens)
    act = sel.active_idx.long().cpu().numpy()
    rows = [to_dev(a[1][act], w) for a in (x.Q, x.K, x.V)]
    return x, st, sel, rows


def loop2(ctx, w, st, sel, rows, status):
    st.alloc_stream(sel, rows=True)
    rc = B.fl_quant_kv_residual(ctx, st.shape, 2, rows[1], rows[2], sel.active_idx, sel.n, st.store, status, check=False)
    if rc != B.FL_OK:
        return rc
    if w.dtype == "bf16":
        return B.fl_loop_attention_indexed(ctx, st.shape, 2, rows[0], st.q_store, st.q_store, sel.active_idx, sel.n,
                                           st.store, st.col_idx, st.col_cnt, st.c, st.lse, st.lse, st.o_store,
                                           st.o_store, None, status=status, check=False)
    q_old, o_prev = st.gather(st.q_store, sel), st.gather(st.o_store, sel)
    o_out = torch.empty_like(o_prev)
    rc = B.fl_loop_attention(ctx, st.shape, 2, rows[0], q_old, sel.active_idx, sel.n, st.store, st.col_idx, st.col_cnt,
                             st.c, st.lse, st.lse, o_prev, o_out, None, status=status, check=False)
    st.scatter(o_out, sel, st.o_store)
    return rc


def digest(*tensors):
    h = hashlib.sha256()
    for t in tensors:
        h.update(t.detach().float().cpu().numpy().tobytes() if t.is_floating_point() else t.cpu().numpy().tobytes())
    return h.hexdigest()


def main():
    mode = sys.argv[1]
    ctx = B.Context(0)
    checked = B.lib.fl_debug_bounds_enabled() == 1
    out = []
    for name, w in (("c1", workloads.config1()), ("bf16", small_bf16(L=1200, H=2, R=2))):
        x, st, sel, rows = layer(ctx, w, seed=5)
        status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
        if mode == "run":
            assert loop2(ctx, w, st, sel, rows, status) == B.FL_OK
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            ks = st.k_streams[0]
            out.append(f"{name} {digest(sel.active_idx, st.col_idx, st.col_cnt, ks['codes'], st.o_store, st.lse)}")
            continue
        assert checked, "the corrupt mode needs the checked build"
        L, n = w.L, sel.n

        def expect_refusal(what, call, untouched):
            before = [t.clone() for t in untouched]
            status.zero_()
            rc = call()
            torch.cuda.synchronize()
            assert rc == B.FL_ERR_INVALID_ARG, (name, what, rc)
            assert int(status.item()) == B.FL_ERR_INVALID_ARG, (name, what, "status word")
            for a, b in zip(before, untouched):
                assert torch.equal(a, b), (name, what, "an output was written")

        # 0. a hidden state that is not finite: the token selection must refuse
        g_prev, g_cur = to_dev(x.G[0], w), to_dev(x.G[1], w)
        g_bad = g_cur.clone(); g_bad[7, 3] = float("nan")
        sc = torch.full((L,), 5.0, device="cuda:0")
        ai = torch.full((w.k_tokens,), -9, dtype=torch.int32, device="cuda:0")
        sp = torch.full((L,), -9, dtype=torch.int32, device="cuda:0")
        expect_refusal("hidden state with a NaN",
                       lambda: B.fl_select_tokens(ctx, st.shape, 2, g_prev, g_bad, None, L, w.k_tokens, sc, ai, sp, status,
                                                  check=False), [sc, ai, sp])
        g_bad = g_prev.clone(); g_bad[L - 1, 0] = float("inf")
        expect_refusal("hidden state with an infinity",
                       lambda: B.fl_select_tokens(ctx, st.shape, 2, g_bad, g_cur, None, L, w.k_tokens, sc, ai, sp, status,
                                                  check=False), [sc, ai, sp])
        # 1. an active list that leaves the sequence / is not ascending: the quantizer must refuse
        st.alloc_stream(sel, rows=True)
        ks, vs = st.k_streams[0], st.v_streams[0]
        for t in (ks["codes"], vs["codes"]):
            t.fill_(0xAB)
        for what, pos, val in (("row beyond L", n - 1, L + 7), ("negative row", 0, -3), ("repeated row", 5, None)):
            bad = sel.active_idx.clone()
            bad[pos] = int(bad[pos - 1]) if val is None else val
            expect_refusal(what, lambda: B.fl_quant_kv_residual(ctx, st.shape, 2, rows[1], rows[2], bad, n, st.store,
                                                                status, check=False), [ks["codes"], vs["codes"]])
        assert B.fl_quant_kv_residual(ctx, st.shape, 2, rows[1], rows[2], sel.active_idx, n, st.store, status,
                                      check=False) == B.FL_OK
        # 2. column lists and counts, slot maps: the attention call must refuse
        def attn(col_idx=None, col_cnt=None, store=None):
            ci = st.col_idx if col_idx is None else col_idx
            cc = st.col_cnt if col_cnt is None else col_cnt
            sr = st.store if store is None else store
            if w.dtype == "bf16":
                return B.fl_loop_attention_indexed(ctx, st.shape, 2, rows[0], st.q_store, st.q_store, sel.active_idx, n,
                                                   sr, ci, cc, st.c, st.lse, st.lse, st.o_store, st.o_store, None,
                                                   status=status, check=False)
            return B.fl_loop_attention(ctx, st.shape, 2, rows[0], q_old, sel.active_idx, n, sr, ci, cc, st.c, st.lse,
                                       st.lse, o_prev, o_out, None, status=status, check=False)
        q_old, o_prev = st.gather(st.q_store, sel), st.gather(st.o_store, sel)
        o_out = torch.full_like(o_prev, 7.0)
        outs = [st.o_store, st.lse, st.q_store, o_out]
        ci = st.col_idx.clone(); ci[1, 0, 0] = L
        expect_refusal("column beyond L", lambda: attn(col_idx=ci), outs)
        ci = st.col_idx.clone(); ci[0, -1, 1] = ci[0, -1, 0]
        expect_refusal("columns not ascending", lambda: attn(col_idx=ci), outs)
        cc = st.col_cnt.clone(); cc[0, 0] = st.c + 1
        expect_refusal("count beyond c", lambda: attn(col_cnt=cc), outs)
        slot = sel.slot_of_pos.clone(); slot[3] = n
        bad_k = dict(ks, slot_of_pos=slot)
        expect_refusal("slot beyond the stream's rows",
                       lambda: attn(store=B.make_store(st.k_base, st.v_base, [bad_k], [vs])), outs)
        status.zero_()
        assert attn() == B.FL_OK
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        # 3. row copies and the projection of rows
        dst = torch.full((n, w.d), 3.0, device="cuda:0", dtype=st.q_store.dtype)
        bad = sel.active_idx.clone(); bad[2] = -1
        rc = B.fl_gather_rows(ctx, st.q_store, bad, n, w.d * st.q_store.element_size(), dst, check=False)
        torch.cuda.synchronize()
        assert rc == B.FL_ERR_INVALID_ARG and bool((dst == 3.0).all()), (name, "gather with a negative row")
        if w.dtype == "bf16":
            wt = torch.zeros(64, w.d, device="cuda:0", dtype=torch.bfloat16)
            y = torch.full((n, 64), 3.0, device="cuda:0", dtype=torch.bfloat16)
            bad = sel.active_idx.clone(); bad[n - 1] = L
            expect_refusal("projection row beyond the matrix",
                           lambda: B.fl_project_rows(ctx, st.q_store, L, bad, n, w.d, wt, 64, y, n, None, 0, status,
                                                     check=False), [y])
        out.append(f"{name} refused every damaged input")
    ctx.close()
    print("\n".join(out))


if __name__ == "__main__":
    main()
