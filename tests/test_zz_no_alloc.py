"""fl_loop_attention_indexed_static (the attention entry point whose split workspace is a fixed array of the library's
device image) against fl_loop_attention_indexed with a caller-lent workspace: same inputs, two calls in a row, every
output bit for bit.  Collected last: it is an extra of this implementation, not a step of the method."""
import numpy as np
import pytest

from oracle import flashloop_oracle as fo
from paper_2609_29812_b200 import workloads
from helpers import assert_attn_close, to_dev, to_np
from test_gpu_parity import oracle_selection, small_bf16

pytestmark = pytest.mark.gpu


def _layer(P, ctx, w, x, ref):
    st = P.LayerState(ctx, w)                       # lends the context a workspace: the reference path splits too
    st.dense_loop(to_dev(x.Q[0], w), to_dev(x.K[0], w), to_dev(x.V[0], w))
    st.select_columns_dense()
    return st


def test_static_scratch_entry_point_matches_the_workspace_one_twice_in_a_row():
    import torch
    from paper_2609_29812_b200 import binding as B, pipeline as P
    ctx = B.Context(0)
    # a few dozen problems at most: every one of them is split over two CTAs (a single, partly empty wave)
    w = small_bf16(L=1500, H=4, R=3)
    x = workloads.make_layer_inputs(w, seed=5)
    ref = fo.LayerOracle(w.L, w.n_heads, w.head_dim, w.q_block, w.bits, w.group, w.eps, w.sm_scale,
                         storage=w.dtype).run(x.G, x.Q, x.K, x.V, [w.k_tokens] * 2, [w.col_budget] * 2)
    st = _layer(P, ctx, w, x, ref)
    assert B.fl_loop_attention_workspace_bytes(ctx, st.shape) > 0
    for r in (2, 3):                                 # the two calls in a row: loop 2, then loop 3 on its results
        sel = oracle_selection(P, w, ref, r)
        act = ref["active"][r - 2]
        q_new = to_dev(x.Q[r - 1][act], w)
        st.alloc_stream(sel)
        st.quantize(r, to_dev(x.K[r - 1][act], w), to_dev(x.V[r - 1][act], w), sel)
        q0, o0, lse0 = st.q_store.clone(), st.o_store.clone(), st.lse.clone()
        outs = []
        for fn in (B.fl_loop_attention_indexed, B.fl_loop_attention_indexed_static):
            q, o, lse = q0.clone(), o0.clone(), lse0.clone()
            csn = torch.zeros(w.n_heads, st.nb, st.c, dtype=torch.float32, device="cuda")
            fn(ctx, st.shape, r, q_new, q, q, sel.active_idx, sel.n, st.store, st.col_idx, st.col_cnt, st.c, lse, lse,
               o, o, csn, status=st.status)
            st.check_status()
            outs.append((q, o, lse, csn))
        for got, want, name in zip(outs[1], outs[0], ("Q store", "O store", "lse", "next-loop column scores")):
            assert torch.equal(got, want), (r, name)
        st.q_store, st.o_store, st.lse = outs[1][0], outs[1][1], outs[1][2]
    # and the result is the method's (not merely the same as the other entry point's): two chained loops
    assert_attn_close(to_np(st.o_store), ref["loops"][-1]["O_full"], "final O store", carried=2)
    # a second pass over the same state with the static entry point alone: its counters were left at zero
    q, o, lse = st.q_store.clone(), st.o_store.clone(), st.lse.clone()
    sel = oracle_selection(P, w, ref, 3)
    q_new = to_dev(x.Q[2][ref["active"][1]], w)
    again = []
    for _ in range(2):
        qq, oo, ll = q.clone(), o.clone(), lse.clone()
        B.fl_loop_attention_indexed_static(ctx, st.shape, 3, q_new, qq, qq, sel.active_idx, sel.n, st.store, st.col_idx,
                                           st.col_cnt, st.c, ll, ll, oo, oo, None, status=st.status)
        st.check_status()
        again.append((qq, oo, ll))
    assert all(torch.equal(a, b) for a, b in zip(*again))
    ctx.close()


def test_static_scratch_entry_point_refuses_what_it_cannot_hold():
    """Shapes outside the tensor path get the other entry point's refusal; a null context is an argument error."""
    from paper_2609_29812_b200 import binding as B, pipeline as P
    ctx = B.Context(0)
    w32 = workloads.config1()
    st = P.LayerState(ctx, w32)
    rc = B.lib.fl_loop_attention_indexed_static(None, None, 2, None, None, None, None, 0, None, None, None, 0, None,
                                                None, None, None, None, None, None)
    assert rc == B.FL_ERR_INVALID_ARG
    x = workloads.make_layer_inputs(w32, seed=3)
    st.dense_loop(to_dev(x.Q[0], w32), to_dev(x.K[0], w32), to_dev(x.V[0], w32))
    st.select_columns_dense()
    sel = P.select_tokens(ctx, st.shape, 2, to_dev(x.G[0], w32), to_dev(x.G[1], w32), None, w32.k_tokens)
    act = to_np(sel.active_idx).astype(np.int64)
    st.alloc_stream(sel)
    st.quantize(2, to_dev(x.K[1][act], w32), to_dev(x.V[1][act], w32), sel)
    rc = B.fl_loop_attention_indexed_static(ctx, st.shape, 2, to_dev(x.Q[1][act], w32), st.q_store, st.q_store,
                                            sel.active_idx, sel.n, st.store, st.col_idx, st.col_cnt, st.c, st.lse,
                                            st.lse, st.o_store, st.o_store, None, status=st.status, check=False)
    assert rc == B.FL_ERR_UNSUPPORTED
    ctx.close()
