"""GPU parity of the old-term economy (fl_loop_attention_indexed_carry): while the column sets stay what they were
and the token sets are nested, the old term of the replacement equation (Appendix D.2) is the previous loop's new
term, so a loop can start from the row's background B = O_prev - old term, written once by the last loop that
recomputed the old term, and compute the new term only.  Checked against the oracle (which caches probabilities
literally and knows nothing of this shortcut) and against the recomputing GPU path."""
import dataclasses

import numpy as np
import pytest

from oracle import flashloop_oracle as fo
from paper_2609_29812_b200 import workloads
from helpers import assert_attn_close, storage_round, to_dev, to_np
from test_gpu_parity import oracle_selection, sets_to_arrays, small_bf16

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


@pytest.fixture(scope="module")
def env():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_29812_b200 import binding, pipeline
    ctx = binding.Context(0)
    yield binding, pipeline, ctx
    ctx.close()


def run_oracle(w, x, k_tok=None, c_cols=None):
    n = w.n_loops - 1
    return fo.LayerOracle(w.L, w.n_heads, w.head_dim, w.q_block, w.bits, w.group, w.eps, w.sm_scale,
                          storage=w.dtype).run(x.G, x.Q, x.K, x.V, k_tok or [w.k_tokens] * n,
                                               c_cols or [w.col_budget] * n)


def oracle_background_and_mass(w, rec):
    """B = O^(r) - new term^(r) of the rows active in loop r and their masses, from the oracle's own record of the
    loop: the new term is its cached probabilities times the (storage-rounded) reconstructed V of the selected
    columns.  Returned by position: bg [L, H, dh] (zeros elsewhere), mass [H, L]."""
    act = rec["active"]
    bg = np.zeros((w.L, w.n_heads, w.head_dim))
    mass = np.zeros((w.n_heads, w.L))
    vhat = fo.round_bf16(rec["vhat"]).astype(np.float64) if w.dtype == "bf16" else rec["vhat"].astype(np.float64)
    bg[act] = rec["O_rows"]
    for (h, b), (rows, p_new) in rec["p_new"].items():
        S = np.asarray(rec["col_sets"][(h, b)], dtype=np.int64)
        if len(rows) == 0:
            continue
        if len(S):
            bg[rows, h] -= p_new @ vhat[S, h]
        mass[h, rows] = rec["mass"][(h, b)]
    return bg, mass


CASES = pytest.mark.parametrize("rows,split", [(True, True), (True, False), (False, True)],
                                ids=["materialized_rows+split", "materialized_rows", "rebuilt_in_kernel+split"])


@CASES
def test_chained_economy_against_oracle_and_recomputing_path(env, rows, split):
    """Constant budgets, four loops: loop 2 recomputes and writes the carried buffers, loops 3 and 4 reuse them."""
    B, P, ctx = env
    w = small_bf16(L=2000, H=2, R=4)
    x = workloads.make_layer_inputs(w, seed=21)
    ref = run_oracle(w, x)
    layers = {}
    for mode in ("recompute", "economy"):
        st = P.LayerState(ctx, w, split=split)
        st.dense_loop(to_dev(x.Q[0], w), to_dev(x.K[0], w), to_dev(x.V[0], w))
        st.select_columns_dense()
        outs = []
        for r in range(2, w.n_loops + 1):
            sel = oracle_selection(P, w, ref, r)
            act = ref["active"][r - 2]
            carry = None if mode == "recompute" else ("write" if r == 2 else "reuse")
            # a reusing loop reads only the rows after the loop's residual: one of the cases lends those alone
            rows_r = "cur" if (rows and not split and carry == "reuse") else rows
            o_rows, _ = st.sparse_loop(r, to_dev(x.Q[r - 1][act], w), to_dev(x.K[r - 1][act], w),
                                       to_dev(x.V[r - 1][act], w), sel, indexed=True, carry=carry, rows=rows_r)
            st.check_status()
            outs.append((o_rows.clone(), st.lse.clone(), st.q_store.clone()))
        layers[mode] = (st, outs)
    st_e, outs_e = layers["economy"]
    st_r, outs_r = layers["recompute"]
    if not rows:
        # without materialized rows loop 2 is the fused recomputing kernel in both runs: writing the carried buffers
        # must not change a bit of its output
        for a_, b_ in zip(outs_e[0], outs_r[0]):
            assert torch.equal(a_, b_)
    else:
        # with them the two terms are separate launches: the background is rounded once on its way between them
        assert_attn_close(to_np(outs_e[0][0]), ref["loops"][0]["O_rows"], "two-pass loop 2 O rows", carried=1)
        assert torch.equal(outs_e[0][2], outs_r[0][2])
        ok2 = np.isfinite(ref["loops"][0]["lse_rows"])
        np.testing.assert_allclose(to_np(outs_e[0][1])[:, ref["active"][0]][ok2], ref["loops"][0]["lse_rows"][ok2],
                                   rtol=0, atol=5e-3)
    # the masses it left are the oracle's cached masses
    _, mass_ref = oracle_background_and_mass(w, ref["loops"][0])
    act2 = ref["active"][0]
    np.testing.assert_allclose(to_np(st_e.mass)[:, act2], mass_ref[:, act2], rtol=3e-3, atol=1e-6)
    for r in range(3, w.n_loops + 1):
        rec = ref["loops"][r - 2]
        o_e, lse_e, q_e = outs_e[r - 2]
        o_r, lse_r, q_r = outs_r[r - 2]
        # one storage rounding is carried into an economy loop whatever its number: that of the background
        assert_attn_close(to_np(o_e), rec["O_rows"], f"economy loop {r} O rows", carried=1)
        assert_attn_close(to_np(o_e), to_np(o_r).astype(np.float64), f"economy vs recompute loop {r}", carried=r - 1)
        act = rec["active"]
        ok = np.isfinite(rec["lse_rows"])
        np.testing.assert_allclose(to_np(lse_e)[:, act][ok], rec["lse_rows"][ok], rtol=0, atol=5e-3)
        assert torch.equal(q_e, q_r)
    assert_attn_close(to_np(st_e.o_store), ref["loops"][-1]["O_full"], "economy final O store", carried=1)


@CASES
def test_economy_stage_isolated(env, rows, split):
    """Loops 3 and 4 as reuse calls fed the ORACLE's upstream state: token set, column sets, background rows and
    masses (rounded to storage precision).  The previous Q / O rows and log-normalisers are not passed at all."""
    B, P, ctx = env
    w = small_bf16(L=2000, H=2, R=4)
    x = workloads.make_layer_inputs(w, seed=22)
    ref = run_oracle(w, x)
    st = P.LayerState(ctx, w, split=split)
    st.k_base, st.v_base = to_dev(x.K[0], w), to_dev(x.V[0], w)
    for r in range(2, w.n_loops + 1):
        rec = ref["loops"][r - 2]
        act = rec["active"]
        sel = oracle_selection(P, w, ref, r)
        st.alloc_stream(sel, rows=rows)
        st.quantize(r, to_dev(x.K[r - 1][act], w), to_dev(x.V[r - 1][act], w), sel)
        if r == 2:
            continue
        bg_np, mass_np = oracle_background_and_mass(w, ref["loops"][r - 3])
        bg = to_dev(storage_round(bg_np, w), w)
        mass = torch.from_numpy(mass_np.astype(np.float32)).cuda()
        idx, cnt = sets_to_arrays(w, st.nb, rec["col_sets"], w.col_budget)
        col_idx, col_cnt = torch.from_numpy(idx).cuda(), torch.from_numpy(cnt).cuda()
        o_store = torch.full((w.L, w.n_heads, w.head_dim), 7.0, dtype=torch.bfloat16, device="cuda")
        q_store = torch.zeros_like(o_store)
        lse = torch.zeros(w.n_heads, w.L, dtype=torch.float32, device="cuda")
        csn = torch.zeros(w.n_heads, st.nb, w.col_budget, dtype=torch.float32, device="cuda")
        q_new = to_dev(x.Q[r - 1][act], w)
        B.fl_loop_attention_indexed_carry(ctx, st.shape, r, q_new, None, q_store, sel.active_idx, sel.n, st.store,
                                          col_idx, col_cnt, w.col_budget, None, lse, None, o_store,
                                          B.make_carry(bg, mass, True), csn, status=st.status)
        st.check_status()
        assert_attn_close(to_np(o_store)[act], rec["O_rows"], f"economy stage-isolated loop {r} O rows")
        ok = np.isfinite(rec["lse_rows"])
        np.testing.assert_allclose(to_np(lse)[:, act][ok], rec["lse_rows"][ok], rtol=0, atol=5e-3)
        csn_np = to_np(csn)
        for (h, b), s_ref in rec["col_scores_next"].items():
            np.testing.assert_allclose(csn_np[h, b, : len(s_ref)], s_ref, rtol=2e-2, atol=2e-4)
        # only active rows were written, and the new Q rows are in the Q store
        untouched = np.ones(w.L, dtype=bool); untouched[act] = False
        assert torch.all(o_store[torch.from_numpy(untouched).cuda()] == 7.0)
        assert torch.equal(q_store[sel.active_idx.long()], q_new)


@pytest.mark.parametrize("rows", [True, False], ids=["materialized_rows", "rebuilt_in_kernel"])
def test_economy_with_shrinking_token_sets(env, rows):
    """Token budgets decay, the column budget does not: the sets stay, every row of loop r was active in loop r-1, and
    the selected columns include tokens that were active in an earlier loop only (their payload is stale: rebuilt
    in the kernel whatever `rows` says)."""
    B, P, ctx = env
    w = dataclasses.replace(small_bf16(L=2000, H=2, R=4), changed_fracs=(0.30, 0.15, 0.08))
    x = workloads.make_layer_inputs(w, seed=23)
    k_tok = [500, 240, 120]
    ref = run_oracle(w, x, k_tok=k_tok)
    acts = ref["active"]
    stale = sum(int(np.sum(np.isin(S, acts[0]) & ~np.isin(S, acts[1]))) for S in ref["loops"][1]["col_sets"].values())
    assert stale > 0
    st = P.LayerState(ctx, w)
    st.dense_loop(to_dev(x.Q[0], w), to_dev(x.K[0], w), to_dev(x.V[0], w))
    st.select_columns_dense()
    for r in range(2, w.n_loops + 1):
        rec = ref["loops"][r - 2]
        sel = oracle_selection(P, w, ref, r)
        act = rec["active"]
        o_rows, _ = st.sparse_loop(r, to_dev(x.Q[r - 1][act], w), to_dev(x.K[r - 1][act], w),
                                   to_dev(x.V[r - 1][act], w), sel, indexed=True,
                                   carry="write" if r == 2 else "reuse", rows=rows)
        st.check_status()
        assert_attn_close(to_np(o_rows), rec["O_rows"], f"economy, shrinking tokens, loop {r}", carried=1)
    assert_attn_close(to_np(st.o_store), ref["loops"][-1]["O_full"], "economy, shrinking tokens, final O store",
                      carried=1)


def test_economy_with_logits_far_apart(env):
    """Queries scaled by 16 (logits tens to hundreds of nats apart): both streams of the reuse kernel rescale their
    accumulators, in either half of a chunk, and are merged on a common reference."""
    B, P, ctx = env
    w = small_bf16(L=1500, H=2, R=3)
    x = workloads.make_layer_inputs(w, seed=7)
    x.Q = [workloads.round_to_bf16(q * np.float32(16.0)) for q in x.Q]
    ref = run_oracle(w, x)
    for split in (True, False):
        st = P.LayerState(ctx, w, split=split)
        st.dense_loop(to_dev(x.Q[0], w), to_dev(x.K[0], w), to_dev(x.V[0], w))
        rec2, rec3 = ref["loops"]
        idx, cnt = sets_to_arrays(w, st.nb, rec2["col_sets"], w.col_budget)
        st.col_idx, st.col_cnt, st.c = torch.from_numpy(idx).cuda(), torch.from_numpy(cnt).cuda(), w.col_budget
        for r, rec in ((2, rec2), (3, rec3)):
            sel = oracle_selection(P, w, ref, r)
            act = rec["active"]
            o_rows, _ = st.sparse_loop(r, to_dev(x.Q[r - 1][act], w), to_dev(x.K[r - 1][act], w),
                                       to_dev(x.V[r - 1][act], w), sel, indexed=True,
                                       carry="write" if r == 2 else "reuse")
            st.check_status()
            assert_attn_close(to_np(o_rows), rec["O_rows"], f"economy, far-apart logits, loop {r}", carried=1)


def test_empty_column_sets_and_no_active_rows(env):
    """Rows whose T_i is empty keep their output through a write and a reuse call; a call without active rows is a
    no-op."""
    B, P, ctx = env
    w = small_bf16(L=1200, H=2, R=3)
    x = workloads.make_layer_inputs(w, seed=24)
    ref = run_oracle(w, x)
    st = P.LayerState(ctx, w)
    st.dense_loop(to_dev(x.Q[0], w), to_dev(x.K[0], w), to_dev(x.V[0], w))
    st.select_columns_dense()
    # empty the column set of block 1 for head 0 and make block 2's start beyond its first rows
    st.col_cnt[0, 1] = 0
    st.col_idx[0, 1] = -1
    o1 = st.o_store.clone()
    for r in (2, 3):
        sel = oracle_selection(P, w, ref, r)
        act = ref["active"][r - 2]
        st.sparse_loop(r, to_dev(x.Q[r - 1][act], w), to_dev(x.K[r - 1][act], w), to_dev(x.V[r - 1][act], w), sel,
                       indexed=True, carry="write" if r == 2 else "reuse")
        st.check_status()
        in_b1 = act[(act // w.q_block) == 1]
        assert len(in_b1) > 0
        assert torch.equal(st.o_store[torch.from_numpy(in_b1).cuda(), 0], o1[torch.from_numpy(in_b1).cuda(), 0])
    assert torch.all(st.mass[0, torch.from_numpy(in_b1).cuda()] == 0)
    rc = B.fl_loop_attention_indexed_carry(ctx, st.shape, 3, None, None, None, None, 0, st.store, st.col_idx,
                                           st.col_cnt, st.c, None, st.lse, None, st.o_store,
                                           B.make_carry(st.bg_store, st.mass, True), None, status=st.status)
    assert rc == 0


def test_two_pass_recompute_matches_oracle(env, monkeypatch):
    """FL_TWO_PASS=1 (read when a context is created): a recomputing call with carried buffers runs as an old-term
    launch followed by a new-term launch of the single-term kernel; constant budgets, then shrinking token sets
    (stale columns are rebuilt inside both passes)."""
    B, P, _ = env
    monkeypatch.setenv("FL_TWO_PASS", "1")
    ctx = B.Context(0)
    monkeypatch.delenv("FL_TWO_PASS")
    for seed, k_tok in ((31, None), (32, [500, 240, 120])):
        w = dataclasses.replace(small_bf16(L=2000, H=2, R=4), changed_fracs=(0.30, 0.15, 0.08))
        x = workloads.make_layer_inputs(w, seed=seed)
        ref = run_oracle(w, x, k_tok=k_tok)
        st = P.LayerState(ctx, w)
        st.dense_loop(to_dev(x.Q[0], w), to_dev(x.K[0], w), to_dev(x.V[0], w))
        st.select_columns_dense()
        for r in range(2, w.n_loops + 1):
            rec = ref["loops"][r - 2]
            sel = oracle_selection(P, w, ref, r)
            act = rec["active"]
            # every loop recomputes (two passes each): the old-term pass of loops 3, 4 reads what the new-term pass of
            # the loop before wrote
            o_rows, _ = st.sparse_loop(r, to_dev(x.Q[r - 1][act], w), to_dev(x.K[r - 1][act], w),
                                       to_dev(x.V[r - 1][act], w), sel, indexed=True, carry="write")
            st.check_status()
            assert_attn_close(to_np(o_rows), rec["O_rows"], f"two-pass loop {r} O rows", carried=r)
            ok = np.isfinite(rec["lse_rows"])
            np.testing.assert_allclose(to_np(st.lse)[:, act][ok], rec["lse_rows"][ok], rtol=0, atol=5e-3 * (r - 1))
    ctx.close()
