"""GPU parity: every stage of the CUDA path, called through the C ABI, against the CPU oracle on the
same seeded inputs.  Integer results (index sets, codes, fp16 metadata) are compared bit for bit;
attention outputs within relative L2 <= 1e-2 and max-abs <= 3e-2."""
import dataclasses

import numpy as np
import pytest

from oracle import flashloop_oracle as fo
from paper_2609_29812_b200 import workloads
from helpers import (assert_attn_close, assert_selection_matches, storage_round, to_dev, to_np)

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


def small_bf16(L=2000, H=2, R=4, **kw):
    """Config-2-shaped workload shrunk so the oracle runs in seconds; L is not a multiple of the block."""
    w = workloads.config2(L=L, n_heads=H)
    return dataclasses.replace(w, n_loops=R, q_block=kw.pop("q_block", 256), col_budget=kw.pop("c", 160),
                               changed_fracs=w.changed_fracs[: R - 1], **kw)


WORKLOADS = {
    "c1": lambda: workloads.config1(),
    "bf16_small": lambda: small_bf16(),
    "bf16_int8_g64": lambda: small_bf16(L=1200, bits=8, group=64),
    "bf16_int2_g32": lambda: small_bf16(L=1200, bits=2, group=32),
    "bf16_off": lambda: small_bf16(L=1200, bits=16),
    # a point of the depth sweep: 7 loops, so the later loops carry more residual streams (up to 6) than the
    # cooperative build of the attention kernel keeps slot tables for (its patch warps then build every chunk)
    "bf16_R7": lambda: dataclasses.replace(workloads.sweep_point(7, 0.25, 160, 4, L=900), n_heads=2, q_block=256),
}


@pytest.fixture(scope="module", params=list(WORKLOADS))
def case(request):
    w = WORKLOADS[request.param]()
    x = workloads.make_layer_inputs(w, seed=3)
    orc = fo.LayerOracle(w.L, w.n_heads, w.head_dim, w.q_block, w.bits, w.group, w.eps, w.sm_scale,
                         storage=w.dtype)
    ref = orc.run(x.G, x.Q, x.K, x.V, [w.k_tokens] * (w.n_loops - 1), [w.col_budget] * (w.n_loops - 1))
    return w, x, ref


# ------------------------------------------------------------------------------------------------
def test_gather_scatter_bit_exact(env):
    B, P, ctx = env
    g = torch.Generator(device="cpu").manual_seed(0)
    for rows, width, dt in [(1000, 2048, torch.bfloat16), (77, 256, torch.float32), (5, 8, torch.bfloat16)]:
        src = torch.randn(rows, width, generator=g).to(dt).cuda()
        idx = torch.sort(torch.randperm(rows, generator=g)[: max(1, rows // 3)])[0].to(torch.int32).cuda()
        n = idx.numel()
        dst = torch.zeros(n, width, dtype=dt, device="cuda")
        B.fl_gather_rows(ctx, src, idx, n, width * src.element_size(), dst)
        assert torch.equal(dst, src[idx.long()])
        full = torch.full((rows, width), 7.0, dtype=dt, device="cuda")
        B.fl_scatter_update(ctx, dst, idx, n, width * src.element_size(), full)
        expect = torch.full((rows, width), 7.0, dtype=dt, device="cuda")
        expect[idx.long()] = dst
        assert torch.equal(full, expect)
    B.fl_gather_rows(ctx, src, idx, 0, 16, dst)        # empty call is a no-op


def test_token_selection(env, case):
    B, P, ctx = env
    w, x, ref = case
    sh = P.shape_of(w)
    cand = None
    for r in range(2, w.n_loops + 1):
        g_prev, g_cur = to_dev(x.G[r - 2], w), to_dev(x.G[r - 1], w)
        sel = P.select_tokens(ctx, sh, r, g_prev, g_cur, cand, w.k_tokens)
        scores = to_np(sel.scores).astype(np.float64)
        cand_np = np.arange(w.L) if cand is None else to_np(cand).astype(np.int64)
        np.testing.assert_allclose(scores, ref["token_scores"][r - 2], rtol=2e-5, atol=1e-9)
        got = to_np(sel.active_idx).astype(np.int64)
        # exact with respect to its own binary32 scores (total order: score desc, index asc)
        own = cand_np[fo.topk_ascending(to_np(sel.scores), w.k_tokens)]
        assert np.array_equal(got, own)
        # and equal to the independent fp64 oracle except inside a near-tie band
        assert_selection_matches(got, ref["token_scores"][r - 2], cand_np, w.k_tokens, f"tokens loop {r}")
        slot = to_np(sel.slot_of_pos)
        assert np.array_equal(slot, fo.slot_map(got, w.L))
        cand = sel.active_idx


def test_token_selection_ties_and_small_budgets(env):
    B, P, ctx = env
    w = dataclasses.replace(workloads.config1(), L=300)
    sh = P.shape_of(w)
    rng = np.random.default_rng(0)
    g1 = rng.standard_normal((w.L, w.d)).astype(np.float32)
    g2 = g1.copy()
    # rows 10, 20, ..., 290 get the SAME update applied to the SAME base row: exactly equal scores
    g1[10::10] = g1[10]
    g2[10::10] = g1[10] + 0.5
    g2[5] = g1[5] + 3.0                                     # one clear winner
    for k in (1, 2, 7, 30, 299, 300, 1000):
        sel = P.select_tokens(ctx, sh, 2, to_dev(g1, w), to_dev(g2, w), None, k)
        s = to_np(sel.scores)
        assert np.all(s[10::10] == s[10])
        expect = fo.topk_ascending(s, k)
        assert np.array_equal(to_np(sel.active_idx), expect), k
        if 1 < k <= 30:
            assert to_np(sel.active_idx).tolist() == [5] + list(range(10, 10 * k, 10))
    # candidate subset
    cand = torch.tensor([3, 5, 10, 20, 30, 44], dtype=torch.int32, device="cuda")
    sel = P.select_tokens(ctx, sh, 3, to_dev(g1, w), to_dev(g2, w), cand, 3)
    assert to_np(sel.active_idx).tolist() == [5, 10, 20]
    assert to_np(sel.slot_of_pos)[[5, 10, 20, 30]].tolist() == [0, 1, 2, -1]


def build_gpu_layer(env, w, x, ref, upto_loop, use_oracle_sets=True):
    """Runs the GPU path through loop `upto_loop` - 1, feeding oracle token sets (stage isolation)."""
    B, P, ctx = env
    st = P.LayerState(ctx, w)
    st.dense_loop(to_dev(x.Q[0], w), to_dev(x.K[0], w), to_dev(x.V[0], w))
    st.select_columns_dense()
    return st


def oracle_selection(P, w, ref, r):
    act = ref["active"][r - 2]
    return P.TokenSelection(torch.from_numpy(act.astype(np.int32)).cuda(),
                            torch.from_numpy(fo.slot_map(act, w.L)).cuda(), None, len(act))


def test_quantizer_codes_bit_exact_all_loops(env, case):
    B, P, ctx = env
    w, x, ref = case
    st = P.LayerState(ctx, w)
    st.k_base, st.v_base = to_dev(x.K[0], w), to_dev(x.V[0], w)
    for r in range(2, w.n_loops + 1):
        sel = oracle_selection(P, w, ref, r)
        act = ref["active"][r - 2]
        st.alloc_stream(sel)
        st.quantize(r, to_dev(x.K[r - 1][act], w), to_dev(x.V[r - 1][act], w), sel)
        rec = ref["loops"][r - 2]
        for side, streams in (("k_payload", st.k_streams), ("v_payload", st.v_streams)):
            pay, got = rec[side], streams[-1]
            if w.dtype == "bf16":
                # the loop's materialized rows: the oracle's reconstruction before / after the residual, rounded
                # once to bf16 (what the attention of this loop consumes), bit for bit
                hat_old, hat_new = rec[side[0] + "hat_old"], rec[side[0] + "hat"]
                for name, want in (("rows_prev", hat_old), ("rows_cur", hat_new)):
                    got_rows = to_np(got[name]).astype(np.float32).reshape(len(act), w.n_heads, -1)
                    assert np.array_equal(got_rows.view(np.uint32), fo.round_bf16(want[act]).view(np.uint32)), \
                        (r, side, name)
            if w.bits == 16:
                assert np.array_equal(to_np(got["codes"]).reshape(pay["raw"].shape), pay["raw"])
                continue
            n = len(act)
            assert np.array_equal(to_np(got["codes"]).reshape(n, w.n_heads, -1), pay["packed"]), (r, side)
            assert np.array_equal(to_np(got["scale"]).view(np.uint16).reshape(pay["scale"].shape),
                                  pay["scale"].view(np.uint16)), (r, side)
            assert np.array_equal(to_np(got["zero"]).view(np.uint16).reshape(pay["zero"].shape),
                                  pay["zero"].view(np.uint16)), (r, side)


def test_dense_source_loop(env, case):
    B, P, ctx = env
    w, x, ref = case
    st = build_gpu_layer(env, w, x, ref, 2)
    d = ref["dense"]
    assert_attn_close(to_np(st.o_store), d["O"], "dense O")
    np.testing.assert_allclose(to_np(st.lse), d["lse"], rtol=0, atol=2e-4)
    cs = to_np(st.col_scores).astype(np.float64)
    for b in range(st.nb):
        end = min(w.L, (b + 1) * w.q_block)
        np.testing.assert_allclose(cs[:, b, :end], d["col_scores"][:, b, :end], rtol=2e-4, atol=1e-7)
    # column selection: exact on its own scores, near-tie protocol against the oracle's scores
    idx, cnt = to_np(st.col_idx), to_np(st.col_cnt)
    n_diff = 0
    for h in range(w.n_heads):
        for b in range(st.nb):
            end = min(w.L, (b + 1) * w.q_block)
            k = min(w.col_budget, end)
            assert cnt[h, b] == k and np.all(idx[h, b, k:] == -1)
            own = fo.topk_ascending(to_np(st.col_scores)[h, b, :end], k)
            assert np.array_equal(idx[h, b, :k], own)
            n_diff += assert_selection_matches(idx[h, b, :k], d["col_scores"][h, b, :end], np.arange(end), k,
                                               f"columns h{h} b{b}")
    assert n_diff <= 0.01 * w.n_heads * st.nb * w.col_budget


def test_select_columns_on_oracle_scores_is_exact(env, case):
    B, P, ctx = env
    w, x, ref = case
    st = P.LayerState(ctx, w)
    cs32 = ref["dense"]["col_scores"].astype(np.float32)
    st.col_scores = torch.from_numpy(cs32).cuda()
    st.select_columns_dense()
    idx = to_np(st.col_idx)
    for h in range(w.n_heads):
        for b in range(st.nb):
            end = min(w.L, (b + 1) * w.q_block)
            k = min(w.col_budget, end)
            assert np.array_equal(idx[h, b, :k], fo.topk_ascending(cs32[h, b, :end], k))


def sets_to_arrays(w, nb, col_sets, c):
    idx = np.full((w.n_heads, nb, c), -1, dtype=np.int32)
    cnt = np.zeros((w.n_heads, nb), dtype=np.int32)
    for (h, b), S in col_sets.items():
        idx[h, b, : len(S)] = S
        cnt[h, b] = len(S)
    return idx, cnt


# rows: the columns active in the loop come from the rows the quantization kernel materialized, or are rebuilt inside
# the attention kernel; split: the problems of the launch's last wave (here: all of them) go to two CTAs each
ROWS = pytest.mark.parametrize("rows,split", [(True, True), (True, False), (False, True)],
                               ids=["materialized_rows+split", "materialized_rows", "rebuilt_in_kernel+split"])


@ROWS
def test_loop_attention_stage_isolated(env, case, rows, split):
    """Each loop's attention is fed the oracle's upstream state (token set, column sets, previous
    outputs and log-normalisers rounded to storage precision; the store is bit-exact anyway).  rows: the columns
    active in the loop come from the rows the quantization kernel materialized, or (without that workspace) are
    rebuilt from the residual streams inside the attention kernel."""
    w, x, ref = case
    run_stage_isolated(env, w, x, ref, rows, split)


def run_stage_isolated(env, w, x, ref, rows, split):
    B, P, ctx = env
    st = P.LayerState(ctx, w, split=split)
    st.k_base, st.v_base = to_dev(x.K[0], w), to_dev(x.V[0], w)
    lse = ref["dense"]["lse"].astype(np.float32).copy()
    q_prev_full = x.Q[0]
    for r in range(2, w.n_loops + 1):
        rec = ref["loops"][r - 2]
        act = rec["active"]
        sel = oracle_selection(P, w, ref, r)
        st.alloc_stream(sel, rows=rows)
        st.quantize(r, to_dev(x.K[r - 1][act], w), to_dev(x.V[r - 1][act], w), sel)
        idx, cnt = sets_to_arrays(w, st.nb, rec["col_sets"], w.col_budget)
        st.col_idx, st.col_cnt, st.c = torch.from_numpy(idx).cuda(), torch.from_numpy(cnt).cuda(), w.col_budget
        st.lse = torch.from_numpy(lse).cuda()
        o_prev = to_dev(storage_round(rec["O_prev_rows"], w), w)
        o_out = torch.empty_like(o_prev)
        csn = torch.zeros(w.n_heads, st.nb, st.c, dtype=torch.float32, device="cuda")
        st.attention(r, to_dev(x.Q[r - 1][act], w), to_dev(q_prev_full[act], w), o_prev, o_out, sel, csn)
        st.check_status()
        assert_attn_close(to_np(o_out), rec["O_rows"], f"loop {r} O rows")
        # log-normaliser of the active rows and next-loop column scores
        got_lse = to_np(st.lse)[:, act]
        ok = np.isfinite(rec["lse_rows"])
        np.testing.assert_allclose(got_lse[ok], rec["lse_rows"][ok], rtol=0, atol=5e-3)
        csn = to_np(csn)
        for (h, b), s_ref in rec["col_scores_next"].items():
            np.testing.assert_allclose(csn[h, b, : len(s_ref)], s_ref, rtol=2e-2, atol=2e-4)
        # oracle state for the next loop
        lse = lse.copy()
        lse[:, act] = np.where(ok, rec["lse_rows"], lse[:, act]).astype(np.float32)
        q_prev_full = q_prev_full.copy()
        q_prev_full[act] = x.Q[r - 1][act]


@ROWS
def test_loop_attention_with_logits_far_apart(env, rows, split):
    """Queries scaled by 16: ordinary logits spread over tens of nats and those of the heavy key rows over more than a
    hundred, so that for most rows a later half-chunk's maximum beats the running reference of the new term by more
    than the rescale threshold (60 in log2 units = 41.6 nats): the accumulator rows and the half of P already
    written are rescaled, in the first as well as in the second half of a chunk.  One loop, so the old term's
    probabilities stay below one and the outputs O(1)."""
    w = small_bf16(L=1500, H=2, R=2)
    x = workloads.make_layer_inputs(w, seed=7)
    x.Q = [workloads.round_to_bf16(q * np.float32(16.0)) for q in x.Q]
    ref = fo.LayerOracle(w.L, w.n_heads, w.head_dim, w.q_block, w.bits, w.group, w.eps, w.sm_scale,
                         storage=w.dtype).run(x.G, x.Q, x.K, x.V, [w.k_tokens], [w.col_budget])
    # the premise, on the oracle's own sets: new-loop logits of a row against its selected columns
    rec, act = ref["loops"][0], ref["loops"][0]["active"]
    far = total = 0
    for (h, b), S in rec["col_sets"].items():
        rows_b = act[(act // w.q_block) == b]
        if len(S) < 64 or len(rows_b) == 0:
            continue
        s_new = (x.Q[1][rows_b, h].astype(np.float64) @ x.K[1][np.asarray(S), h].astype(np.float64).T) * w.sm_scale
        s_new = np.where(np.asarray(S)[None, :] <= rows_b[:, None], s_new, -np.inf)
        first32 = s_new[:, :32].max(axis=1)
        far += int(np.sum(np.isfinite(first32) & (s_new.max(axis=1) - first32 > 2 * 41.6)))
        total += len(rows_b)
    assert far > total // 4, (far, total)
    run_stage_isolated(env, w, x, ref, rows, split)


def test_chained_layer_all_on_gpu(env, case):
    """Everything on the GPU, loop after loop; only the final comparison uses the oracle."""
    B, P, ctx = env
    w, x, ref = case
    st = build_gpu_layer(env, w, x, ref, 2)
    sh = st.shape
    cand = None
    for r in range(2, w.n_loops + 1):
        sel = P.select_tokens(ctx, sh, r, to_dev(x.G[r - 2], w), to_dev(x.G[r - 1], w), cand, w.k_tokens)
        act = to_np(sel.active_idx).astype(np.int64)
        o_rows, _ = st.sparse_loop(r, to_dev(x.Q[r - 1][act], w), to_dev(x.K[r - 1][act], w),
                                   to_dev(x.V[r - 1][act], w), sel)
        cand = sel.active_idx
        st.check_status()
        # The GPU carries O between loops in storage precision (the oracle carries fp64): the output entering
        # loop r has been rounded r - 1 times on the GPU side only (loops 1 .. r-1), each by up to half a storage
        # ulp, on top of this loop's own error; the relative L2 bound is kept as stated.
        if np.array_equal(act, ref["active"][r - 2]):
            assert_attn_close(to_np(o_rows), ref["loops"][r - 2]["O_rows"], f"chained loop {r}", carried=r - 1,
                              bf16=w.dtype == "bf16")
    assert_attn_close(to_np(st.o_store), ref["loops"][-1]["O_full"], "chained final O store", carried=w.n_loops - 1,
                      bf16=w.dtype == "bf16")
    # KV accounting of the real store
    fl, dense = B.fl_kv_store_bytes(sh, st.store, w.n_loops, 1)
    n_r = [len(a) for a in ref["active"]]
    fl_ref, dense_ref = fo.kv_bytes_per_token_layer(w.L, w.d, n_r, w.bits, w.group, 1,
                                                    elem_bytes=4 if w.dtype == "f32" else 2)
    assert dense == dense_ref * w.L and abs(fl - fl_ref * w.L) <= 4 * w.n_loops


def test_indexed_attention_matches_compact_path_and_oracle(env):
    """fl_loop_attention_indexed on the position-indexed stores (updated in place): same rows as gather -> fl_loop_attention ->
    scatter (bit for bit: the same kernel arithmetic), and the oracle's within the stated tolerance; the Q store
    ends up holding the new rows, inactive rows stay untouched."""
    import torch
    B, P, ctx = env
    w = small_bf16(L=1500, H=2, R=3)
    x = workloads.make_layer_inputs(w, seed=11)
    ref = fo.LayerOracle(w.L, w.n_heads, w.head_dim, w.q_block, w.bits, w.group, w.eps, w.sm_scale,
                         storage=w.dtype).run(x.G, x.Q, x.K, x.V, [w.k_tokens] * 2, [w.col_budget] * 2)
    states = []
    for indexed in (False, True):
        st = P.LayerState(ctx, w)
        st.dense_loop(to_dev(x.Q[0], w), to_dev(x.K[0], w), to_dev(x.V[0], w))
        st.select_columns_dense()
        q0 = st.q_store.clone()
        for r in (2, 3):
            sel = oracle_selection(P, w, ref, r)
            act = ref["active"][r - 2]
            st.sparse_loop(r, to_dev(x.Q[r - 1][act], w), to_dev(x.K[r - 1][act], w), to_dev(x.V[r - 1][act], w),
                           sel, indexed=indexed)
            st.check_status()
        states.append((st, q0))
    (a, _), (b, q0) = states
    assert torch.equal(a.o_store, b.o_store)
    assert torch.equal(a.q_store, b.q_store)
    assert torch.equal(a.lse, b.lse)
    assert_attn_close(to_np(b.o_store), ref["loops"][-1]["O_full"], "indexed final O store", carried=2)
    touched = np.zeros(w.L, dtype=bool)
    touched[ref["active"][0]] = True
    assert torch.equal(b.q_store[torch.from_numpy(~touched).to(b.q_store.device)],
                       q0[torch.from_numpy(~touched).to(q0.device)])
    # shapes outside the tensor path are refused before anything is launched
    w32 = workloads.config1()
    x32 = workloads.make_layer_inputs(w32, seed=3)
    st32 = P.LayerState(ctx, w32)
    st32.dense_loop(to_dev(x32.Q[0], w32), to_dev(x32.K[0], w32), to_dev(x32.V[0], w32))
    st32.select_columns_dense()
    sel = P.select_tokens(ctx, st32.shape, 2, to_dev(x32.G[0], w32), to_dev(x32.G[1], w32), None, w32.k_tokens)
    act = to_np(sel.active_idx).astype(np.int64)
    st32.alloc_stream(sel)
    st32.quantize(2, to_dev(x32.K[1][act], w32), to_dev(x32.V[1][act], w32), sel)
    o_before = st32.o_store.clone()
    rc = st32.attention_indexed(2, to_dev(x32.Q[1][act], w32), sel, check=False)
    assert rc == -2 and torch.equal(st32.o_store, o_before)


def test_attention_workspace_calls(env):
    """Size query and hand-over of the workspace that lets the attention launch split its last wave."""
    import torch
    B, P, ctx = env
    sh = P.shape_of(small_bf16(L=1200))
    need = B.fl_loop_attention_workspace_bytes(ctx, sh)
    per_problem = 2 * 4 * (2 * 128 * 128 + 4 * 128)          # two partial results of binary32 values
    assert need > 1024 and (need - 1024) % per_problem == 0  # counters, then a whole number of split problems
    assert B.fl_loop_attention_workspace_bytes(ctx, P.shape_of(workloads.config1())) == 0   # f32: never split
    buf = torch.empty(need + 512, dtype=torch.uint8, device="cuda")
    assert B.fl_set_workspace(ctx, buf[1:], need, check=False) == B.FL_ERR_INVALID_ARG      # not 256-byte aligned
    assert B.fl_set_workspace(ctx, buf, 512, check=False) == -3                             # too small to be of use
    assert B.fl_set_workspace(ctx, buf, need, check=False) == 0
    assert B.fl_set_workspace(ctx, None, 0, check=False) == 0                               # detached again
    ctx._workspace = None


def test_programmatic_launch_off_gives_the_same_bits(env, monkeypatch):
    """FL_NO_PDL=1 (read when a context is created) launches every kernel fully serialized: same results."""
    import torch
    B, P, ctx = env
    w = small_bf16(L=1300, H=2, R=3)
    x = workloads.make_layer_inputs(w, seed=4)
    ref = fo.LayerOracle(w.L, w.n_heads, w.head_dim, w.q_block, w.bits, w.group, w.eps, w.sm_scale,
                         storage=w.dtype).run(x.G, x.Q, x.K, x.V, [w.k_tokens] * 2, [w.col_budget] * 2)
    monkeypatch.setenv("FL_NO_PDL", "1")
    ctx_plain = B.Context(0)
    monkeypatch.delenv("FL_NO_PDL")
    outs = []
    for c in (ctx, ctx_plain):
        st = P.LayerState(c, w)
        st.dense_loop(to_dev(x.Q[0], w), to_dev(x.K[0], w), to_dev(x.V[0], w))
        st.select_columns_dense()
        for r in (2, 3):
            sel = oracle_selection(P, w, ref, r)
            act = ref["active"][r - 2]
            st.sparse_loop(r, to_dev(x.Q[r - 1][act], w), to_dev(x.K[r - 1][act], w), to_dev(x.V[r - 1][act], w),
                           sel, indexed=True)
            st.check_status()
        outs.append((st.o_store.clone(), st.q_store.clone(), st.lse.clone(), st.col_idx.clone()))
    for a_, b_ in zip(*outs):
        assert torch.equal(a_, b_)
    ctx_plain.close()


def test_binary32_simt_attention_path_on_bf16_storage(env):
    """The SIMT attention kernels also serve bf16 storage (forced here; normally the tensor path runs)."""
    import os
    B, P, _ = env
    w = small_bf16(L=900, H=2, R=3)
    x = workloads.make_layer_inputs(w, seed=4)
    ref = fo.LayerOracle(w.L, w.n_heads, w.head_dim, w.q_block, w.bits, w.group, w.eps, w.sm_scale,
                         storage=w.dtype).run(x.G, x.Q, x.K, x.V, [w.k_tokens] * 2, [w.col_budget] * 2)
    os.environ["FL_FORCE_SIMT"] = "1"
    try:
        ctx = B.Context(0)
    finally:
        del os.environ["FL_FORCE_SIMT"]
    st = P.LayerState(ctx, w)
    st.dense_loop(to_dev(x.Q[0], w), to_dev(x.K[0], w), to_dev(x.V[0], w))
    st.select_columns_dense()
    for r in (2, 3):
        sel = oracle_selection(P, w, ref, r)
        act = ref["active"][r - 2]
        o_rows, _ = st.sparse_loop(r, to_dev(x.Q[r - 1][act], w), to_dev(x.K[r - 1][act], w),
                                   to_dev(x.V[r - 1][act], w), sel)
    assert_attn_close(to_np(st.o_store), ref["loops"][-1]["O_full"], "SIMT path final O store", carried=2)
    ctx.close()


@ROWS
def test_many_patched_columns_and_wide_budgets(env, rows, split):
    """Half of the rows active and a column budget of several chunks: long runs of columns that carry
    residual payloads (two ring slots per chunk) and several 128-row tiles per query block."""
    B, P, ctx = env
    w = dataclasses.replace(small_bf16(L=1536, H=2, R=3, c=640, q_block=512), token_frac=0.5,
                            changed_fracs=(0.6, 0.5))
    x = workloads.make_layer_inputs(w, seed=7)
    ref = fo.LayerOracle(w.L, w.n_heads, w.head_dim, w.q_block, w.bits, w.group, w.eps, w.sm_scale,
                         storage=w.dtype).run(x.G, x.Q, x.K, x.V, [w.k_tokens] * 2, [w.col_budget] * 2)
    st = P.LayerState(ctx, w, split=split)
    st.dense_loop(to_dev(x.Q[0], w), to_dev(x.K[0], w), to_dev(x.V[0], w))
    lse = ref["dense"]["lse"].astype(np.float32).copy()
    q_prev_full = x.Q[0]
    for r in (2, 3):
        rec = ref["loops"][r - 2]
        act = rec["active"]
        sel = oracle_selection(P, w, ref, r)
        st.alloc_stream(sel, rows=rows)
        st.quantize(r, to_dev(x.K[r - 1][act], w), to_dev(x.V[r - 1][act], w), sel)
        idx, cnt = sets_to_arrays(w, st.nb, rec["col_sets"], w.col_budget)
        st.col_idx, st.col_cnt, st.c = torch.from_numpy(idx).cuda(), torch.from_numpy(cnt).cuda(), w.col_budget
        st.lse = torch.from_numpy(lse).cuda()
        o_prev = to_dev(storage_round(rec["O_prev_rows"], w), w)
        o_out = torch.empty_like(o_prev)
        st.attention(r, to_dev(x.Q[r - 1][act], w), to_dev(q_prev_full[act], w), o_prev, o_out, sel)
        st.check_status()
        assert_attn_close(to_np(o_out), rec["O_rows"], f"loop {r} O rows (many patched columns)")
        ok = np.isfinite(rec["lse_rows"])
        lse = lse.copy(); lse[:, act] = np.where(ok, rec["lse_rows"], lse[:, act]).astype(np.float32)
        q_prev_full = q_prev_full.copy(); q_prev_full[act] = x.Q[r - 1][act]


def test_column_selection_exact_on_long_problems(env):
    """fl_select_columns on problems too long to list whole (a sampled pre-threshold, a candidate list, the bit map
    read-out) against brute force with the total order, for score distributions that stress every branch: heavy
    tails, a plateau of exact ties across the boundary, all zeros (the in-kernel fallback), a budget too wide for
    the candidate list, and a sparse source with a candidate list of columns."""
    B, P, ctx = env
    rng = np.random.default_rng(5)
    L, q_block, H = 24576, 8192, 2
    w = dataclasses.replace(workloads.config2(L=L, n_heads=H), q_block=q_block)
    sh = P.shape_of(w)
    nb = 3
    def scores(kind):
        s = np.zeros((H, nb, L), dtype=np.float32)
        for h in range(H):
            for b in range(nb):
                if kind == "lognormal":
                    v = np.exp(rng.standard_normal(L) * 3.0 - 6.0)
                elif kind == "plateau":
                    v = np.exp(rng.standard_normal(L) * 2.0 - 8.0)
                    v[rng.permutation(L)[: L // 8]] = 0.125          # thousands of exact ties, some across the boundary
                elif kind == "few_levels":
                    v = rng.integers(0, 4, L).astype(np.float64)     # four values only: ties everywhere
                else:
                    v = np.zeros(L)
                s[h, b] = v.astype(np.float32)
        return s
    for kind in ("lognormal", "plateau", "few_levels", "zeros"):
        cs = scores(kind)
        for c in (1, 300, 1024, 5000):
            col_idx = torch.empty(H, nb, c, dtype=torch.int32, device="cuda")
            col_cnt = torch.empty(H, nb, dtype=torch.int32, device="cuda")
            B.fl_select_columns(ctx, sh, torch.from_numpy(cs).cuda(), None, None, L, c, col_idx, col_cnt)
            idx, cnt = to_np(col_idx), to_np(col_cnt)
            for h in range(H):
                for b in range(nb):
                    end = min(L, (b + 1) * q_block)
                    k = min(c, end)
                    assert cnt[h, b] == k and np.all(idx[h, b, k:] == -1)
                    assert np.array_equal(idx[h, b, :k], fo.topk_ascending(cs[h, b, :end], k)), (kind, c, h, b)
    # sparse source: candidates are a subset of the columns (ascending), scores aligned with the list
    n_cand = 20000
    cand = np.sort(rng.permutation(L)[:n_cand]).astype(np.int32)
    cand_cols = np.broadcast_to(cand, (H, nb, n_cand)).copy()
    cand_cnt = np.array([[n_cand, 9000, 0]] * H, dtype=np.int32)
    cs = np.exp(rng.standard_normal((H, nb, n_cand)) * 3.0).astype(np.float32)
    for c in (700, 10000):
        col_idx = torch.empty(H, nb, c, dtype=torch.int32, device="cuda")
        col_cnt = torch.empty(H, nb, dtype=torch.int32, device="cuda")
        B.fl_select_columns(ctx, sh, torch.from_numpy(cs).cuda(), torch.from_numpy(cand_cols).cuda(),
                            torch.from_numpy(cand_cnt).cuda(), n_cand, c, col_idx, col_cnt)
        idx, cnt = to_np(col_idx), to_np(col_cnt)
        for h in range(H):
            for b in range(nb):
                n = cand_cnt[h, b]
                k = min(c, n)
                assert cnt[h, b] == k and np.all(idx[h, b, k:] == -1)
                assert np.array_equal(idx[h, b, :k], cand[fo.topk_ascending(cs[h, b, :n], k)]), (c, h, b)


@pytest.mark.parametrize("bits,group", [(4, 128), (4, 64), (8, 32), (2, 16), (2, 128)])
def test_quantizer_wide_rows_bit_exact(env, bits, group):
    """Rows of 512 elements (4 heads): the quantizer's 16-elements-per-thread kernel, five loops (up to three earlier
    streams in the chain, then the general kernel), codes, metadata and materialized rows against the oracle's codec
    alone (no attention: the oracle's residual_update chained by hand)."""
    B, P, ctx = env
    w = dataclasses.replace(small_bf16(L=700, H=4, R=4, bits=bits, group=group), n_loops=6,
                            changed_fracs=(0.3, 0.2, 0.15, 0.1, 0.08))
    x = workloads.make_layer_inputs(w, seed=23)
    st = P.LayerState(ctx, w)
    st.k_base, st.v_base = to_dev(x.K[0], w), to_dev(x.V[0], w)
    hats = [np.asarray(storage_round(x.K[0], w), dtype=np.float32), np.asarray(storage_round(x.V[0], w), dtype=np.float32)]
    rng = np.random.default_rng(5)
    act = np.arange(w.L)
    for r in range(2, w.n_loops + 1):
        act = np.sort(rng.choice(act, size=max(33, int(len(act) * 0.6)), replace=False))     # nested, odd counts
        sel = P.TokenSelection(torch.from_numpy(act.astype(np.int32)).cuda(),
                               torch.from_numpy(fo.slot_map(act, w.L)).cuda(), None, len(act))
        st.alloc_stream(sel)
        new = [storage_round(x.K[r - 1][act], w), storage_round(x.V[r - 1][act], w)]
        st.quantize(r, to_dev(new[0], w), to_dev(new[1], w), sel)
        for side, streams in enumerate((st.k_streams, st.v_streams)):
            hat_new, pay = fo.residual_update(new[side], hats[side], act, bits, group)
            got = streams[-1]
            n = len(act)
            assert np.array_equal(to_np(got["codes"]).reshape(n, w.n_heads, -1), pay["packed"]), (r, side)
            assert np.array_equal(to_np(got["scale"]).view(np.uint16).reshape(pay["scale"].shape), pay["scale"].view(np.uint16))
            assert np.array_equal(to_np(got["zero"]).view(np.uint16).reshape(pay["zero"].shape), pay["zero"].view(np.uint16))
            for name, want in (("rows_prev", hats[side]), ("rows_cur", hat_new)):
                got_rows = to_np(got[name]).astype(np.float32).reshape(n, w.n_heads, -1)
                assert np.array_equal(got_rows.view(np.uint32), fo.round_bf16(want[act]).view(np.uint32)), (r, side, name)
            hats[side] = hat_new
