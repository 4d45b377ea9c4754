"""Parity at the benchmark's full size and launch configuration: one layer of the 48-layer workload (L = 32768,
16 x 128 heads, 3277 active rows, 1024 columns per block, int4 g128), run through the same entry points and launch
shapes that bench.py times (fl_loop_attention_indexed on the position-indexed stores).  The oracle cannot afford the
whole layer, so token selection is checked in full and everything downstream on sampled (head, block) pairs, each
computed by the oracle on its own from the inputs."""
import numpy as np
import pytest

from oracle import flashloop_oracle as fo
from paper_2609_29812_b200 import workloads
from helpers import assert_attn_close, assert_selection_matches, to_np

pytestmark = pytest.mark.gpu

# (head, query block): first, early, middle and last blocks (every block of this workload holds 84-120 active rows,
# i.e. one 128-row tile)
SAMPLES = [(0, 0), (5, 1), (3, 7), (12, 13), (9, 20), (6, 26), (1, 30), (15, 31)]


def test_full_size_layer_loops_2_and_3_sampled_against_oracle():
    import torch
    from paper_2609_29812_b200 import binding as B, pipeline as P
    w = workloads.config3(n_layers=1)
    dev = "cuda:0"
    ctx = B.Context(0)
    stack = workloads.DeviceStack(w, seed=0, device=dev)
    G = stack.stack_hidden()
    gen = stack.layer(0)
    q1, k1, v1 = gen.qkv1()
    st = P.LayerState(ctx, w, dev)
    st.dense_loop(q1, k1, v1)
    st.select_columns_dense()
    col_idx, col_cnt = to_np(st.col_idx), to_np(st.col_cnt)
    nb = st.nb

    # ---- the GPU path, loops 2 and 3, through the calls and launch shapes bench.py times --------------------
    gpu = {}
    cand = None
    for r in (2, 3):
        sel = P.select_tokens(ctx, st.shape, r, G[r - 2], G[r - 1], cand, w.k_tokens)
        act = to_np(sel.active_idx).astype(np.int64)
        # stage 1 in full: fp64 scores of every candidate and their exact top-k (near-tie band at the boundary)
        cand_np = np.arange(w.L) if cand is None else to_np(cand).astype(np.int64)
        s_ref = fo.token_scores(to_np(G[r - 2]), to_np(G[r - 1]), cand_np, w.eps)
        assert_selection_matches(act, s_ref, cand_np, w.k_tokens, f"token set of loop {r} at L=32768")
        np.testing.assert_allclose(to_np(sel.scores)[: len(cand_np)], s_ref, rtol=2e-5, atol=0)
        assert np.array_equal(to_np(sel.slot_of_pos), fo.slot_map(act, w.L))
        qr, kr, vr = gen.rows(r, sel.active_idx)
        st.alloc_stream(sel)
        st.quantize(r, kr, vr, sel)
        o_before = st.o_store.clone()
        assert st.attention_indexed(r, qr, sel) == 0
        st.check_status()
        untouched = np.ones(w.L, dtype=bool)
        untouched[act] = False
        keep = torch.from_numpy(untouched).to(dev)
        assert torch.equal(st.o_store[keep], o_before[keep])
        gpu[r] = dict(act=act, q=qr, k=kr, v=vr, o=to_np(st.o_store), lse=to_np(st.lse),
                      k_codes=to_np(st.k_streams[-1]["codes"]).reshape(len(act), w.n_heads, -1),
                      v_codes=to_np(st.v_streams[-1]["codes"]).reshape(len(act), w.n_heads, -1),
                      k_scale=to_np(st.k_streams[-1]["scale"]).view(np.uint16).reshape(len(act), w.n_heads, -1),
                      k_zero=to_np(st.k_streams[-1]["zero"]).view(np.uint16).reshape(len(act), w.n_heads, -1),
                      v_scale=to_np(st.v_streams[-1]["scale"]).view(np.uint16).reshape(len(act), w.n_heads, -1),
                      v_zero=to_np(st.v_streams[-1]["zero"]).view(np.uint16).reshape(len(act), w.n_heads, -1))
        cand = sel.active_idx

    # ---- the oracle, on its own, for sampled (head, block) pairs -------------------------------------------
    for h, b in SAMPLES:
        hs = slice(h, h + 1)
        q1h, k1h, v1h = (to_np(t[:, hs, :]) for t in (q1, k1, v1))
        end = min(w.L, (b + 1) * w.q_block)
        act2 = gpu[2]["act"]
        # dense source loop of the block's rows, column scores, column set (Eq. 6)
        d1 = fo.dense_loop_attention(q1h, k1h, v1h, w.sm_scale, w.q_block, rows_to_cache=act2, head_list=[0],
                                     block_list=[b])
        S_gpu = col_idx[h, b, : col_cnt[h, b]].astype(np.int64)
        assert col_cnt[h, b] == min(w.col_budget, end)
        assert_selection_matches(S_gpu, d1["col_scores"][0, b, :end], np.arange(end), w.col_budget,
                                 f"column set of head {h}, block {b}")
        sets = {(0, bb): np.zeros(0, dtype=np.int64) for bb in range(nb)}
        cache = {(0, bb): (np.zeros(0, dtype=np.int64), np.zeros((0, 0))) for bb in range(nb)}
        rows, P1 = d1["probs"][(0, b)]
        sets[(0, b)] = S_gpu
        cache[(0, b)] = (rows, P1[:, S_gpu])
        khat, vhat = k1h.astype(np.float32), v1h.astype(np.float32)
        o_full = d1["O"]
        for r in (2, 3):
            g = gpu[r]
            act = g["act"]
            # residual codec of this head's rows (Eq. 8): codes and metadata bit for bit
            khat_new, kpay = fo.residual_update(to_np(g["k"][:, hs, :]), khat, act, w.bits, w.group)
            vhat_new, vpay = fo.residual_update(to_np(g["v"][:, hs, :]), vhat, act, w.bits, w.group)
            assert np.array_equal(g["k_codes"][:, h], kpay["packed"][:, 0]), (r, h, "K codes")
            assert np.array_equal(g["v_codes"][:, h], vpay["packed"][:, 0]), (r, h, "V codes")
            assert np.array_equal(g["k_scale"][:, h], kpay["scale"][:, 0].view(np.uint16)), (r, h, "K scale")
            assert np.array_equal(g["k_zero"][:, h], kpay["zero"][:, 0].view(np.uint16)), (r, h, "K offset")
            assert np.array_equal(g["v_scale"][:, h], vpay["scale"][:, 0].view(np.uint16)), (r, h, "V scale")
            assert np.array_equal(g["v_zero"][:, h], vpay["zero"][:, 0].view(np.uint16)), (r, h, "V offset")
            # attention replacement of the block's active rows (Eq. 7) over the GPU's column set
            res = fo.sparse_loop_attention(to_np(g["q"][:, hs, :]), khat_new, vhat_new, vhat, o_full[act], act, sets,
                                           cache, w.sm_scale, w.q_block, head_list=[0], block_list=[b],
                                           kv_round=fo.round_bf16)
            in_block = np.nonzero(act // w.q_block == b)[0]
            assert len(in_block) > 0
            assert_attn_close(g["o"][act[in_block], h], res["O"][in_block, 0],
                              f"O rows of loop {r}, head {h}, block {b}", carried=r - 1)
            np.testing.assert_allclose(g["lse"][h, act[in_block]], res["lse"][0, in_block], rtol=0, atol=5e-3 * (r - 1))
            o_full = o_full.copy()
            o_full[act] = res["O"]
            cache = {key: (res["probs"][key] if key[1] == b else cache[key]) for key in cache}
            khat, vhat = khat_new, vhat_new
    ctx.close()


def test_config2_full_size_chained_on_gpu_against_the_full_oracle():
    """One layer at L = 8192 with all 16 heads, loops 2-4 chained on the GPU through the indexed entry point, against
    the oracle run in full on the same inputs: token sets, codes of every head, O rows of every loop and the final
    O store."""
    import torch
    from paper_2609_29812_b200 import binding as B, pipeline as P
    from helpers import to_dev
    w = workloads.config2()
    x = workloads.make_layer_inputs(w, seed=0)
    ref = fo.LayerOracle(w.L, w.n_heads, w.head_dim, w.q_block, w.bits, w.group, w.eps, w.sm_scale,
                         storage=w.dtype).run(x.G, x.Q, x.K, x.V, [w.k_tokens] * 3, [w.col_budget] * 3)
    ctx = B.Context(0)
    st = P.LayerState(ctx, w)
    st.dense_loop(to_dev(x.Q[0], w), to_dev(x.K[0], w), to_dev(x.V[0], w))
    st.select_columns_dense()
    assert_attn_close(to_np(st.o_store), ref["dense"]["O"], "config 2 dense source O")
    idx, cnt = to_np(st.col_idx), to_np(st.col_cnt)
    n_diff = 0
    for (h, b), S in ref["loops"][0]["col_sets"].items():
        end = min(w.L, (b + 1) * w.q_block)
        n_diff += assert_selection_matches(idx[h, b, : cnt[h, b]], ref["dense"]["col_scores"][h, b, :end],
                                           np.arange(end), w.col_budget, f"config 2 columns h{h} b{b}")
    assert n_diff <= 0.01 * w.n_heads * st.nb * w.col_budget
    cand = None
    for r in range(2, w.n_loops + 1):
        rec = ref["loops"][r - 2]
        sel = P.select_tokens(ctx, st.shape, r, to_dev(x.G[r - 2], w), to_dev(x.G[r - 1], w), cand, w.k_tokens)
        act = to_np(sel.active_idx).astype(np.int64)
        assert np.array_equal(act, rec["active"]), f"token set of loop {r}"
        o_rows, _ = st.sparse_loop(r, to_dev(x.Q[r - 1][act], w), to_dev(x.K[r - 1][act], w),
                                   to_dev(x.V[r - 1][act], w), sel, indexed=True)
        st.check_status()
        for side, streams in (("k_payload", st.k_streams), ("v_payload", st.v_streams)):
            pay, got = rec[side], streams[-1]
            assert np.array_equal(to_np(got["codes"]).reshape(len(act), w.n_heads, -1), pay["packed"]), (r, side)
            assert np.array_equal(to_np(got["scale"]).view(np.uint16).reshape(pay["scale"].shape),
                                  pay["scale"].view(np.uint16)), (r, side)
            assert np.array_equal(to_np(got["zero"]).view(np.uint16).reshape(pay["zero"].shape),
                                  pay["zero"].view(np.uint16)), (r, side)
        assert_attn_close(to_np(o_rows), rec["O_rows"], f"config 2 chained loop {r} O rows", carried=r - 1)
        cand = sel.active_idx
    assert_attn_close(to_np(st.o_store), ref["loops"][-1]["O_full"], "config 2 chained final O store",
                      carried=w.n_loops - 1)
    ctx.close()


def test_packed_base_at_bench_size_sampled_against_oracle():
    """The packed loop-1 base at the benchmark's size (L = 32768, d = 2048, int4, groups of 64, tail 64): sampled token
    groups of the keys and sampled rows of the values bit for bit against the oracle (groups are independent, so the
    oracle packs just the sampled slices), the rebuilt rows of the same samples, and the tail."""
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_29812_b200 import binding as B, pipeline as P
    w = workloads.config3(n_layers=1)
    L, d, g, tail, bits = w.L, w.d, 64, 64, 4
    Lq, n_tg = L - tail, (L - tail + g - 1) // g
    gen = torch.Generator(device="cuda:0"); gen.manual_seed(11)
    scale_c = 10.0 ** (torch.rand(d, device="cuda:0", generator=gen) * 3 - 2)              # channels of mixed magnitude
    k = (torch.randn(L, d, device="cuda:0", generator=gen) * scale_c).to(torch.bfloat16)
    v = (torch.randn(L, d, device="cuda:0", generator=gen) * (10.0 ** (torch.rand(L, 1, device="cuda:0", generator=gen) * 3 - 2))
         ).to(torch.bfloat16)
    u8 = lambda *s: torch.empty(s, dtype=torch.uint8, device="cuda:0")
    f16 = lambda *s: torch.empty(s, dtype=torch.float16, device="cuda:0")
    t = [u8(Lq, d // 2), f16(n_tg, d), f16(n_tg, d), u8(Lq, d // 2), f16(Lq, d // g), f16(Lq, d // g),
         torch.empty(tail, d, dtype=torch.bfloat16, device="cuda:0"), torch.empty(tail, d, dtype=torch.bfloat16, device="cuda:0")]
    with B.Context(0) as ctx:
        sh = P.shape_of(w)
        q = B.make_base_q(*t, g, tail)
        B.fl_quant_kv_base(ctx, sh, k, v, q)
        k_out, v_out = torch.empty_like(k), torch.empty_like(v)
        B.fl_dequant_kv_base(ctx, sh, q, k_out, v_out)
        torch.cuda.synchronize()
        assert B.fl_kv_base_q_bytes(sh, g, tail) == fo.base_q_bytes(L, d, bits, g, tail)
    rng = np.random.default_rng(3)
    for tg in [0, n_tg - 1] + rng.choice(n_tg, size=4, replace=False).tolist():        # the last group is 0 .. 63 rows short
        lo, hi = tg * g, min(Lq, (tg + 1) * g)
        ks = to_np(k[lo:hi]); vs = to_np(v[lo:hi])
        ref = fo.quantize_base(ks, vs, bits, g, 0, storage_round=fo.round_bf16)
        assert np.array_equal(t[0][lo:hi].cpu().numpy(), fo.pack_codes(ref["k_codes"], bits)), tg
        assert np.array_equal(t[1][tg].cpu().numpy().view(np.uint16), ref["k_scale"][0].view(np.uint16)), tg
        assert np.array_equal(t[2][tg].cpu().numpy().view(np.uint16), ref["k_zero"][0].view(np.uint16)), tg
        assert np.array_equal(t[3][lo:hi].cpu().numpy(), fo.pack_codes(ref["v_codes"], bits)), tg
        assert np.array_equal(t[4][lo:hi].cpu().numpy().view(np.uint16), ref["v_scale"].view(np.uint16)), tg
        assert np.array_equal(t[5][lo:hi].cpu().numpy().view(np.uint16), ref["v_zero"].view(np.uint16)), tg
        assert np.array_equal(to_np(k_out[lo:hi]), ref["khat"]) and np.array_equal(to_np(v_out[lo:hi]), ref["vhat"]), tg
    assert torch.equal(k_out[Lq:], k[Lq:]) and torch.equal(v_out[Lq:], v[Lq:]) and torch.equal(t[6], k[Lq:])
