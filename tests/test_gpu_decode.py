"""GPU parity of the sparse decode attention (fl_decode_attention) against the oracle's per-position form of the
replacement equation (Appendix D.2): a batch of decode queries over the store a prefill has left (base + residual
streams, bit-exact on both sides), every (query, head) with its own column subset chosen from a dense first loop."""
import dataclasses

import numpy as np
import pytest

from oracle import flashloop_oracle as fo
from paper_2609_29812_b200 import workloads
from helpers import assert_attn_close, storage_round, to_dev, to_np
from test_gpu_parity import oracle_selection, small_bf16

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


def dense_decode_loop(q, k, v, scale):
    """Loop 1 of the decode queries: textbook softmax attention over all cached keys (fp64)."""
    logits = np.einsum("thd,lhd->thl", q.astype(np.float64), k.astype(np.float64)) * scale
    mx = logits.max(axis=2, keepdims=True)
    e = np.exp(logits - mx)
    p = e / e.sum(axis=2, keepdims=True)
    o = np.einsum("thl,lhd->thd", p, v.astype(np.float64))
    lse = (mx + np.log(e.sum(axis=2, keepdims=True)))[:, :, 0]
    return o, p, lse


@pytest.mark.parametrize("name", ["bf16_int4", "bf16_int8_g64", "bf16_off", "c1_f32"])
def test_decode_attention_two_chained_loops(env, name):
    B, P, ctx = env
    w = {"bf16_int4": lambda: small_bf16(L=1500, H=2, R=3),
         "bf16_int8_g64": lambda: small_bf16(L=1200, H=2, R=3, bits=8, group=64),
         "bf16_off": lambda: small_bf16(L=1200, H=2, R=3, bits=16),
         "c1_f32": lambda: dataclasses.replace(workloads.config1(), n_loops=3, changed_fracs=(0.25, 0.12))}[name]()
    x = workloads.make_layer_inputs(w, seed=41)
    ref = fo.LayerOracle(w.L, w.n_heads, w.head_dim, w.q_block, w.bits, w.group, w.eps, w.sm_scale,
                         storage=w.dtype).run(x.G, x.Q, x.K, x.V, [w.k_tokens] * 2, [w.col_budget] * 2)
    bf16 = w.dtype == "bf16"
    rd = fo.round_bf16 if bf16 else None
    # the store, as the prefill leaves it (codes are bit-exact, checked elsewhere)
    st = P.LayerState(ctx, w)
    st.k_base, st.v_base = to_dev(x.K[0], w), to_dev(x.V[0], w)
    for r in (2, 3):
        sel = oracle_selection(P, w, ref, r)
        act = ref["active"][r - 2]
        st.alloc_stream(sel, rows=False)
        st.quantize(r, to_dev(x.K[r - 1][act], w), to_dev(x.V[r - 1][act], w), sel)
    # decode queries: one set per loop, storage precision
    rng = np.random.default_rng(3)
    Bq, H, dh, c = 5, w.n_heads, w.head_dim, 96
    store_r = lambda a: storage_round(a, w)
    q = [store_r(rng.standard_normal((Bq, H, dh)) * (1.0 if r == 0 else 1.0) + (0 if r == 0 else 0)) for r in range(3)]
    q[1] = store_r(q[0] + 0.2 * rng.standard_normal((Bq, H, dh)))
    q[2] = store_r(q[1] + 0.1 * rng.standard_normal((Bq, H, dh)))
    o1, p1, lse1 = dense_decode_loop(q[0], x.K[0], x.V[0], w.sm_scale)
    sets, p_old = {}, {}
    col_idx = np.full((Bq, H, c), -1, dtype=np.int32)
    col_cnt = np.zeros((Bq, H), dtype=np.int32)
    for t in range(Bq):
        for h in range(H):
            k_sel = c if (t, h) != (1, 0) else 7            # one short subset
            S = fo.select_columns(p1[t, h], np.arange(w.L), k_sel)
            if (t, h) == (2, 1):
                S = S[:0]                                   # and one empty one
            sets[(t, h)], p_old[(t, h)] = S, p1[t, h][S]
            col_idx[t, h, : len(S)] = S
            col_cnt[t, h] = len(S)
    d_idx, d_cnt = torch.from_numpy(col_idx).cuda(), torch.from_numpy(col_cnt).cuda()
    o_dev = to_dev(store_r(o1), w)
    lse_dev = torch.from_numpy(lse1.astype(np.float32)).cuda()
    o_or = o1
    for r in (2, 3):
        rec = ref["loops"][r - 2]
        res = fo.decode_sparse_attention(q[r - 1], rec["khat"], rec["vhat"], rec["vhat_old"], o_or, sets, p_old,
                                         w.sm_scale, kv_round=rd)
        p_out = torch.zeros(Bq, H, c, dtype=torch.float32, device="cuda")
        B.fl_decode_attention(ctx, st.shape, r, to_dev(q[r - 1], w), to_dev(q[r - 2], w), Bq, st.store, d_idx, d_cnt, c,
                              lse_dev, lse_dev, o_dev, o_dev, p_out)
        torch.cuda.synchronize()
        assert_attn_close(to_np(o_dev), res["O"], f"decode loop {r} ({name})", carried=r - 1, bf16=bf16)
        got_p = to_np(p_out)
        for (t, h), pn in res["p_new"].items():
            np.testing.assert_allclose(got_p[t, h, : len(pn)], pn, rtol=2e-3 if not bf16 else 2e-2, atol=1e-6)
            assert np.all(got_p[t, h, len(pn):] == 0)
        ok = np.isfinite(res["lse"])
        np.testing.assert_allclose(to_np(lse_dev)[ok], res["lse"][ok], rtol=0, atol=5e-3 * (r - 1))
        assert to_np(lse_dev)[2, 1] == np.float32(lse1[2, 1])          # empty subset: untouched
        o_or, p_old = res["O"], res["p_new"]
    assert np.array_equal(to_np(o_dev)[2, 1], store_r(o1)[2, 1])
