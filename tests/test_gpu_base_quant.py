"""GPU parity of the quantized loop-1 base (fl_quant_kv_base / fl_dequant_kv_base) against the oracle's quantize_base
(Appendix E, "Quantization Setting": keys per channel over token groups, values per token, recent tokens kept): codes,
scales and offsets bit for bit, rebuilt rows bit for bit, and one sparse loop run on the rebuilt base."""
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


def alloc_base(B, w, bits, group, tail, dev="cuda:0"):
    L, d = w.L, w.d
    Lq = max(0, L - tail)
    n_tg = (Lq + group - 1) // group
    dt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    u8 = lambda *s: torch.full(s, 0xEE, dtype=torch.uint8, device=dev)
    f16 = lambda *s: torch.full(s, -7.0, dtype=torch.float16, device=dev)
    t = dict(k_codes=u8(max(Lq, 1), d * bits // 8), k_scale=f16(max(n_tg, 1), d), k_zero=f16(max(n_tg, 1), d),
             v_codes=u8(max(Lq, 1), d * bits // 8), v_scale=f16(max(Lq, 1), d // group), v_zero=f16(max(Lq, 1), d // group),
             k_tail=torch.zeros(max(L - Lq, 1), d, dtype=dt, device=dev),
             v_tail=torch.zeros(max(L - Lq, 1), d, dtype=dt, device=dev))
    q = B.make_base_q(t["k_codes"], t["k_scale"], t["k_zero"], t["v_codes"], t["v_scale"], t["v_zero"], t["k_tail"],
                      t["v_tail"], group, tail)
    return q, t, Lq, n_tg


CASES = {"bf16_int4_g64_tail64": (lambda: small_bf16(L=1500, H=2, R=2), 4, 64, 64),      # 1436 quantized rows: 22 groups + 28 rows
         "bf16_int8_g128_tail0": (lambda: small_bf16(L=1200, H=2, R=2), 8, 128, 0),
         "bf16_int2_g32_tail200": (lambda: small_bf16(L=1200, H=2, R=2), 2, 32, 200),
         "f32_int4_g64": (lambda: workloads.config1(), 4, 64, 64),
         "shorter_than_tail": (lambda: small_bf16(L=300, H=2, R=2), 4, 64, 512)}


@pytest.mark.parametrize("name", list(CASES))
def test_base_codes_metadata_and_rebuilt_rows_bit_exact(env, name):
    B, P, ctx = env
    mk, bits, group, tail = CASES[name]
    w = mk()
    x = workloads.make_layer_inputs(w, seed=13)
    k1 = storage_round(x.K[0], w).reshape(w.L, w.d)
    v1 = storage_round(x.V[0], w).reshape(w.L, w.d)
    ref = fo.quantize_base(k1, v1, bits, group, tail, storage_round=fo.round_bf16 if w.dtype == "bf16" else None)
    sh = P.shape_of(w, bits=bits)
    q, t, Lq, n_tg = alloc_base(B, w, bits, group, tail)
    kd, vd = to_dev(k1, w), to_dev(v1, w)
    B.fl_quant_kv_base(ctx, sh, kd, vd, q)
    torch.cuda.synchronize()
    if Lq > 0:
        for side in "kv":
            assert np.array_equal(t[f"{side}_codes"][:Lq].cpu().numpy(), fo.pack_codes(ref[f"{side}_codes"], bits)), side
        assert np.array_equal(t["k_scale"][:n_tg].cpu().numpy().view(np.uint16), ref["k_scale"].view(np.uint16))
        assert np.array_equal(t["k_zero"][:n_tg].cpu().numpy().view(np.uint16), ref["k_zero"].view(np.uint16))
        assert np.array_equal(t["v_scale"][:Lq].cpu().numpy().view(np.uint16), ref["v_scale"].view(np.uint16))
        assert np.array_equal(t["v_zero"][:Lq].cpu().numpy().view(np.uint16), ref["v_zero"].view(np.uint16))
    n_tail = w.L - Lq
    if n_tail:
        assert np.array_equal(to_np(t["k_tail"][:n_tail]), k1[Lq:]) and np.array_equal(to_np(t["v_tail"][:n_tail]), v1[Lq:])
    k_out, v_out = torch.full_like(kd, 9.0), torch.full_like(vd, 9.0)
    B.fl_dequant_kv_base(ctx, sh, q, k_out, v_out)
    torch.cuda.synchronize()
    assert np.array_equal(to_np(k_out), ref["khat"]) and np.array_equal(to_np(v_out), ref["vhat"])
    assert B.fl_kv_base_q_bytes(sh, group, tail) == fo.base_q_bytes(w.L, w.d, bits, group, tail,
                                                                    2 if w.dtype == "bf16" else 4)


def test_masked_rebuild_touches_only_the_rows_the_sparse_loops_read(env):
    B, P, ctx = env
    w = small_bf16(L=1500, H=2, R=2)
    x = workloads.make_layer_inputs(w, seed=19)
    k1 = storage_round(x.K[0], w).reshape(w.L, w.d)
    v1 = storage_round(x.V[0], w).reshape(w.L, w.d)
    ref = fo.quantize_base(k1, v1, 4, 64, 64, storage_round=fo.round_bf16)
    sh = P.shape_of(w)
    q, t, Lq, n_tg = alloc_base(B, w, 4, 64, 64)
    B.fl_quant_kv_base(ctx, sh, to_dev(k1, w), to_dev(v1, w), q)
    # column lists with ragged counts and an active list, as a sparse loop would hand them over
    rng = np.random.default_rng(4)
    nb, c = (w.L + w.q_block - 1) // w.q_block, 40
    col_idx = np.full((w.n_heads, nb, c), -1, dtype=np.int32)
    col_cnt = np.zeros((w.n_heads, nb), dtype=np.int32)
    sets = {}
    for h in range(w.n_heads):
        for b in range(nb):
            m = int(rng.integers(0, c + 1)) if (h, b) != (0, 0) else 0
            S = np.sort(rng.choice(min(w.L, (b + 1) * w.q_block), size=m, replace=False))
            col_idx[h, b, :m], col_cnt[h, b], sets[(h, b)] = S, m, S
    active = np.sort(rng.choice(w.L, size=97, replace=False)).astype(np.int32)
    need = fo.base_rows_needed(sets, active, w.n_heads, w.L)
    words = (w.L + 31) // 32
    mask = torch.full((w.n_heads, words), -1, dtype=torch.int32, device="cuda:0")      # the call clears it first
    B.fl_mark_base_rows(ctx, sh, torch.from_numpy(col_idx).cuda(), torch.from_numpy(col_cnt).cuda(), c,
                        torch.from_numpy(active).cuda(), len(active), mask)
    torch.cuda.synchronize()
    bits = mask.cpu().numpy().view(np.uint32)
    got = ((bits[:, :, None] >> np.arange(32, dtype=np.uint32)) & 1).reshape(w.n_heads, -1)[:, :w.L].astype(bool)
    assert np.array_equal(got, need)
    k_out = torch.full((w.L, w.n_heads, w.head_dim), 9.0, dtype=torch.bfloat16, device="cuda:0")
    v_out = torch.full_like(k_out, 9.0)
    B.fl_dequant_kv_base(ctx, sh, q, k_out, v_out, row_mask=mask)
    torch.cuda.synchronize()
    shp = (w.L, w.n_heads, w.head_dim)
    want_k = np.where(need.T[:, :, None], ref["khat"].reshape(shp), np.float32(9.0))
    want_v = np.where(need.T[:, :, None], ref["vhat"].reshape(shp), np.float32(9.0))
    want_k[Lq:], want_v[Lq:] = ref["khat"].reshape(shp)[Lq:], ref["vhat"].reshape(shp)[Lq:]   # the tail is always copied
    assert np.array_equal(to_np(k_out), want_k) and np.array_equal(to_np(v_out), want_v)


def test_dense_and_sparse_loop_on_the_rebuilt_base(env):
    """The base is packed and rebuilt first, then loop 1 (dense) and loop 2 (sparse) both read the rebuilt rows: the
    attention of every loop sees the cache as it is stored, so the old term recomputed from the previous loop's
    log-normalisers is the one the previous loop produced.  The oracle runs the same layer on its own dequantized base."""
    B, P, ctx = env
    w = small_bf16(L=1500, H=2, R=2)
    x = workloads.make_layer_inputs(w, seed=17)
    shp = (w.L, w.n_heads, w.head_dim)
    k1 = storage_round(x.K[0], w).reshape(w.L, w.d)
    v1 = storage_round(x.V[0], w).reshape(w.L, w.d)
    qb = fo.quantize_base(k1, v1, 4, 64, 64, storage_round=fo.round_bf16)
    orc = fo.LayerOracle(w.L, w.n_heads, w.head_dim, w.q_block, w.bits, w.group, w.eps, w.sm_scale, storage=w.dtype)
    ref = orc.run(x.G, x.Q, [qb["khat"].reshape(shp), x.K[1]], [qb["vhat"].reshape(shp), x.V[1]], [w.k_tokens],
                  [w.col_budget])
    st = P.LayerState(ctx, w)
    assert st.pack_base(to_dev(k1, w), to_dev(v1, w), 64, 64) == fo.base_q_bytes(w.L, w.d, 4, 64, 64)
    k_re = torch.empty(shp, dtype=torch.bfloat16, device="cuda:0")
    v_re = torch.empty_like(k_re)
    st.rebuild_base(k_re, v_re)                    # every row: the dense loop reads all of them
    st.dense_loop(to_dev(x.Q[0], w), k_re, v_re)
    st.select_columns_dense()
    sel = oracle_selection(P, w, ref, 2)
    act = ref["active"][0]
    # before the sparse loop only the rows it reads are rebuilt, into a buffer that holds nothing else
    k_tr, v_tr = torch.full_like(k_re, float("nan")), torch.full_like(v_re, float("nan"))
    st.rebuild_base(k_tr, v_tr, sel)
    o_rows, _ = st.sparse_loop(2, to_dev(x.Q[1][act], w), to_dev(x.K[1][act], w), to_dev(x.V[1][act], w), sel,
                               indexed=True)
    st.check_status()
    rec = ref["loops"][0]
    assert np.array_equal(st.k_streams[0]["codes"].cpu().numpy().reshape(len(act), -1),
                          rec["k_payload"]["packed"].reshape(len(act), -1))
    assert_attn_close(to_np(o_rows), rec["O_rows"], "loop 2 on the rebuilt int4 base", carried=1)
