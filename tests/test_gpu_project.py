"""GPU parity of fl_project_rows (one tensor-core GEMM with gathered A rows and an indexed, optionally accumulating
epilogue) against the oracle's fp64 projection of the listed rows (Section 4.4 / Appendix G).

Tolerance, element by element: the inputs are bf16 on both sides, the kernel accumulates in binary32 and rounds each
output once to bf16, so |got - ref| <= 2^-8 |ref| (half a bf16 ulp, relative to the value's binade) + the binary32
accumulation bound d_in * 2^-23 * sum_k |x_k w_k|."""
import numpy as np
import pytest

from oracle import flashloop_oracle as fo
from paper_2609_29812_b200.workloads import round_to_bf16

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


@pytest.fixture(scope="module")
def env():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_29812_b200 import binding
    ctx = binding.Context(0)
    yield binding, ctx
    ctx.close()


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a)).to("cuda:0")
    return t.to(dtype) if dtype is not None else t


def make(seed, x_rows, y_rows, n, d_in, d_out, gather, scatter):
    rng = np.random.default_rng(seed)
    x = round_to_bf16(rng.standard_normal((x_rows, d_in)).astype(np.float32))
    w = round_to_bf16((rng.standard_normal((d_out, d_in)) / np.sqrt(d_in)).astype(np.float32))
    y = round_to_bf16(rng.standard_normal((y_rows, d_out)).astype(np.float32))
    src = np.sort(rng.choice(x_rows, size=n, replace=False)).astype(np.int32) if gather else None
    dst = np.sort(rng.choice(y_rows, size=n, replace=False)).astype(np.int32) if scatter else None
    return x, w, y, src, dst


def check(B, ctx, x, w, y, src, dst, n, accumulate, rows=None):
    d_in, d_out = x.shape[1], w.shape[0]
    xd, wd, yd = dev(x, torch.bfloat16), dev(w, torch.bfloat16), dev(y, torch.bfloat16)
    sd = dev(src) if src is not None else None
    dd = dev(dst) if dst is not None else None
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    B.fl_project_rows(ctx, xd, x.shape[0], sd, n, d_in, wd, d_out, yd, y.shape[0], dd, accumulate, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got = yd.float().cpu().numpy()
    touched = (dst if dst is not None else np.arange(n)).astype(np.int64)
    mask = np.ones(y.shape[0], dtype=bool)
    mask[touched] = False
    assert np.array_equal(got[mask], y[mask]), "rows that are not listed must stay bit-identical"
    # the oracle, on all listed rows or on a sample of them
    pick = np.arange(n) if rows is None else rows
    s_pick = (src[pick] if src is not None else pick)
    d_pick = (dst[pick] if dst is not None else pick)
    ref = fo.project_rows(x, s_pick, w, y, d_pick, bool(accumulate))[d_pick]
    mag = np.abs(x[s_pick].astype(np.float64)) @ np.abs(w.astype(np.float64)).T
    bound = 2.0 ** -8 * np.abs(ref) + d_in * 2.0 ** -23 * (mag + np.abs(y[d_pick])) + 1e-30
    err = np.abs(got[d_pick].astype(np.float64) - ref)
    worst = float(np.max(err / bound))
    assert worst <= 1.0, f"worst error / bound = {worst:.3f}"
    return worst


@pytest.mark.parametrize("gather,scatter,accumulate", [(True, False, 0), (False, True, 1), (True, True, 0),
                                                       (True, True, 1), (False, False, 0)])
def test_project_rows_ragged_tiles(env, gather, scatter, accumulate):
    B, ctx = env
    n = 300                                     # 2 full row tiles + 44 rows
    x, w, y, src, dst = make(7, 1000 if gather else n, 1000 if scatter else n, n, 256, 520, gather, scatter)
    check(B, ctx, x, w, y, src, dst, n, accumulate)       # d_out = 2 x 256 + 8: a ragged column tile


def test_project_rows_several_tiles_per_cta(env):
    """357 wide output tiles (21 x 17, the last column tile 8 columns wide, the last row tile 40 rows high) on at most
    148 CTAs: every CTA runs two or three tiles, so both accumulators are reused and the stage ring wraps many times.
    The small cases above run with the narrow tile, this one and the benchmark's Q/K/V shape with the wide one."""
    B, ctx = env
    n = 2600
    x, w, y, src, dst = make(8, 4000, 4000, n, 512, 4104, True, True)
    rows = np.sort(np.random.default_rng(1).choice(n, size=400, replace=False))
    check(B, ctx, x, w, y, src, dst, n, 1, rows=rows)


def test_project_rows_single_row_and_empty(env):
    B, ctx = env
    x, w, y, src, dst = make(9, 50, 50, 1, 64, 8, True, True)
    check(B, ctx, x, w, y, src, dst, 1, 0)
    yd = dev(y, torch.bfloat16)
    B.fl_project_rows(ctx, dev(x, torch.bfloat16), 50, None, 0, 64, dev(w, torch.bfloat16), 8, yd, 50, None, 0)
    torch.cuda.synchronize()
    assert np.array_equal(yd.float().cpu().numpy(), y)


def test_project_rows_benchmark_shape_sampled(env):
    """The QKV projection of the benchmark shape (3277 active rows of 32768, d = 2048, 3 d outputs) and the output
    projection with its residual add scattered back, checked on sampled rows."""
    B, ctx = env
    n, L, d = 3277, 32768, 2048
    rows = np.sort(np.random.default_rng(2).choice(n, size=48, replace=False))
    x, w, y, src, _ = make(10, L, n, n, d, 3 * d, True, False)
    check(B, ctx, x, w, y, src, None, n, 0, rows=rows)
    x, w, y, _, dst = make(11, n, L, n, d, d, False, True)
    check(B, ctx, x, w, y, None, dst, n, 1, rows=rows)


# ---- the stacked Q/K/V projection with the residual codec as its epilogue ---------------------------------------
from paper_2609_29812_b200 import workloads            # noqa: E402
from helpers import to_dev, to_np                       # noqa: E402
from test_gpu_parity import small_bf16                  # noqa: E402


@pytest.mark.parametrize("bits,group,H,n_loops", [(4, 128, 2, 3), (8, 64, 2, 2), (2, 32, 4, 2)])
def test_projection_with_codec_epilogue(env, bits, group, H, n_loops):
    """Loops 2..n_loops of one small layer through fl_project_qkv_quant.  Q and the new K | V rows against the oracle's
    fp64 projection; codes, scales, offsets and the materialized rows bit for bit against the oracle's residual codec
    applied to the kernel's own bf16 K | V rows (the reading: the codes are those of the GEMM's own outputs); and every
    output bit for bit against the unfused calls (fl_project_rows, then fl_quant_kv_residual)."""
    from paper_2609_29812_b200 import pipeline as P
    B, ctx = env
    w = small_bf16(L=700, H=H, R=n_loops, bits=bits, group=group)
    L, d = w.L, w.d
    rng = np.random.default_rng(31)
    hid = [round_to_bf16(rng.standard_normal((L, d)).astype(np.float32)) for _ in range(n_loops)]
    wqkv = round_to_bf16((rng.standard_normal((3 * d, d)) / np.sqrt(d)).astype(np.float32))
    k1 = round_to_bf16(rng.standard_normal((L, d)).astype(np.float32))
    v1 = round_to_bf16(rng.standard_normal((L, d)).astype(np.float32))
    shp = (L, w.n_heads, w.head_dim)
    st, st_ref = P.LayerState(ctx, w), P.LayerState(ctx, w)
    for s_ in (st, st_ref):
        s_.k_base, s_.v_base = to_dev(k1.reshape(shp), w), to_dev(v1.reshape(shp), w)
    wd = dev(wqkv, torch.bfloat16)
    khat, vhat = k1.reshape(shp).copy(), v1.reshape(shp).copy()
    act = np.arange(L)
    for r in range(2, n_loops + 1):
        act = np.sort(rng.choice(act, size=max(40, len(act) // 3), replace=False))     # nested, ragged against 128
        n = len(act)
        sel = P.TokenSelection(torch.from_numpy(act.astype(np.int32)).cuda(),
                               torch.from_numpy(fo.slot_map(act, L)).cuda(), None, n)
        hd = dev(hid[r - 1], torch.bfloat16)
        st.alloc_stream(sel)
        q_out = torch.full((n, d), 5.0, dtype=torch.bfloat16, device="cuda:0")
        kv_out = torch.full((n, 2 * d), 5.0, dtype=torch.bfloat16, device="cuda:0")
        status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
        B.fl_project_qkv_quant(ctx, st.shape, r, hd, L, sel.active_idx, n, wd, q_out, kv_out, st.store, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        rows_prev = [to_np(st.k_streams[-1]["rows_prev"]).copy(), to_np(st.v_streams[-1]["rows_prev"]).copy()]
        rows_cur = [to_np(st.k_streams[-1]["rows_cur"]).copy(), to_np(st.v_streams[-1]["rows_cur"]).copy()]
        # (1) the projection itself
        ref = fo.project_rows(hid[r - 1], act, wqkv, np.zeros((n, 3 * d)), None, False)
        mag = np.abs(hid[r - 1][act].astype(np.float64)) @ np.abs(wqkv.astype(np.float64)).T
        got = np.concatenate([to_np(q_out), to_np(kv_out)], axis=1).astype(np.float64)
        assert np.max(np.abs(got - ref) / (2.0 ** -8 * np.abs(ref) + d * 2.0 ** -23 * mag + 1e-30)) <= 1.0
        # (2) the codec, on the kernel's own K | V rows
        kv = to_np(kv_out)
        for side, (streams, hat, new) in enumerate(((st.k_streams, khat, kv[:, :d]), (st.v_streams, vhat, kv[:, d:]))):
            hat_new, pay = fo.residual_update(new.reshape(n, w.n_heads, w.head_dim), hat, act, bits, group)
            got_s = streams[-1]
            assert np.array_equal(got_s["codes"].cpu().numpy().reshape(n, -1), pay["packed"].reshape(n, -1)), (r, side)
            assert np.array_equal(got_s["scale"].cpu().numpy().view(np.uint16).reshape(-1), pay["scale"].view(np.uint16).reshape(-1))
            assert np.array_equal(got_s["zero"].cpu().numpy().view(np.uint16).reshape(-1), pay["zero"].view(np.uint16).reshape(-1))
            assert np.array_equal(rows_prev[side].reshape(n, -1), fo.round_bf16(hat[act]).reshape(n, -1))
            assert np.array_equal(rows_cur[side].reshape(n, -1), fo.round_bf16(hat_new[act]).reshape(n, -1))
            if side == 0:
                khat = hat_new
            else:
                vhat = hat_new
        # (3) the unfused calls on a second store
        st_ref.alloc_stream(sel)
        qkv = torch.empty(n, 3 * d, dtype=torch.bfloat16, device="cuda:0")
        B.fl_project_rows(ctx, hd, L, sel.active_idx, n, d, wd, 3 * d, qkv, n, None, 0, status)
        k_new, v_new = qkv[:, d:2 * d].contiguous(), qkv[:, 2 * d:].contiguous()
        B.fl_quant_kv_residual(ctx, st_ref.shape, r, k_new, v_new, sel.active_idx, n, st_ref.store)
        torch.cuda.synchronize()
        assert torch.equal(qkv[:, :d], q_out) and torch.equal(qkv[:, d:], kv_out)
        for a_, b_ in ((st.k_streams[-1], st_ref.k_streams[-1]), (st.v_streams[-1], st_ref.v_streams[-1])):
            for key in ("codes", "scale", "zero"):
                assert torch.equal(a_[key], b_[key]), (r, key)
        assert np.array_equal(to_np(st_ref.k_streams[-1]["rows_cur"]), rows_cur[0])
        assert np.array_equal(to_np(st_ref.v_streams[-1]["rows_prev"]), rows_prev[1])
