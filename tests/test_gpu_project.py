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
