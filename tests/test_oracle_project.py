"""Pins for the oracle's projection of the active rows (Section 4.4 / Appendix G)."""
import numpy as np

from oracle import flashloop_oracle as fo


def test_hand_values_gather_project_scatter():
    x = np.array([[1.0, 2.0], [3.0, 4.0], [5.0, 6.0]])
    w = np.array([[1.0, 0.0], [0.0, 1.0], [1.0, 1.0], [2.0, -1.0]])       # [d_out = 4, d_in = 2]
    y = np.full((5, 4), 10.0)
    out = fo.project_rows(x, [2, 0], w, y, [1, 3], accumulate=False)
    assert out[1].tolist() == [5.0, 6.0, 11.0, 4.0]        # row 2 of x lands in row 1 of y
    assert out[3].tolist() == [1.0, 2.0, 3.0, 0.0]         # row 0 of x lands in row 3
    assert np.all(out[[0, 2, 4]] == 10.0)                  # untouched rows keep their contents
    acc = fo.project_rows(x, [2, 0], w, y, [1, 3], accumulate=True)
    assert acc[1].tolist() == [15.0, 16.0, 21.0, 14.0]
    assert np.all(acc[[0, 2, 4]] == 10.0)
    assert np.all(y == 10.0)                               # the input is not modified


def test_equals_full_matmul_then_selection():
    rng = np.random.default_rng(5)
    x = rng.standard_normal((40, 24))
    w = rng.standard_normal((56, 24))
    y = rng.standard_normal((64, 56))
    src = np.sort(rng.choice(40, size=17, replace=False))
    dst = np.sort(rng.choice(64, size=17, replace=False))
    full = np.einsum("ik,nk->in", x, w)                    # every row projected, then the listed ones picked
    want = y.copy()
    want[dst] += full[src]
    np.testing.assert_allclose(fo.project_rows(x, src, w, y, dst, True), want, rtol=0, atol=1e-12)
    want2 = y.copy()
    want2[:17] = full[src]
    np.testing.assert_allclose(fo.project_rows(x, src, w, y, None, False), want2, rtol=0, atol=1e-12)
    want3 = y.copy()
    want3[dst] = full[:17]
    np.testing.assert_allclose(fo.project_rows(x, None, w, y, dst, False), want3, rtol=0, atol=1e-12)


def test_identity_weight_copies_rows():
    rng = np.random.default_rng(6)
    x = rng.standard_normal((9, 8))
    out = fo.project_rows(x, [8, 1, 4], np.eye(8), np.zeros((3, 8)), None, False)
    assert np.array_equal(out, x[[8, 1, 4]])
