"""Pins for the oracle's dense looped attention (Section 3.2) and the sparse attention
replacement (Appendix D.2): textbook special cases, a library routine, rational closed forms
and the identities the equations imply."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import flashloop_oracle as fo
from paper_2609_29812_b200 import workloads


def rand_qkv(rng, L, H, dh, scale=1.0):
    return [scale * rng.standard_normal((L, H, dh)) for _ in range(3)]


def test_dense_attention_textbook_cases():
    rng = np.random.default_rng(0)
    L, H, dh = 37, 2, 8
    q, k, v = rand_qkv(rng, L, H, dh)
    d = fo.dense_loop_attention(q, k, v, dh ** -0.5, q_block=8)
    # row 0 sees only key 0
    np.testing.assert_allclose(d["O"][0], v[0], rtol=1e-13)
    # every probability row sums to one => column scores summed over blocks and columns give L
    np.testing.assert_allclose(d["col_scores"].sum(axis=(1, 2)), L, rtol=1e-12)
    # nothing beyond a block's last row
    for b in range(fo.n_blocks(L, 8)):
        assert np.all(d["col_scores"][:, b, min(L, (b + 1) * 8):] == 0)
    # identical keys => causal running mean of V, and lse_i = logit + log(i+1)
    k_same = np.broadcast_to(k[:1], k.shape)
    d2 = fo.dense_loop_attention(q, k_same, v, dh ** -0.5, q_block=16)
    run_mean = np.cumsum(v, axis=0) / np.arange(1, L + 1)[:, None, None]
    np.testing.assert_allclose(d2["O"], run_mean, rtol=1e-12, atol=1e-13)
    logit = np.einsum("lhd,hd->hl", q, k[0]) * dh ** -0.5
    np.testing.assert_allclose(d2["lse"], logit + np.log(np.arange(1, L + 1))[None, :], rtol=1e-12)


def test_dense_attention_against_library_routine():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(1)
    L, H, dh = 50, 3, 16
    q, k, v = rand_qkv(rng, L, H, dh)
    d = fo.dense_loop_attention(q, k, v, dh ** -0.5, q_block=7)
    tq, tk, tv = [torch.from_numpy(a).permute(1, 0, 2)[None] for a in (q, k, v)]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)[0].permute(1, 0, 2).numpy()
    np.testing.assert_allclose(d["O"], ref, rtol=1e-10, atol=1e-12)
    rows = [0, 13, 49]
    np.testing.assert_allclose(fo.dense_attention_rows(q, k, v, dh ** -0.5, rows, 1), ref[rows, 1], rtol=1e-10)


def test_column_scores_brute_force():
    rng = np.random.default_rng(2)
    L, H, dh, Bq = 11, 1, 4, 4
    q, k, v = rand_qkv(rng, L, H, dh)
    d = fo.dense_loop_attention(q, k, v, 0.5, q_block=Bq)
    for b in range(3):
        for j in range(L):
            tot = 0.0
            for i in range(b * Bq, min(L, (b + 1) * Bq)):
                if j > i:
                    continue
                w = [np.exp(0.5 * float(q[i, 0] @ k[t, 0])) for t in range(i + 1)]
                tot += w[j] / sum(w)
            assert d["col_scores"][0, b, j] == pytest.approx(tot, rel=1e-12, abs=1e-15)


def run_two_loops(q1, k1, v1, q2, k2, v2, active, c, Bq, bits=16, group=None, scale=None):
    L, H, dh = q1.shape
    scale = dh ** -0.5 if scale is None else scale
    orc = fo.LayerOracle(L, H, dh, Bq, bits, group or dh, 1e-6, scale)
    # drive the stages by hand so that the active set can be imposed
    d1 = fo.dense_loop_attention(q1, k1, v1, scale, Bq, rows_to_cache=active)
    sets, cache = {}, {}
    for h in range(H):
        for b in range(orc.nb):
            end = min(L, (b + 1) * Bq)
            S = fo.select_columns(d1["col_scores"][h, b, :end], np.arange(end), c)
            rows, P = d1["probs"][(h, b)]
            sets[(h, b)] = S; cache[(h, b)] = (rows, P[:, S])
    khat1, vhat1 = k1.astype(np.float32), v1.astype(np.float32)
    khat2, _ = fo.residual_update(k2[active], khat1, active, bits, group or dh)
    vhat2, _ = fo.residual_update(v2[active], vhat1, active, bits, group or dh)
    res = fo.sparse_loop_attention(q2[active], khat2, vhat2, vhat1, d1["O"][active], active, sets, cache, scale, Bq)
    return d1, res, sets, (khat1, vhat1, khat2, vhat2)


def f32r(a):
    return a.astype(np.float32).astype(np.float64)


def test_full_budgets_quantization_off_equals_dense_looped_attention():
    """All tokens active, all columns selected, codec off: the sparse step must reproduce dense
    attention of loop 2 (the algebra of the replacement equation with m = 1)."""
    rng = np.random.default_rng(3)
    L, H, dh, Bq = 40, 2, 8, 8
    q1, k1, v1 = [f32r(a) for a in rand_qkv(rng, L, H, dh)]
    q2, k2, v2 = [f32r(a + 0.3 * rng.standard_normal(a.shape)) for a in (q1, k1, v1)]
    active = np.arange(L)
    d1, res, sets, _ = run_two_loops(q1, k1, v1, q2, k2, v2, active, c=L, Bq=Bq)
    dense2 = fo.dense_loop_attention(q2, k2, v2, dh ** -0.5, Bq)
    np.testing.assert_allclose(res["O"], dense2["O"], rtol=1e-9, atol=1e-11)
    for key, m in res["mass"].items():
        np.testing.assert_allclose(m, 1.0, rtol=1e-12)


def test_fixed_point_unchanged_inputs_any_column_set():
    rng = np.random.default_rng(4)
    L, H, dh, Bq = 48, 2, 8, 16
    q1, k1, v1 = [f32r(a) for a in rand_qkv(rng, L, H, dh)]
    active = np.sort(rng.permutation(L)[:20])
    for c in (1, 5, 17):
        d1, res, _, _ = run_two_loops(q1, k1, v1, q1, k1, v1, active, c=c, Bq=Bq)
        np.testing.assert_allclose(res["O"], d1["O"][active], rtol=1e-12, atol=1e-13)


def test_mass_properties_and_probability_sum():
    rng = np.random.default_rng(5)
    L, H, dh, Bq, c = 64, 2, 8, 16, 6
    q1, k1, v1 = [f32r(a) for a in rand_qkv(rng, L, H, dh)]
    q2, k2, v2 = [f32r(a + 0.3 * rng.standard_normal(a.shape)) for a in (q1, k1, v1)]
    active = np.sort(rng.permutation(L)[:30])
    d1, res, sets, _ = run_two_loops(q1, k1, v1, q2, k2, v2, active, c=c, Bq=Bq)
    for (h, b), m in res["mass"].items():
        rows, P = res["probs"][(h, b)]
        S = sets[(h, b)]
        np.testing.assert_allclose(P.sum(axis=1), m, rtol=1e-12, atol=1e-15)     # sum_S p^(r) = m
        for t, i in enumerate(rows):
            T = S[S <= i]
            if len(T) == 0:
                assert m[t] == 0
                continue
            assert 0 < m[t] <= 1 + 1e-12
            if len(T) == i + 1:                                                # all causal keys selected
                assert m[t] == pytest.approx(1.0, rel=1e-12)
            else:
                assert m[t] < 1.0
            assert np.all(P[t, S > i] == 0)


def test_rational_closed_form_per_position():
    """dh = 1, q = 1, scale = 1, keys = log(weights): probabilities are ratios of integers.
    With one query per block the block rule is the per-position rule of Appendix D.2.
    Expected values are computed with exact fractions from the weights."""
    L, c = 6, 2
    w1 = [3, 1, 4, 1, 5, 9]            # loop-1 weights of the keys
    w2 = [2, 7, 1, 8, 2, 8]            # loop-2 weights
    v1 = [Fraction(x) for x in (1, -2, 3, 5, -1, 2)]
    v2 = [Fraction(x) for x in (2, 0, -3, 4, 1, 7)]
    q = np.ones((L, 1, 1))
    k1 = np.log(np.array(w1, float)).reshape(L, 1, 1); k2 = np.log(np.array(w2, float)).reshape(L, 1, 1)
    V1 = np.array([float(x) for x in v1]).reshape(L, 1, 1); V2 = np.array([float(x) for x in v2]).reshape(L, 1, 1)
    active = np.arange(L)
    d1, res, sets, _ = run_two_loops(q, k1, V1, q, k2, V2, active, c=c, Bq=1, scale=1.0)
    for i in range(L):
        tot1 = sum(w1[: i + 1])
        p1 = [Fraction(w1[j], tot1) for j in range(i + 1)]
        o1 = sum(p1[j] * v1[j] for j in range(i + 1))
        order = sorted(range(i + 1), key=lambda j: (-p1[j], j))[:c]            # ties -> lowest index
        S = sorted(order)
        assert sets[(0, i)].tolist() == S
        m = sum(p1[j] for j in S)
        tot2 = sum(w2[j] for j in S)
        p2 = {j: m * Fraction(w2[j], tot2) for j in S}
        o2 = o1 - sum(p1[j] * v1[j] for j in S) + sum(p2[j] * v2[j] for j in S)
        assert d1["O"][i, 0, 0] == pytest.approx(float(o1), rel=1e-12)
        # the reconstructed keys are kept in binary32, so log(weights) carry a 2^-24 rounding
        assert res["O"][i, 0, 0] == pytest.approx(float(o2), rel=1e-6, abs=1e-7)
        assert res["mass"][(0, i)][0] == pytest.approx(float(m), rel=1e-12)      # loop-1 keys are fp64
        # the row's one-number summary: p2_j = exp(logit_j - lse) with logit_j = log w2_j, hence
        # lse = log(sum_S w2) - log m  (a sign slip in either term moves it by 2 log m or 2 log tot2)
        assert res["lse"][0, i] == pytest.approx(np.log(float(tot2)) - np.log(float(m)), rel=1e-6, abs=1e-6)
        for u, j in enumerate(S):
            assert np.exp(np.log(w2[j]) - res["lse"][0, i]) == pytest.approx(float(p2[j]), rel=1e-6)


def test_uniform_attention_closed_form_blocks():
    """q = 0 in both loops: p_ij = 1/(i+1).  All block scores tie except by how many rows see the
    column, so the selected set is the c lowest columns.  Only ACTIVE rows get new K/V (token-sparse
    update), so the result is the mean of [vhat2_0..vhat2_{c-1}, v1_c..v1_i] with vhat2_j = v2_j for
    active j and v1_j otherwise."""
    rng = np.random.default_rng(6)
    L, H, dh, Bq, c = 24, 1, 4, 8, 3
    z = np.zeros((L, H, dh))
    k1, v1, k2, v2 = [f32r(rng.standard_normal((L, H, dh))) for _ in range(4)]
    active = np.array([0, 2, 4, 9, 17, 23])
    d1, res, sets, _ = run_two_loops(z, k1, v1, z, k2, v2, active, c=c, Bq=Bq)
    for b in range(3):
        assert sets[(0, b)].tolist() == [0, 1, 2]
    for t, i in enumerate(active):
        vhat2 = v1.copy(); vhat2[active] = v2[active]
        mix = np.concatenate([vhat2[:c, 0], v1[c: i + 1, 0]], axis=0)[: i + 1].mean(axis=0)
        np.testing.assert_allclose(res["O"][t, 0], mix, rtol=1e-12, atol=1e-14)


def test_old_term_two_formulations_agree():
    """The cached-probability old term equals m * softmax_S(q^(r-1) K_S^(r-1)) V_S^(r-1)."""
    rng = np.random.default_rng(7)
    L, H, dh, Bq, c = 32, 1, 8, 8, 5
    q1, k1, v1 = [f32r(a) for a in rand_qkv(rng, L, H, dh)]
    active = np.sort(rng.permutation(L)[:12])
    d1, res, sets, (khat1, vhat1, _, _) = run_two_loops(q1, k1, v1, q1, k1, v1, active, c=c, Bq=Bq)
    blk = active // Bq
    for b in range(4):
        t_idx = np.nonzero(blk == b)[0]
        rows = active[t_idx]
        S = sets[(0, b)]
        c_rows, P = d1["probs"][(0, b)]
        P_S = np.where(S[None, :] <= rows[:, None], P[np.searchsorted(c_rows, rows)][:, S], 0.0)
        cached = P_S @ vhat1[S, 0].astype(np.float64)
        local = fo.old_term_local_softmax(q1[rows, 0], khat1, vhat1, rows, S, res["mass"][(0, b)], dh ** -0.5, 0)
        np.testing.assert_allclose(cached, local, rtol=1e-11, atol=1e-13)


def test_layer_oracle_constant_budget_sets_and_mass_are_loop_invariant():
    w = workloads.config2(L=256, n_heads=2)
    x = workloads.make_layer_inputs(w, seed=5)
    orc = fo.LayerOracle(w.L, 2, 128, 64, 4, 128, w.eps, w.sm_scale)
    out = orc.run(x.G, x.Q, x.K, x.V, [w.k_tokens] * 3, [32] * 3)
    l2, l3, l4 = out["loops"]
    for key in l2["col_sets"]:
        assert l2["col_sets"][key].tolist() == l3["col_sets"][key].tolist() == l4["col_sets"][key].tolist()
        np.testing.assert_allclose(l2["mass"][key], l3["mass"][key], rtol=1e-10, atol=1e-300)
        np.testing.assert_allclose(l3["mass"][key], l4["mass"][key], rtol=1e-10, atol=1e-300)
    # inactive rows keep their loop-1 output
    inactive = np.setdiff1d(np.arange(w.L), l2["active"])
    assert np.array_equal(l4["O_full"][inactive], out["dense"]["O"][inactive])


def test_layer_oracle_pruning_is_nested_and_error_shrinks_with_budget():
    w = workloads.config2(L=256, n_heads=2)
    x = workloads.make_layer_inputs(w, seed=6)
    orc = fo.LayerOracle(w.L, 2, 128, 64, 16, 128, w.eps, w.sm_scale)
    out = orc.run(x.G, x.Q, x.K, x.V, [64, 32, 16], [48, 24, 12])
    l2, l3, l4 = out["loops"]
    for key in l2["col_sets"]:
        assert set(l4["col_sets"][key]) <= set(l3["col_sets"][key]) <= set(l2["col_sets"][key])
        assert len(l3["col_sets"][key]) == min(24, len(l2["col_sets"][key]))
    # soft trend (Section 3.2): more columns => closer to dense loop-2 attention on the active rows
    errs = []
    for c in (8, 64, 256):
        o = fo.LayerOracle(w.L, 2, 128, 64, 16, 128, w.eps, w.sm_scale).run(x.G[:2], x.Q[:2], x.K[:2], x.V[:2], [256], [c])
        k2 = x.K[0].copy(); v2 = x.V[0].copy(); act = o["active"][0]
        k2[act] = x.K[1][act]; v2[act] = x.V[1][act]              # token-sparse K/V of loop 2, codec off
        dense = fo.dense_loop_attention(x.Q[1], k2, v2, w.sm_scale, 64)["O"]
        errs.append(np.linalg.norm(o["loops"][0]["O_full"] - dense) / np.linalg.norm(dense))
    assert errs[0] > errs[1] > errs[2] and errs[2] < 1e-9


def test_kv_round_is_applied_to_all_three_operands_values_by_hand():
    """One head, dh = 1, q = 1, scale = 1, two selected columns, one query: every number of the replacement equation
    can be written down.  K and V are chosen so that bf16 rounding moves each of the three operands the attention
    reads (Khat_new, Vhat_old, Vhat_new) by an amount that shows in the output; the expected value is computed from
    operands rounded with torch's own bfloat16 conversion (a library routine), not with the oracle's helper.
    Leaving any one operand unrounded fails the comparison."""
    torch = pytest.importorskip("torch")
    bf = lambda a: torch.tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16).double().numpy()
    L, S = 3, np.array([0, 1])
    k_new = np.array([0.3, 1.7, 0.0], dtype=np.float32).reshape(L, 1, 1)          # bf16: 0.30078125, 1.703125
    v_old = np.array([1.0 + 2.0 ** -9, -2.0 - 2.0 ** -8, 0.0], dtype=np.float32).reshape(L, 1, 1)
    v_new = np.array([3.0 + 2.0 ** -8, 5.0 + 2.0 ** -7, 0.0], dtype=np.float32).reshape(L, 1, 1)
    for arr in (k_new, v_old, v_new):
        assert np.all(bf(arr)[:2] != arr[:2].astype(np.float64))                    # rounding moves every operand
    p_old = np.array([[0.25, 0.5]])                                                # cached loop r-1 probabilities
    o_prev = np.array([[[0.75]]])
    active = np.array([2])
    sets = {(0, 0): S}
    cache = {(0, 0): (active, p_old)}
    q = np.ones((1, 1, 1))
    got = {}
    for name, rd in (("rounded", fo.round_bf16), ("plain", None)):
        got[name] = fo.sparse_loop_attention(q, k_new, v_new, v_old, o_prev, active, sets, cache, 1.0, q_block=4,
                                             kv_round=rd)
    m = 0.75
    def expect(kn, vo, vn):
        e = np.exp(kn[:2, 0, 0]); p_new = m * e / e.sum()
        return 0.75 - p_old[0] @ vo[:2, 0, 0] + p_new @ vn[:2, 0, 0], np.log(e.sum()) - np.log(m)
    want, want_lse = expect(bf(k_new), bf(v_old), bf(v_new))
    assert got["rounded"]["O"][0, 0, 0] == pytest.approx(want, rel=1e-13)
    assert got["rounded"]["lse"][0, 0] == pytest.approx(want_lse, rel=1e-13)
    plain, _ = expect(k_new.astype(np.float64), v_old.astype(np.float64), v_new.astype(np.float64))
    assert got["plain"]["O"][0, 0, 0] == pytest.approx(plain, rel=1e-13)
    # each operand on its own: an implementation that forgot one of the three roundings lands on one of these
    for miss in range(3):
        ops = [bf(k_new), bf(v_old), bf(v_new)]
        ops[miss] = (k_new, v_old, v_new)[miss].astype(np.float64)
        wrong, _ = expect(*ops)
        assert abs(wrong - want) > 1e-4 and got["rounded"]["O"][0, 0, 0] != pytest.approx(wrong, rel=1e-6)


def test_decode_oracle_pins():
    """decode_sparse_attention: (i) all keys selected with mass 1 = textbook softmax attention over the new K/V
    (library routine); (ii) unchanged query, keys and values leave the output where it was, for any subset;
    (iii) it is the per-position case (q_block = 1) of the prefill replacement, so the two must agree on a position
    appended after the prompt; (iv) hand values for one query, two columns."""
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(11)
    L, H, dh, Bq = 30, 2, 8, 3
    k1, v1, k2, v2 = [f32r(rng.standard_normal((L, H, dh))) for _ in range(4)]
    q1, q2 = [f32r(rng.standard_normal((Bq, H, dh))) for _ in range(2)]
    scale = dh ** -0.5
    def dense(q, k, v):
        out = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(q).permute(1, 0, 2)[None], torch.from_numpy(k).permute(1, 0, 2)[None],
            torch.from_numpy(v).permute(1, 0, 2)[None])[0].permute(1, 0, 2).numpy()
        logits = np.einsum("thd,lhd->thl", q, k) * scale
        p = np.exp(logits - logits.max(axis=2, keepdims=True)); p /= p.sum(axis=2, keepdims=True)
        return out, p
    o1, p1 = dense(q1, k1, v1)
    # (i) full sets: loop 2 equals dense attention over loop-2 K/V
    full = {(t, h): np.arange(L) for t in range(Bq) for h in range(H)}
    res = fo.decode_sparse_attention(q2, k2.astype(np.float32), v2.astype(np.float32), v1.astype(np.float32), o1, full,
                                     {(t, h): p1[t, h] for t in range(Bq) for h in range(H)}, scale)
    o2, p2 = dense(q2, k2, v2)
    np.testing.assert_allclose(res["O"], o2, rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(res["mass"], 1.0, rtol=1e-12)
    for t in range(Bq):
        for h in range(H):
            np.testing.assert_allclose(res["p_new"][(t, h)], p2[t, h], rtol=1e-9)
    # (ii) fixed point for arbitrary subsets
    sets = {(t, h): np.sort(rng.permutation(L)[: 1 + 3 * t + h]) for t in range(Bq) for h in range(H)}
    pold = {key: p1[key[0], key[1]][S] for key, S in sets.items()}
    same = fo.decode_sparse_attention(q1, k1.astype(np.float32), v1.astype(np.float32), v1.astype(np.float32), o1, sets,
                                      pold, scale)
    np.testing.assert_allclose(same["O"], o1, rtol=1e-12, atol=1e-13)
    # (iii) against the prefill form with one position per block: the decode position is row L of an extended prompt
    t, h = 1, 0
    ext = lambda a: np.concatenate([a, np.zeros((1, H, dh))], axis=0).astype(np.float32)
    S = sets[(t, h)]
    pre = fo.sparse_loop_attention(q2[t:t + 1], ext(k2), ext(v2), ext(v1), o1[t:t + 1], np.array([L]), {(h, L): S},
                                   {(h, L): (np.array([L]), pold[(t, h)][None, :])}, scale, q_block=1, head_list=[h],
                                   block_list=[L])
    dec = fo.decode_sparse_attention(q2, k2.astype(np.float32), v2.astype(np.float32), v1.astype(np.float32), o1, sets,
                                     pold, scale)
    np.testing.assert_allclose(dec["O"][t, h], pre["O"][0, h], rtol=1e-12, atol=1e-14)
    assert dec["lse"][t, h] == pytest.approx(pre["lse"][h, 0], rel=1e-12)
    # (iv) by hand: dh = 1, q = 1, scale = 1, keys log 2 and log 6, cached p = (1/4, 1/2): m = 3/4,
    # p_new = 3/4 * (2/8, 6/8) = (3/16, 9/16); o = 1 - (1/4 * 4 + 1/2 * (-2)) + (3/16 * 8 + 9/16 * 16) = 1 + 10.5
    one = fo.decode_sparse_attention(np.ones((1, 1, 1)), np.log(np.array([2.0, 6.0], dtype=np.float32)).reshape(2, 1, 1),
                                     np.array([8.0, 16.0], dtype=np.float32).reshape(2, 1, 1),
                                     np.array([4.0, -2.0], dtype=np.float32).reshape(2, 1, 1), np.ones((1, 1, 1)),
                                     {(0, 0): np.array([0, 1])}, {(0, 0): np.array([0.25, 0.5])}, 1.0)
    assert one["O"][0, 0, 0] == pytest.approx(11.5, rel=1e-6)
    np.testing.assert_allclose(one["p_new"][(0, 0)], [3 / 16, 9 / 16], rtol=1e-6)
    assert one["lse"][0, 0] == pytest.approx(np.log(8.0) - np.log(0.75), rel=1e-6)
