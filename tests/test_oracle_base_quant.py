"""Pins for the oracle's quantization of the loop-1 base (Appendix E "Quantization Setting": keys per channel, values
per token, the most recent tokens unquantized)."""
import numpy as np

from oracle import flashloop_oracle as fo


def test_hand_values_two_bits():
    # one channel, four tokens 0..3 with 2 bits: offset 0, step 1, codes are the values themselves
    k = np.array([[0.0], [1.0], [2.0], [3.0]], dtype=np.float32)
    # one token, four channels 10, 13, 16, 19: offset 10, step 3, codes 0..3
    v = np.tile(np.array([[10.0, 13.0, 16.0, 19.0]], dtype=np.float32), (4, 1))
    k4 = np.tile(k, (1, 4))
    q = fo.quantize_base(k4, v, bits=2, group=4, tail=0)
    assert q["k_codes"][:, 0].tolist() == [0, 1, 2, 3] and float(q["k_scale"][0, 0]) == 1.0 and float(q["k_zero"][0, 0]) == 0.0
    assert q["v_codes"][0].tolist() == [0, 1, 2, 3] and float(q["v_scale"][0, 0]) == 3.0 and float(q["v_zero"][0, 0]) == 10.0
    assert np.array_equal(q["khat"], k4) and np.array_equal(q["vhat"], v)


def test_keys_are_grouped_per_channel_and_values_per_token():
    """Channels (for K) and tokens (for V) of very different magnitude: each must keep an error of at most half a step
    of ITS OWN range, which only the right grouping axis gives."""
    rng = np.random.default_rng(0)
    L, d, g = 192, 128, 64
    mag_c = 10.0 ** rng.uniform(-3, 3, size=d)           # per-channel magnitude of the keys
    mag_t = 10.0 ** rng.uniform(-3, 3, size=L)           # per-token magnitude of the values
    k = (rng.standard_normal((L, d)) * mag_c[None, :]).astype(np.float32)
    v = (rng.standard_normal((L, d)) * mag_t[:, None]).astype(np.float32)
    q = fo.quantize_base(k, v, bits=4, group=g, tail=0)
    for t0 in range(0, L, g):
        blk = k[t0:t0 + g]
        step = (blk.max(axis=0) - blk.min(axis=0)) / 15.0                  # per channel, over the group's tokens
        err = np.abs(q["khat"][t0:t0 + g] - blk).max(axis=0)
        assert np.all(err <= 0.5 * step * 1.01 + 1e-3 * np.abs(blk).max(axis=0)), "K error exceeds the channel's own half step"
    vb = v.reshape(L, d // g, g)
    step = (vb.max(axis=2) - vb.min(axis=2)) / 15.0                        # per token and channel group
    err = np.abs(q["vhat"].reshape(L, d // g, g) - vb).max(axis=2)
    assert np.all(err <= 0.5 * step * 1.01 + 1e-3 * np.abs(vb).max(axis=2)), "V error exceeds the token's own half step"
    assert q["k_scale"].shape == (L // g, d) and q["v_scale"].shape == (L, d // g)
    assert q["k_codes"].max() <= 15 and q["v_codes"].max() <= 15


def test_tail_rows_untouched_and_ragged_last_token_group():
    rng = np.random.default_rng(1)
    L, d, g, tail = 150, 64, 64, 20                      # 130 quantized positions: token groups of 64, 64 and 2
    k = rng.standard_normal((L, d)).astype(np.float32)
    v = rng.standard_normal((L, d)).astype(np.float32)
    q = fo.quantize_base(k, v, bits=4, group=g, tail=tail)
    assert np.array_equal(q["khat"][L - tail:], k[L - tail:]) and np.array_equal(q["vhat"][L - tail:], v[L - tail:])
    assert np.array_equal(q["k_tail"], k[L - tail:]) and q["k_codes"].shape == (130, d) and q["k_scale"].shape == (3, d)
    # the short group's range is that of its two tokens only: both are hit exactly (codes 0 and 15) up to fp16 metadata
    last = k[128:130]
    assert np.all(np.abs(q["khat"][128:130] - last) <= 2e-3 * np.abs(last).max() + 1e-6)
    # a sequence no longer than the tail is kept whole
    q2 = fo.quantize_base(k[:16], v[:16], bits=4, group=g, tail=tail)
    assert np.array_equal(q2["khat"], k[:16]) and q2["k_codes"].shape == (0, d)


def test_constant_groups_are_exact_and_storage_rounding_is_applied():
    k = np.full((64, 64), 0.75, dtype=np.float32)
    v = np.full((64, 64), -2.5, dtype=np.float32)
    q = fo.quantize_base(k, v, bits=4, group=64, tail=0, storage_round=fo.round_bf16)
    assert np.array_equal(q["khat"], k) and np.array_equal(q["vhat"], v) and not q["k_scale"].any()
    rng = np.random.default_rng(2)
    k = rng.standard_normal((64, 64)).astype(np.float32)
    q = fo.quantize_base(k, k, bits=4, group=64, tail=0, storage_round=fo.round_bf16)
    assert np.array_equal(q["khat"], fo.round_bf16(q["khat"]))             # already bf16 values
    q32 = fo.quantize_base(k, k, bits=4, group=64, tail=0)
    assert np.array_equal(q["khat"], fo.round_bf16(q32["khat"]))


def test_base_bytes_by_hand():
    # L = 128 + 64 tail, d = 128, int4, groups of 64: codes 2 * 128 * 64 B; K metadata 2 groups * 128 channels * 4 B;
    # V metadata 128 tokens * 2 groups * 4 B; tail 2 * 64 * 128 * 2 B
    assert fo.base_q_bytes(192, 128, 4, 64, 64) == 2 * 128 * 64 + 2 * 128 * 4 + 128 * 2 * 4 + 2 * 64 * 128 * 2
    # the configuration of the paper's setting at scale approaches 4.5 bits per element against 16
    full = 2 * 32768 * 2048 * 2
    assert 3.3 < full / fo.base_q_bytes(32768, 2048, 4, 64, 64) < 3.6


def test_rows_needed_by_hand():
    sets = {(0, 0): np.array([0, 2]), (0, 1): np.array([2, 5]), (1, 0): np.array([], dtype=np.int64), (1, 1): np.array([7])}
    need = fo.base_rows_needed(sets, [3, 6], H=2, L=8)
    assert np.flatnonzero(need[0]).tolist() == [0, 2, 3, 5, 6]
    assert np.flatnonzero(need[1]).tolist() == [3, 6, 7]


def test_packed_base_plus_residuals_against_the_papers_reported_reductions():
    """Table 1's peak KV reductions (5.85x and 6.06x, stored in tests/golden/kv_accounting.txt with the schedules of
    Table 6) from the oracle's own byte counts: loop 1 as the packed base (int4, groups of 64, 64-token tail), every
    later loop as residual payloads of the retained rows.  The reported figures are peaks of whole runs, a few percent
    below the steady-state count."""
    import os
    g = {}
    for line in open(os.path.join(os.path.dirname(__file__), "golden", "kv_accounting.txt")):
        line = line.split("#")[0].strip()
        if "=" in line:
            k, v = [t.strip() for t in line.split("=")]
            g[k] = [float(t) for t in v.split()]
    L, d = int(g["context"][0]), int(g["d_model"][0])
    bits, grp = int(g["quant_bits"][0]), int(g["quant_group"][0])
    for name in ("ouro14", "ouro26"):
        rho = g[name + "_tokens"]
        fl = fo.base_q_bytes(L, d, bits, grp, 64) + sum(r * L * fo.payload_bytes_per_row(d, bits, grp) for r in rho[1:])
        dense = len(rho) * 2 * L * d * 2
        rep = g[name + "_reported_reduction"][0]
        assert rep <= dense / fl <= 1.04 * rep, (name, dense / fl)
