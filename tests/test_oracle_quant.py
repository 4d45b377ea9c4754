"""Pins for the oracle's residual codec (Section 4.3, Appendix D.3, Appendix E quantizer) and
the KV-cache accounting."""
import os

import numpy as np
import pytest

from oracle import flashloop_oracle as fo
from paper_2609_29812_b200 import workloads

F32 = np.float32


def test_worked_examples_by_hand():
    # 16 integers 0..15 at 4 bits: offset 0, range 15, scale 1, codes are the values themselves
    d = np.arange(16, dtype=F32)[None, :]
    codes, s, z = fo.quantize_groups(d, 4, 16)
    assert z[0, 0] == 0 and s[0, 0] == 1 and codes[0].tolist() == list(range(16))
    assert np.array_equal(fo.dequantize_groups(codes, s, z, 16), d)
    # half-way cases round to the even code: (x - 0)/1 = 0.5, 1.5, 2.5, 3.5 -> 0, 2, 2, 4
    d = np.array([[0, 0.5, 1.5, 2.5, 3.5, 15, 7, 7]], dtype=F32)
    codes, s, z = fo.quantize_groups(d, 4, 8)
    assert s[0, 0] == 1 and codes[0].tolist() == [0, 0, 2, 2, 4, 15, 7, 7]
    # offset is rounded DOWN to fp16, scale UP: group min 0.1 (not an fp16 number)
    d = np.array([[0.1, 0.2, 0.3, 0.4]], dtype=F32)
    codes, s, z = fo.quantize_groups(d, 2, 4)
    assert float(z[0, 0]) == 0.0999755859375                      # fp16 neighbour below 0.1
    assert float(z[0, 0]) <= 0.1 < float(np.nextafter(z[0, 0], np.float16(1)))
    ratio = (F32(0.4) - F32(z[0, 0])) / F32(3)
    assert float(s[0, 0]) >= float(ratio) > float(np.nextafter(s[0, 0], np.float16(0)))
    assert codes[0].tolist() == [0, 1, 2, 3]
    # negative groups and the two-level case at 2 bits
    d = np.array([[-3, -3, 0, 0]], dtype=F32)
    codes, s, z = fo.quantize_groups(d, 2, 4)
    assert z[0, 0] == -3 and s[0, 0] == 1 and codes[0].tolist() == [0, 0, 3, 3]


def test_constant_group_is_exact_when_representable():
    d = np.full((3, 32), 0.75, dtype=F32)
    codes, s, z = fo.quantize_groups(d, 4, 16)
    assert np.all(s == 0) and np.all(codes == 0) and np.all(z == np.float16(0.75))
    assert np.array_equal(fo.dequantize_groups(codes, s, z, 16), d)
    d0 = np.zeros((2, 16), dtype=F32)
    codes, s, z = fo.quantize_groups(d0, 8, 16)
    assert np.all(fo.dequantize_groups(codes, s, z, 16) == 0)


@pytest.mark.parametrize("bits", [2, 4, 8])
@pytest.mark.parametrize("group", [16, 64, 128])
def test_half_step_bound_codes_in_range_and_monotone(bits, group):
    rng = np.random.default_rng(bits * 100 + group)
    for mag, shift in [(1.0, 0.0), (1e-3, 0.0), (0.05, 30.0), (5.0, -200.0), (1e-6, 1.0)]:
        d = (rng.standard_normal((64, 128)) * mag + shift).astype(F32)
        codes, s, z = fo.quantize_groups(d, bits, group)
        deq = fo.dequantize_groups(codes, s, z, group)
        sf = np.repeat(s.astype(np.float64), group, axis=-1)
        zf = np.repeat(z.astype(np.float64), group, axis=-1)
        ulp = np.spacing((np.abs(d) + np.abs(zf)).astype(F32)).astype(np.float64)
        assert np.all(np.abs(d.astype(np.float64) - deq) <= sf / 2 + 4 * ulp)
        assert codes.max() <= 2 ** bits - 1
        g = d.reshape(64, 128 // group, group)
        cg = codes.reshape(g.shape)
        # codes are monotone in the values; the minimum takes code 0 whenever the fp16 offset
        # equals it (an offset rounded down below the minimum may leave code 0 unused)
        order = np.argsort(g, axis=-1, kind="stable")
        assert np.all(np.diff(np.take_along_axis(cg.astype(int), order, -1), axis=-1) >= 0)
        exact = z.astype(np.float64) == g.min(-1)
        assert np.all(np.take_along_axis(cg, g.argmin(-1)[..., None], -1)[..., 0][exact] == 0)
        # the representable interval covers the group: offset <= min and offset + qmax*scale >= max
        assert np.all(z.astype(np.float64) <= g.min(-1))
        assert np.all(z.astype(np.float64) + (2 ** bits - 1) * s.astype(np.float64) >= g.max(-1))


def test_pack_layout_and_roundtrip():
    assert fo.pack_codes(np.array([1, 2, 3, 4], np.uint8), 4).tolist() == [0x21, 0x43]
    assert fo.pack_codes(np.array([1, 2, 3, 0, 3, 3, 0, 0], np.uint8), 2).tolist() == [0b00111001, 0b00001111]
    assert fo.pack_codes(np.array([200, 7], np.uint8), 8).tolist() == [200, 7]
    rng = np.random.default_rng(0)
    for bits in (2, 4, 8):
        c = rng.integers(0, 2 ** bits, size=(5, 3, 64)).astype(np.uint8)
        assert np.array_equal(fo.unpack_codes(fo.pack_codes(c, bits), bits), c)
        assert fo.pack_codes(c, bits).shape == (5, 3, 64 * bits // 8)


def test_residual_recurrence_error_does_not_accumulate():
    """Closed loop of Eq. 4: |X^(r) - Xhat^(r)| <= scale_r / 2 for active rows at every loop;
    inactive rows are bit-identical to the previous loop."""
    rng = np.random.default_rng(11)
    L, H, dh, g = 40, 2, 128, 64
    x = rng.standard_normal((L, H, dh)).astype(F32)
    xhat = x.copy()
    active = np.sort(rng.permutation(L)[:15])
    for r in range(2, 7):
        x = (x + 0.05 * rng.standard_normal(x.shape)).astype(F32)
        prev = xhat
        xhat, pay = fo.residual_update(x[active], prev, active, 4, g)
        inactive = np.setdiff1d(np.arange(L), active)
        assert np.array_equal(xhat[inactive], prev[inactive])
        s = np.repeat(pay["scale"].astype(np.float64), g, axis=-1)
        err = np.abs(x[active].astype(np.float64) - xhat[active])
        assert np.all(err <= s / 2 + 1e-6)
        active = active[: len(active) - 2]                         # nested, shrinking
    # codec off: the new rows are stored as they are
    xh16, pay16 = fo.residual_update(x[active], prev, active, 16, g)
    assert np.array_equal(xh16[active], x[active])


def test_residual_beats_full_state_quantization_when_updates_are_small():
    """Section 3.3: at equal bit width the residual codec reconstructs better than quantizing the
    full state, when the cross-loop change is small next to the state."""
    rng = np.random.default_rng(12)
    x1 = rng.standard_normal((32, 1, 128)).astype(F32)
    x2 = (x1 + 0.05 * rng.standard_normal(x1.shape)).astype(F32)
    act = np.arange(32)
    xhat_res, _ = fo.residual_update(x2, x1, act, 4, 64)
    c, s, z = fo.quantize_groups(x2, 4, 64)
    xhat_full = fo.dequantize_groups(c, s, z, 64)
    assert np.linalg.norm(xhat_res - x2) < 0.2 * np.linalg.norm(xhat_full - x2)


def _golden():
    out = {}
    path = os.path.join(os.path.dirname(__file__), "golden", "kv_accounting.txt")
    for line in open(path):
        line = line.split("#")[0].strip()
        if "=" in line:
            k, v = [t.strip() for t in line.split("=")]
            out[k] = [float(t) for t in v.split()]
    return out


def test_kv_accounting_against_the_papers_figures():
    g = _golden()
    L, d, R, N = int(g["context"][0]), int(g["d_model"][0]), int(g["loops"][0]), int(g["layers"][0])
    _, dense = fo.kv_bytes_per_token_layer(L, d, [L] * (R - 1), 16, 128, N)
    assert dense * L * N / 2 ** 30 == g["dense_kv_gib_32k"][0]                 # 48 GiB, Section 1
    # INT4, group 64, fp16 scale + offset: 4.5 bits per element
    bits, grp = int(g["quant_bits"][0]), int(g["quant_group"][0])
    assert fo.payload_bytes_per_row(d, bits, grp) * 8 / (2 * d) == 4.5
    # paper schedules: reduction if every loop (base included) were stored at 4.5 bits,
    # 16 R / (4.5 sum_r rho_r); the reported peak-memory figures are a few percent lower
    for name in ("ouro14", "ouro26"):
        rho = g[name + "_tokens"]
        ratio = 16 * len(rho) / (4.5 * sum(rho))
        rep = g[name + "_reported_reduction"][0]
        assert rep <= ratio <= 1.04 * rep
    # this build's layout at the 32K configuration: bf16 base + int4 g=128 residuals of 10% rows
    w = workloads.config3()
    fl, dense = fo.kv_bytes_per_token_layer(w.L, w.d, [w.k_tokens] * 3, w.bits, w.group, w.n_layers)
    assert dense == 32768 and 8840 < fl < 8850 and dense / fl > 3.0


def test_bf16_rounding_helper():
    """round_bf16: exact on bf16 values, ties to even, nearest otherwise (checked against torch)."""
    torch = pytest.importorskip("torch")
    x = np.array([1.0, 1.00390625, 1.01171875, -3.14159, 1e-30, 65504.0, 0.1], dtype=np.float32)
    # 1 + 2^-8 is a tie between 1 and 1 + 2^-7 -> even mantissa (1.0); 1 + 3*2^-8 ties up to 1 + 2^-6
    got = fo.round_bf16(x)
    assert got[0] == 1.0 and got[1] == 1.0 and got[2] == np.float32(1.015625)
    ref = torch.from_numpy(x).to(torch.bfloat16).float().numpy()
    assert np.array_equal(got, ref)
    r = np.random.default_rng(0).standard_normal(10000).astype(np.float32) * 37
    assert np.array_equal(fo.round_bf16(r), torch.from_numpy(r).to(torch.bfloat16).float().numpy())
