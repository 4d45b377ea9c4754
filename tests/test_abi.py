"""Host-side checks that need no GPU: the shared library loads, exports every symbol the header
declares, and rejects bad arguments before anything is launched."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2609_29812_b200 import build
    build.build()
    from paper_2609_29812_b200 import binding
    return binding


def declared_functions():
    text = open(os.path.join(ROOT, "include", "flashloop.h")).read()
    return sorted(set(re.findall(r"FL_API\s+[\w\s\*]+?\b(fl_\w+)\s*\(", text)))


def test_library_exports_every_declared_symbol(B):
    names = declared_functions()
    assert len(names) >= 12 and "fl_loop_attention" in names and "fl_select_tokens" in names
    for n in names:
        assert hasattr(B.lib, n), n
    assert B.lib.fl_version() >= 100
    assert B.status_string(0) == "ok" and "invalid" in B.status_string(B.FL_ERR_INVALID_ARG)


def good_shape(B, **kw):
    base = dict(L=1024, n_heads=2, head_dim=128, dtype=B.FL_BF16, q_block=256, bits=4, group=128, eps=1e-6,
                sm_scale=128 ** -0.5)
    base.update(kw)
    return B.make_shape(**base)


def fake_store(B, n_streams=1, n_rows=16, **over):
    s = dict(codes=0x1000, scale=0x2000, zero=0x3000, slot_of_pos=0x4000, n_rows=n_rows)
    s.update(over)
    return B.make_store(0x10000, 0x20000, [s] * n_streams, [s] * n_streams)


def test_argument_validation_happens_before_any_launch(B):
    """There is no GPU here: any launch or CUDA call would yield FL_ERR_CUDA, so getting the
    argument errors proves the checks come first."""
    ctx = C.cast(C.create_string_buffer(256), C.c_void_p)     # opaque stand-in, never dereferenced on these paths
    P = 0x100000                                              # a 16-byte aligned non-null "device pointer"
    INV, UNS = B.FL_ERR_INVALID_ARG, B.FL_ERR_UNSUPPORTED
    sh = good_shape(B)
    call = dict(check=False, stream=0)
    # null context / shape fields
    assert B.fl_select_tokens(None, sh, 2, P, P, None, 1024, 10, P, P, P, **call) == INV
    for bad in (dict(L=0), dict(n_heads=0), dict(q_block=0), dict(bits=3), dict(bits=0), dict(group=48),
                dict(group=64, head_dim=128, bits=5), dict(dtype=7), dict(sm_scale=0.0), dict(eps=-1.0)):
        assert B.fl_select_tokens(ctx, good_shape(B, **bad), 2, P, P, None, 1024, 10, P, P, P, **call) == INV, bad
    assert B.fl_select_tokens(ctx, good_shape(B, head_dim=96, group=32), 2, P, P, None, 1024, 10, P, P, P, **call) == UNS
    assert B.fl_select_tokens(ctx, good_shape(B, head_dim=128, group=256), 2, P, P, None, 1024, 10, P, P, P, **call) == INV
    # fl_select_tokens
    assert B.fl_select_tokens(ctx, sh, 1, P, P, None, 1024, 10, P, P, P, **call) == INV        # loop_r < 2
    assert B.fl_select_tokens(ctx, sh, 2, None, P, None, 1024, 10, P, P, P, **call) == INV
    assert B.fl_select_tokens(ctx, sh, 2, P, P, None, 1024, 0, P, P, P, **call) == INV         # k < 1
    assert B.fl_select_tokens(ctx, sh, 2, P, P, None, 512, 10, P, P, P, **call) == INV         # cand NULL needs n_cand == L
    assert B.fl_select_tokens(ctx, sh, 2, P, P, P, 2048, 10, P, P, P, **call) == INV           # n_cand > L
    assert B.fl_select_tokens(ctx, sh, 2, P + 4, P, None, 1024, 10, P, P, P, **call) == INV    # misaligned
    # gather / scatter
    assert B.fl_gather_rows(ctx, P, P, 4, 100, P, **call) == INV                               # row_bytes % 16
    assert B.fl_gather_rows(ctx, P, P, -1, 64, P, **call) == INV
    assert B.fl_gather_rows(ctx, None, P, 4, 64, P, **call) == INV
    assert B.fl_scatter_update(ctx, P, P, 4, 64, P + 8, **call) == INV
    assert B.fl_gather_rows(ctx, P, P, 0, 64, P, **call) == B.FL_OK                            # empty is a no-op
    # projection of the active rows
    pr = lambda **kw: B.fl_project_rows(ctx, kw.get("x", P), kw.get("xr", 1024), kw.get("si", P), kw.get("n", 16),
                                        kw.get("din", 256), kw.get("w", P + 0x100000), kw.get("dout", 512),
                                        kw.get("y", P + 0x200000), kw.get("yr", 1024), kw.get("di", None),
                                        kw.get("acc", 0), **call)
    assert pr(x=None) == INV and pr(w=None) == INV and pr(y=None) == INV and pr(n=-1) == INV and pr(acc=2) == INV
    assert pr(x=P + 4) == INV and pr(y=P) == INV                         # misaligned; y aliases x
    assert pr(si=None, n=2000) == INV and pr(di=None, n=2000, yr=100) == INV   # no index list: n must fit the matrix
    assert pr(din=100) == UNS and pr(dout=100) == UNS
    assert pr(n=0) == B.FL_OK
    assert pr() == UNS                                                   # the stand-in context has no tensor path
    st = fake_store(B)
    pq = lambda **kw: B.fl_project_qkv_quant(ctx, kw.get("sh", sh), kw.get("r", 2), kw.get("x", P), 1024, P,
                                             kw.get("n", 16), P + 0x100000, kw.get("q", P + 0x200000), None,
                                             kw.get("st", st), **call)
    assert pq(r=1) == INV and pq(r=3) == INV and pq(n=17) == INV and pq(st=None) == INV and pq(x=None) == INV
    assert pq(q=None) == INV and pq(x=P + 4) == INV
    assert pq(sh=good_shape(B, dtype=B.FL_F32)) == UNS and pq(sh=good_shape(B, bits=16)) == UNS
    assert pq(sh=good_shape(B, n_heads=1)) == UNS                                               # d = 128
    assert pq(n=0, st=fake_store(B, n_rows=0)) == B.FL_OK
    assert pq() == UNS                                                   # the stand-in context has no tensor path
    # quantizer
    st = fake_store(B)
    assert B.fl_quant_kv_residual(ctx, sh, 1, P, P, P, 16, st, **call) == INV                  # loop_r < 2
    assert B.fl_quant_kv_residual(ctx, sh, 3, P, P, P, 16, st, **call) == INV                  # needs 2 streams
    assert B.fl_quant_kv_residual(ctx, sh, 2, P, P, P, 17, st, **call) == INV                  # n_rows mismatch
    assert B.fl_quant_kv_residual(ctx, sh, 2, None, P, P, 16, st, **call) == INV
    assert B.fl_quant_kv_residual(ctx, sh, 2, P, P, P, 16, None, **call) == INV
    assert B.fl_quant_kv_residual(ctx, sh, 2, P, P, P, 16, fake_store(B, scale=None), **call) == INV
    assert B.fl_quant_kv_residual(ctx, sh, 2, P, P, P, 16, fake_store(B, slot_of_pos=None), **call) == INV
    assert B.fl_quant_kv_residual(ctx, sh, 2, P, P, P, 16, fake_store(B, codes=0x1004), **call) == INV
    assert B.fl_quant_kv_residual(ctx, sh, 2, P, P, P, 0, fake_store(B, n_rows=0), **call) == B.FL_OK
    assert B.fl_quant_kv_residual(ctx, good_shape(B, n_heads=1), 2, P, P, P, 16, st, **call) == UNS   # d = 128
    # dense loop / column selection / loop attention
    assert B.fl_dense_loop_attention(ctx, sh, P, P, None, P, P, None, **call) == INV
    assert B.fl_dense_loop_attention(ctx, sh, P, P, P, P, None, P, **call) == INV              # col_scores needs lse
    assert B.fl_select_columns(ctx, sh, P, None, None, 1024, 0, P, P, **call) == INV           # c < 1
    assert B.fl_select_columns(ctx, sh, P, None, None, 512, 8, P, P, **call) == INV            # dense stride != L
    assert B.fl_select_columns(ctx, sh, P, P, None, 64, 8, P, P, **call) == INV                # cand_cnt missing
    la = lambda **kw: B.fl_loop_attention(ctx, kw.get("sh", sh), kw.get("r", 2), kw.get("q", P), P, P,
                                          kw.get("n", 16), kw.get("st", st), kw.get("ci", P), P, kw.get("c", 64),
                                          P, P, P, P, None, **call)
    assert la(r=1) == INV and la(c=0) == INV and la(q=None) == INV and la(ci=None) == INV
    assert la(r=3) == INV and la(st=None) == INV and la(n=-1) == INV and la(n=4096) == INV
    # the carried old term of the indexed form
    idx = lambda carry, **kw: B.fl_loop_attention_indexed_carry(
        ctx, sh, 2, P, kw.get("qs", P), P, P, 16, st, P, P, 64, kw.get("lse", P), P, kw.get("o", P + 0x1000),
        P + 0x2000, carry, None, **call)
    assert idx(B.make_carry(None, P, False)) == INV and idx(B.make_carry(P + 0x4000, None, True)) == INV
    assert idx(B.make_carry(P + 0x2000, P, False)) == INV                                      # background = O store
    assert idx(B.make_carry(P + 0x4004, P, False)) == INV                                      # misaligned
    assert idx(B.make_carry(P + 0x4000, P, False), qs=None) == INV         # recomputing needs the previous Q rows
    # a reusing call needs none of the previous loop's rows: the checks pass and the stand-in context, which has no
    # tensor path, answers "unsupported"
    assert idx(B.make_carry(P + 0x4000, P, True), qs=None, lse=None, o=None) == UNS
    # sparse decode attention
    dec = lambda **kw: B.fl_decode_attention(ctx, sh, kw.get("r", 2), kw.get("q", P), P, kw.get("n", 4), kw.get("st", st),
                                             kw.get("ci", P), P, kw.get("c", 64), P, P, P, P, None, **call)
    assert dec(r=1) == INV and dec(c=0) == INV and dec(q=None) == INV and dec(ci=None) == INV and dec(st=None) == INV
    assert dec(n=-1) == INV and dec(r=3) == INV and dec(n=0) == B.FL_OK
    # quantized base
    bq = lambda **kw: B.make_base_q(kw.get("kc", P), P, P, P, P, P, kw.get("kt", P), P, kw.get("g", 64), kw.get("t", 64))
    qb = lambda base, k=P: B.fl_quant_kv_base(ctx, kw_sh.get("sh", sh), k, P, base, **call)
    kw_sh = {}
    assert qb(bq(g=48)) == INV and qb(bq(t=-1)) == INV and qb(bq(kc=None)) == INV and qb(bq(kt=None)) == INV
    assert qb(bq(kc=P + 4)) == INV and qb(None) == INV and qb(bq(), k=None) == INV
    kw_sh["sh"] = good_shape(B, bits=16)
    assert qb(bq()) == UNS
    kw_sh["sh"] = good_shape(B, n_heads=1)
    assert qb(bq()) == UNS                                                                     # d = 128
    assert B.fl_dequant_kv_base(ctx, sh, bq(), None, P, **call) == INV
    assert B.fl_kv_base_q_bytes(good_shape(B, L=192, n_heads=2, head_dim=64, group=64), 64, 64) == \
        2 * 128 * 64 + 2 * 128 * 4 + 128 * 2 * 4 + 2 * 64 * 128 * 2
    # accounting
    rc = B.lib.fl_kv_store_bytes(C.byref(sh), C.byref(st), 3, 1, C.byref(C.c_int64()), C.byref(C.c_int64()))
    assert rc == INV                                                                          # only one stream


def test_kv_store_bytes_matches_closed_form(B):
    from paper_2609_29812_b200 import workloads
    w = workloads.config3()
    sh = B.make_shape(w.L, w.n_heads, w.head_dim, B.FL_BF16, w.q_block, w.bits, w.group, w.eps, w.sm_scale)
    st = fake_store(B, n_streams=3, n_rows=w.k_tokens)
    fl, dense = B.fl_kv_store_bytes(sh, st, 4, w.n_layers)
    assert dense == 4 * 2 * w.L * w.d * 2 and dense * w.n_layers == 48 * 2 ** 30       # the 48 GiB example
    pay = 2 * (w.d // 2 + 4 * (w.d // 128))
    expect = 2 * w.L * w.d * 2 + 3 * (w.k_tokens * pay + -(-4 * (w.L + w.k_tokens) // w.n_layers))
    assert fl == expect and dense / fl > 3.0
    fl16, _ = B.fl_kv_store_bytes(B.make_shape(w.L, 16, 128, B.FL_BF16, 1024, 16, 128, 1e-6, 0.1), st, 4, 1)
    assert fl16 == 2 * w.L * w.d * 2 + 3 * (w.k_tokens * 2 * w.d * 2 + 4 * (w.L + w.k_tokens))
