"""Checks the tensor-path building blocks (shared-memory operand layouts, matrix and instruction
descriptors, tensor-memory loads and stores) on a single tile against plain matrix products."""
import ctypes as C
import os

import numpy as np
import pytest

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def test_umma_tile_products_match_matmul():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_29812_b200 import build
    assert os.path.exists(build.SELFTEST_LIB_PATH), "self-test library not built"
    lib = C.CDLL(build.SELFTEST_LIB_PATH)
    lib.fl_selftest_umma.argtypes = [C.c_void_p] * 7
    lib.fl_selftest_umma.restype = C.c_int
    g = torch.Generator(device="cpu").manual_seed(1)
    q = torch.randn(128, 128, generator=g).to(torch.bfloat16).cuda()
    k = torch.randn(64, 128, generator=g).to(torch.bfloat16).cuda()
    v = torch.randn(64, 128, generator=g).to(torch.bfloat16).cuda()
    s_out = torch.zeros(128, 64, dtype=torch.float32, device="cuda")
    o_out = torch.zeros(128, 128, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rc = lib.fl_selftest_umma(q.data_ptr(), k.data_ptr(), v.data_ptr(), s_out.data_ptr(), o_out.data_ptr(),
                              status.data_ptr(), None)
    assert rc == 0
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "a bounded wait ran out"
    s_ref = q.double() @ k.double().T
    np.testing.assert_allclose(s_out.cpu().numpy(), s_ref.cpu().numpy(), rtol=1e-4, atol=1e-3)
    p = s_out.to(torch.bfloat16).double()
    o_ref = p @ v.double()
    np.testing.assert_allclose(o_out.cpu().numpy(), o_ref.cpu().numpy(), rtol=1e-3, atol=5e-2)


def test_tma_row_gather_feeds_the_tensor_core():
    """tile::gather4 row gather into a swizzled operand tile, including an out-of-range row (zero fill)."""
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_29812_b200 import build
    lib = C.CDLL(build.SELFTEST_LIB_PATH)
    lib.fl_selftest_gather4.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.fl_selftest_gather4.restype = C.c_int
    g = torch.Generator(device="cpu").manual_seed(2)
    rows = 1000
    base = torch.randn(rows, 128, generator=g).to(torch.bfloat16).cuda()
    q = torch.randn(128, 128, generator=g).to(torch.bfloat16).cuda()
    idx = torch.randperm(rows, generator=g)[:64].to(torch.int32)
    idx[5] = rows                      # out of range: must read as a zero row
    idx[63] = 0
    idx_d = idx.cuda()
    s_out = torch.zeros(128, 64, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rc = lib.fl_selftest_gather4(base.data_ptr(), rows, q.data_ptr(), idx_d.data_ptr(), s_out.data_ptr(),
                                 status.data_ptr(), None)
    assert rc == 0
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    kg = torch.zeros(64, 128, dtype=torch.float64)
    for t, j in enumerate(idx.tolist()):
        if j < rows:
            kg[t] = base[j].double().cpu()
    s_ref = q.double().cpu() @ kg.T
    np.testing.assert_allclose(s_out.cpu().numpy(), s_ref.numpy(), rtol=1e-4, atol=1e-3)


def test_bounded_wait_runs_out_and_reports_a_timeout():
    """A wait on a barrier that nothing completes gives up after its poll limit, the kernel reports FL_ERR_TIMEOUT
    through the status word and returns; the context stays usable (a normal launch right after works)."""
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_29812_b200 import binding as B, build
    lib = C.CDLL(build.SELFTEST_LIB_PATH)
    lib.fl_selftest_timeout.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
    lib.fl_selftest_timeout.restype = C.c_int
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    gave_up = torch.zeros(1, dtype=torch.int32, device="cuda")
    assert lib.fl_selftest_timeout(status.data_ptr(), gave_up.data_ptr(), None) == 0
    torch.cuda.synchronize()
    assert int(gave_up.item()) == 1
    assert int(status.item()) == B.FL_ERR_TIMEOUT
    assert "wait" in B.status_string(int(status.item()))
    x = torch.arange(8, device="cuda")
    assert int((x + 1).sum().item()) == 36
