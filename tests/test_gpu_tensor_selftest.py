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
