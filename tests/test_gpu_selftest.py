"""Hardware self-check of the sm_100a primitives (TMA tiles, swizzled descriptors, tcgen05.mma, TMEM loads)
in every operand-major combination the kernels rely on."""
import ctypes

import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("by_threads", [0, 1, 2])
@pytest.mark.parametrize("a_mn,b_mn", [(0, 0), (1, 0), (0, 1), (1, 1)])
@pytest.mark.parametrize("N,K", [(64, 64), (64, 128), (128, 64), (128, 128)])
def test_umma_product(N, K, a_mn, b_mn, by_threads):
    from paper_2606_08804_b200 import binding as qd
    if by_threads == 2 and a_mn:
        pytest.skip("an A operand in tensor memory is always row = lane, K along the columns")
    lib = qd.load()
    fn = lib.qdelta_selftest_umma
    fn.restype = ctypes.c_int
    fn.argtypes = [ctypes.c_void_p] * 3 + [ctypes.c_int] * 5 + [ctypes.c_void_p, ctypes.c_void_p]
    g = torch.Generator(device="cuda").manual_seed(N * 7 + K * 3 + a_mn * 2 + b_mn)
    A = torch.randn((K, 128) if a_mn else (128, K), device="cuda", generator=g).to(torch.bfloat16)
    B = torch.randn((K, N) if b_mn else (N, K), device="cuda", generator=g).to(torch.bfloat16)
    D = torch.full((128, N), float("nan"), device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rc = fn(A.data_ptr(), B.data_ptr(), D.data_ptr(), N, K, a_mn, b_mn, by_threads, status.data_ptr(),
            torch.cuda.current_stream().cuda_stream)
    assert rc == 0, qd.status_string(rc)
    torch.cuda.synchronize()
    assert status.item() == 0, "bounded wait expired"
    Aop = A.float().t() if a_mn else A.float()          # [128, K]
    Bop = B.float().t() if b_mn else B.float()          # [N, K]
    ref = Aop.double() @ Bop.double().t()
    err = (D.double() - ref).abs().max().item() / ref.abs().max().item()
    assert err < 1e-5, err
