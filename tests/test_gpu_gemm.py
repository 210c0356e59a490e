"""The tensor-core GEMM building block (C = A B^T, bf16 operands, fp32 accumulation) against the plain
definition evaluated in float64 on the same bf16 values: several tiles, ragged edges, a channel count
that is not a multiple of the 64-channel stage, and strided operands."""
import numpy as np
import pytest
import torch

import paper_2501_10054_b200 as T

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("M,N,K", [(1, 32, 64), (200, 300, 136), (128, 256, 64), (257, 4544, 4544), (1024, 2048, 4096), (64, 16384, 512)])
def test_gemm_matches_definition(M, N, K):
    g = torch.Generator(device="cuda").manual_seed(M * 7 + N * 3 + K)
    A = torch.randn(M, K, generator=g, device="cuda").bfloat16()
    B = (torch.randn(N, K, generator=g, device="cuda") * 0.05).bfloat16()
    C = torch.full((M, N), float("nan"), device="cuda")
    T.tardis_gemm_bf16(A, B, C)
    torch.cuda.synchronize()
    ref = A.double().cpu().numpy() @ B.double().cpu().numpy().T
    got = C.double().cpu().numpy()
    assert np.isfinite(got).all()
    # exact products, fp32 accumulation: error well below K * 2^-23 * sum |a b|
    bound = (np.abs(A.double().cpu().numpy()) @ np.abs(B.double().cpu().numpy()).T) * K * 2.0 ** -23
    assert (np.abs(got - ref) <= bound + 1e-30).all()
    assert np.abs(got - ref).max() <= 2e-3 * np.abs(ref).max()


def test_gemm_strided_operands_and_output():
    g = torch.Generator(device="cuda").manual_seed(5)
    Abig = torch.randn(150, 512, generator=g, device="cuda").bfloat16()
    Bbig = torch.randn(90, 512, generator=g, device="cuda").bfloat16()
    A, B = Abig[:, 64:64 + 200], Bbig[:, 8:8 + 200]          # leading dimension 512, 16-byte aligned starts
    Cbig = torch.zeros(150, 128, device="cuda")
    C = Cbig[:, :90]
    T.tardis_gemm_bf16(A, B, C)
    torch.cuda.synchronize()
    ref = A.double().cpu().numpy() @ B.double().cpu().numpy().T
    assert np.abs(C.double().cpu().numpy() - ref).max() <= 1e-3 * np.abs(ref).max()
    assert (Cbig[:, 90:] == 0).all()


def test_gemm_argument_errors():
    lib = T.load_library()
    A = torch.zeros(8, 64, device="cuda", dtype=torch.bfloat16)
    C = torch.zeros(8, 8, device="cuda")
    assert lib.tardis_gemm_bf16(8, 8, 60, A.data_ptr(), 64, A.data_ptr(), 64, C.data_ptr(), 8, None) == 1   # K % 8
    assert lib.tardis_gemm_bf16(8, 8, 64, A.data_ptr() + 2, 64, A.data_ptr(), 64, C.data_ptr(), 8, None) == 1
    assert lib.tardis_gemm_bf16(8, 8, 64, A.data_ptr(), 64, A.data_ptr(), 64, C.data_ptr(), 4, None) == 1   # ldc < N
    assert lib.tardis_gemm_bf16(0, 8, 64, A.data_ptr(), 64, A.data_ptr(), 64, C.data_ptr(), 8, None) == 1
