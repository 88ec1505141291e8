"""GPU: the tcgen05 building blocks of the chunked kernel (tensor-memory allocation and moves,
TF32 MMA with A in tensor memory and B in shared memory, mbarrier completion) reproduce a plain
matrix product."""
import pytest
import torch

pytestmark = pytest.mark.gpu


def _tf32(x: torch.Tensor) -> torch.Tensor:
    """Keep the 10 explicit mantissa bits TF32 has, so products are exact in fp32."""
    return (x.view(torch.int32) & ~0x1FFF).view(torch.float32)


@pytest.mark.parametrize("N,K", [(32, 32), (128, 32), (32, 128), (64, 128)])
def test_tf32_mma_matches_matmul(N, K):
    assert torch.cuda.is_available()
    from paper_2609_39034_b200 import binding

    g = torch.Generator(device="cuda").manual_seed(N * 1000 + K)
    A = _tf32(torch.randn((128, K), device="cuda", generator=g))
    B = _tf32(torch.randn((N, K), device="cuda", generator=g))
    D = binding.selftest_tf32_mma(A, B)
    ref = A.double() @ B.double().T
    err = float((D.double() - ref).abs().max() / ref.abs().max())
    assert err < 1e-5, err


@pytest.mark.parametrize("N,K,a_in_smem", [(64, 128, 0), (128, 32, 0), (32, 32, 0), (64, 64, 1), (64, 64, 2), (32, 64, 2), (128, 32, 3)])
def test_bf16_mma_matches_matmul(N, K, a_in_smem):
    assert torch.cuda.is_available()
    from paper_2609_39034_b200 import binding

    g = torch.Generator(device="cuda").manual_seed(N * 1000 + K + 7)
    A = torch.randn((128, K), device="cuda", generator=g)
    B = torch.randn((N, K), device="cuda", generator=g)
    D = binding.selftest_bf16_mma(A, B, a_in_smem)
    ref = A.bfloat16().double() @ B.bfloat16().double().T  # the kernel rounds to bf16 the same way
    err = float((D.double() - ref).abs().max() / ref.abs().max())
    assert err < 1e-5, err
