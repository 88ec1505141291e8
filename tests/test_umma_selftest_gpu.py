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


def test_a_wait_that_runs_out_is_reported_and_the_context_survives():
    """Failure detection without a fault: a bounded wait on a barrier that nothing arrives at gives up after about two
    seconds, the kernel ends normally, swila_device_status reports it once, and the next launch works."""
    import ctypes
    import time

    from paper_2609_39034_b200 import binding, workloads as wl

    binding.device_status()  # clean before
    gave_up = torch.zeros(1, device="cuda", dtype=torch.int32)
    t0 = time.time()
    binding.check(binding.lib.swila_selftest_wait_timeout(ctypes.c_void_p(gave_up.data_ptr()),
                                                          ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)))
    torch.cuda.synchronize()
    assert 1.5 < time.time() - t0 < 10.0
    assert int(gave_up.item()) == 1
    with pytest.raises(binding.SwilaError) as e:
        binding.device_status()
    assert e.value.status == binding.ERR_CUDA and "bounded wait" in str(e.value)
    binding.device_status()  # reported once, then clean again
    w = wl.CONFIGS[1].with_(B=1, H=1, T=64)  # and the context still runs kernels
    inp = wl.make_inputs(w, device="cuda")
    o = binding.swila_forward(w, inp, state_in=None, state_out=None, algo=binding.ALGO_CHUNK)
    torch.cuda.synchronize()
    binding.device_status()
    assert bool(torch.isfinite(o.float()).all())
