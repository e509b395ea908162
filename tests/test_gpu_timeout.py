"""The way out of an expired device-side wait, exercised without a fault, a trap or an unbounded loop.

Every wait of the matmul kernels is bounded: when its limit passes, the waiting thread raises the CTA's abort flag,
every role leaves its loop, the kernel writes BITLINEAR_ERR_TIMEOUT into the workspace's status word, gives copies in
flight time to land, releases tensor memory and RETURNS.  The test hook bitlinear_test_expire_next_wait shortens the
limit of the next matmul launch to two milliseconds and makes one producer thread of its first CTA leave out one
barrier arrival together with the copy it announces (nothing is left in flight), on a problem of one CTA.  Checked: the call returns, the
status word says timeout, and the SAME workspace gives the oracle's bits on the next, ordinary call.
"""
import numpy as np
import pytest
import torch

from conftest import torch_bf16_to_bits
from paper_2402_17764_b200 import binding as B
from paper_2402_17764_b200 import synthetic as S

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    from paper_2402_17764_b200 import build
    build.build()
    B.load_library()
    yield
    B.test_expire_next_wait(0, False)  # nothing stays armed
    torch.cuda.synchronize()


# (M, K, N, kernel that runs): all of them one CTA
CASES = [(1, 128, 64, "decode_mma_kernel"), (12, 128, 512, "decode_wide_kernel"),
         (40, 128, 256, "decode_tc_kernel"), (100, 128, 256, "prefill_gemm_kernel, one token tile"),
         (200, 128, 256, "prefill_gemm_kernel, two token tiles")]


@pytest.mark.parametrize("M,K,N,kernel", CASES)
def test_expired_wait_ends_the_kernel_with_a_status(oracle, M, K, N, kernel):
    W = S.latent_weights(N, K, 3)
    X = S.activations(M, K, 3, outlier_frac=0.02, outlier_scale=10.0)
    T_ref, g_ref = oracle.quantize_weights(W.numpy())
    want = oracle.forward(T_ref, g_ref, torch_bf16_to_bits(X))
    packed, gamma = B.quantize_weights(W.cuda())
    Xd = X.cuda()
    ws = B.alloc_workspace(M, N, K)
    Y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")

    B.forward(packed, gamma, Xd, N, Y=Y, workspace=ws)           # an ordinary call first
    assert B.poll_status(ws) == B.OK
    assert np.array_equal(torch_bf16_to_bits(Y), want)

    B.test_expire_next_wait(2000, True)                          # 2 ms; one arrival left out
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    B.forward(packed, gamma, Xd, N, Y=Y, workspace=ws)           # returns: the kernel gives up by itself
    end.record()
    assert B.poll_status(ws) == B.ERR_TIMEOUT, f"{kernel}: the wait did not run out"
    assert 1.5 < start.elapsed_time(end) < 500.0                 # about the limit plus the 0.2 ms for copies in flight

    for _ in range(2):                                           # the same workspace, ordinary calls again
        Y.zero_()
        B.forward(packed, gamma, Xd, N, Y=Y, workspace=ws)
        assert B.poll_status(ws) == B.OK
        assert np.array_equal(torch_bf16_to_bits(Y), want), f"{kernel}: wrong result after an expired wait"


def test_the_hook_arms_one_launch_only(oracle):
    M, K, N = 1, 128, 64
    W = S.latent_weights(N, K, 4)
    X = S.activations(M, K, 4).cuda()
    packed, gamma = B.quantize_weights(W.cuda())
    ws = B.alloc_workspace(M, N, K)
    B.test_expire_next_wait(2000, True)
    B.forward(packed, gamma, X, N, workspace=ws)
    assert B.poll_status(ws) == B.ERR_TIMEOUT
    B.forward(packed, gamma, X, N, workspace=ws)
    assert B.poll_status(ws) == B.OK
    # a short limit alone (no arrival left out) changes nothing: no legitimate wait lasts 50 ms
    B.test_expire_next_wait(50000, False)
    B.forward(packed, gamma, X, N, workspace=ws)
    assert B.poll_status(ws) == B.OK


def test_validate_packed_finds_the_unused_code(oracle):
    N, K = 48, 144
    W = S.latent_weights(N, K, 5)
    packed, _ = B.quantize_weights(W.cuda())
    assert B.validate_packed(packed, N, K) == 0
    L = B.load_library()
    bad = torch.zeros(1, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    assert L.bitlinear_validate_packed(packed.data_ptr(), N, K, bad.data_ptr(), stream) == B.OK
    broken = packed.clone()
    broken[1000] = 0xFF   # four fields with code 3
    broken[17] = 0x03 | (int(broken[17].item()) & 0xFC)   # one more (field 0 of another byte)
    assert L.bitlinear_validate_packed(broken.data_ptr(), N, K, bad.data_ptr(), stream) == B.ERR_BADCODE
    assert bad.item() == 5 and B.validate_packed(broken, N, K) == 5
