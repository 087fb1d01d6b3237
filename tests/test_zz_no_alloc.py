"""codenet_matvec_noalloc, the entry point for callers that cannot allocate device memory at the
time of the call (a latency-critical loop that cannot take cudaMalloc's synchronisation, a process
whose memory pool already owns the whole device, a no-allocation-after-start-up policy).  It must give what the allocating path gives, call after call, although all calls
share one fixed scratch array that keeps its previous contents.

Collected last on purpose: a run that stops at the first failure has then run every other test."""
import numpy as np
import pytest
import torch

from paper_1903_01042_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def cn():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device (there is no CPU path)")
    from paper_1903_01042_b200 import codenet
    codenet.lib()
    return codenet


def test_matches_the_allocating_forward_on_two_calls_in_a_row(cn):
    rows, cols, n_blocks = 1536, 2048, 8             # 8 block-columns of 256; several CTAs and a ragged last one
    W = torch.tensor(wl.weights(rows, cols, seed=21), device="cuda")
    # the existing entry point: an uncoded 1 x 8 grid, no check
    layer = cn.encode_layer(W, 1, n_blocks, 0, 0, batch_max=1, locate_mode=cn.LOCATE_OFF)
    s_static = torch.full((rows,), float("nan"), device="cuda")
    for call in range(2):
        x = torch.tensor(wl.gaussian_inputs(1, cols, seed=22, iteration=call), device="cuda")
        want = cn.forward(layer, x)
        got = cn.matvec_noalloc(W, n_blocks, x, s_static)
        torch.cuda.synchronize()
        a, b = got.cpu().numpy().ravel(), want.cpu().numpy().ravel()
        err = np.max(np.abs(a - b)) / np.max(np.abs(b))
        assert err <= 1e-5, (call, err)               # the tolerance of the fp32 parity tests
        assert np.array_equal(a, b), call             # same kernels, same order: in fact identical
        ref = W.double().cpu().numpy() @ x.double().cpu().numpy().ravel()
        assert np.max(np.abs(a - ref)) / np.max(np.abs(ref)) <= 1e-5


def test_a_smaller_problem_after_a_larger_one_ignores_stale_scratch(cn):
    big = torch.tensor(wl.weights(4096, 1024, seed=23), device="cuda")
    small = torch.tensor(wl.weights(40, 64, seed=24), device="cuda")
    xb = torch.tensor(wl.gaussian_inputs(1, 1024, seed=25), device="cuda")
    xs = torch.tensor(wl.gaussian_inputs(1, 64, seed=26), device="cuda")
    cn.matvec_noalloc(big, 4, xb, torch.empty(4096, device="cuda"))
    got = cn.matvec_noalloc(small, 2, xs, torch.empty(40, device="cuda")).cpu().numpy()
    ref = small.double().cpu().numpy() @ xs.double().cpu().numpy().ravel()
    assert np.max(np.abs(got - ref)) / np.max(np.abs(ref)) <= 1e-5


def test_rejects_what_does_not_fit_the_fixed_scratch(cn):
    rows, n_blocks = (1 << 20) // 8 + 1, 8           # rows * n_blocks just above 2^20 floats
    W = torch.zeros((rows, 32), device="cuda")
    x = torch.zeros(32, device="cuda")
    s = torch.zeros(rows, device="cuda")
    with pytest.raises(cn.CodenetError, match="scratch"):
        cn.matvec_noalloc(W, n_blocks, x, s)
    with pytest.raises(cn.CodenetError):
        cn.matvec_noalloc(torch.zeros((8, 30), device="cuda"), 3, torch.zeros(30, device="cuda"),
                          torch.zeros(8, device="cuda"))   # block width not a multiple of 4


def test_a_warmed_up_call_allocates_nothing_even_while_kernels_are_being_timed(cn):
    """Free device memory and torch's own allocator count stay where they were across calls, also with the
    library's per-kernel timing switched on (its event brackets are the one thing in the forward launch that
    would allocate)."""
    rows, cols, n_blocks = 512, 1024, 4
    W = torch.tensor(wl.weights(rows, cols, seed=27), device="cuda")
    x = torch.tensor(wl.gaussian_inputs(1, cols, seed=28), device="cuda")
    s = torch.empty(rows, device="cuda")
    cn.matvec_noalloc(W, n_blocks, x, s)                # first call on the device: looks up the scratch address
    torch.cuda.synchronize()
    for timed in (False, True):
        cn.profile_enable(timed)
        try:
            free0, _ = torch.cuda.mem_get_info()
            held0 = torch.cuda.memory_allocated()
            before = cn.profile_read(cn.KERNEL_FORWARD)[1] if timed else 0
            for _ in range(3):
                cn.matvec_noalloc(W, n_blocks, x, s)
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info()[0] == free0
            assert torch.cuda.memory_allocated() == held0
            if timed:                                    # and its launches are not booked on the forward kernel's account
                assert cn.profile_read(cn.KERNEL_FORWARD)[1] == before
        finally:
            cn.profile_enable(False)
    ref = W.double().cpu().numpy() @ x.double().cpu().numpy().ravel()
    assert np.max(np.abs(s.cpu().numpy() - ref)) / np.max(np.abs(ref)) <= 1e-5
