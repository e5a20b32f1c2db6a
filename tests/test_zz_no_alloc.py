"""The GEMM entry point that allocates nothing, against the oracle's matmul and against the
context-based entry point (same kernel, scratch from the context's workspace).  Named so that it is
collected after every other test file: it must pass on a GPU that earlier tests have already used,
and on its own."""
import numpy as np
import pytest

from oracle import sdv_oracle as O
from sdv_inputs import bf16_bits_to_f32, f32_to_bf16_bits, get_config
import paper_2510_15312_b200 as pkg
from paper_2510_15312_b200.binding import Sdv, config_from

pytestmark = pytest.mark.gpu


def _case(seed, M, N, K):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((M, K)).astype(np.float32)
    wb = f32_to_bf16_bits(rng.standard_normal((N, K)).astype(np.float32))
    return x, wb


def test_noalloc_gemm_matches_context_gemm_twice_in_a_row():
    import torch
    ctx = Sdv(config_from(get_config("tiny"), k_max=16, max_seq=4096))
    try:
        # two calls back to back with different shapes and data: the second one finds the scratch
        # array as the first left it, so it also checks that stale contents are cleared
        for seed, (M, N, K) in enumerate([(17, 1024, 256), (9, 768, 1024), (32, 1024, 1024)]):  # the last one fills the scratch
            x, wb = _case(100 + seed, M, N, K)
            ref, _ = ctx.debug_gemm(x, wb)
            dx = torch.from_numpy(x).cuda()
            dw = torch.from_numpy(wb.view(np.int16)).cuda()
            dy = torch.full((M, N), float("nan"), device="cuda")
            if seed == 0:
                assert pkg.gemm_noalloc(dx, dw, dy) == pkg.OK   # first call: module load and the symbol look-up
            torch.cuda.synchronize()
            before, free_before = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
            rc = pkg.gemm_noalloc(dx, dw, dy)
            assert rc == pkg.OK
            # neither torch's allocator nor the driver handed out memory during the call
            assert torch.cuda.memory_allocated() == before
            assert torch.cuda.mem_get_info()[0] == free_before
            y = dy.cpu().numpy()
            # the oracle's product of the same operands: x is rounded to bf16 on the way in (the weights are
            # bf16 already), accumulation is fp32 on both sides
            xr = bf16_bits_to_f32(f32_to_bf16_bits(x))
            np.testing.assert_allclose(y, O.matmul(xr, wb), rtol=0, atol=2e-5 * np.sqrt(K))
            # same kernel, same partition: only the order of the fp32 atomic adds may differ
            np.testing.assert_allclose(y, ref, rtol=0, atol=2e-5 * np.sqrt(K))
        # one more call that repeats the first case must give the first case's answer again
        x, wb = _case(100, 17, 1024, 256)
        ref, _ = ctx.debug_gemm(x, wb)
        dy = torch.zeros((17, 1024), device="cuda")
        assert pkg.gemm_noalloc(torch.from_numpy(x).cuda(), torch.from_numpy(wb.view(np.int16)).cuda(), dy) == pkg.OK
        np.testing.assert_allclose(dy.cpu().numpy(), ref, rtol=0, atol=2e-5 * np.sqrt(256))
    finally:
        ctx.close()


def test_noalloc_gemm_rejects_sizes_beyond_its_scratch():
    import torch
    L = pkg.lib()
    buf = torch.zeros(1024, device="cuda")
    p = buf.data_ptr()
    # shape checks come before any access, so small dummy buffers are enough
    assert L.sdv_gemm_noalloc(p, p, p, 33, 64, 64, None) == pkg.ETOOBIG       # too many rows
    assert L.sdv_gemm_noalloc(p, p, p, 4, 4096 + 16, 64, None) == pkg.ETOOBIG  # too many outputs
    assert L.sdv_gemm_noalloc(p, p, p, 4, 64, 4096 + 64, None) == pkg.ETOOBIG  # too long a contraction
    assert L.sdv_gemm_noalloc(p, p, p, 4, 2048, 1024, None) == pkg.ETOOBIG     # weights above 2 MiB
    assert L.sdv_gemm_noalloc(p, p, p, 4, 24, 64, None) == pkg.EINVAL          # N not a multiple of 16
    assert L.sdv_gemm_noalloc(p, p, p, 4, 64, 96, None) == pkg.EINVAL          # K not a multiple of 64
    assert L.sdv_gemm_noalloc(None, p, p, 4, 64, 64, None) == pkg.EINVAL
    # x and w are read 16 bytes at a time: a view that starts 4 bytes into a tensor is refused, not faulted on
    assert L.sdv_gemm_noalloc(p + 4, p, p, 4, 64, 64, None) == pkg.EINVAL
    assert L.sdv_gemm_noalloc(p, p + 2, p, 4, 64, 64, None) == pkg.EINVAL
    assert L.sdv_gemm_noalloc(p, p, p + 2, 4, 64, 64, None) == pkg.EINVAL
    odd = torch.zeros((5, 65), device="cuda")[1:, :64].contiguous()[0:4]      # contiguous again: aligned
    assert odd.data_ptr() % 16 == 0
    view = torch.zeros(4 * 64 + 1, device="cuda")[1:].view(4, 64)            # starts at element 1: 4-byte aligned only
    dw = torch.zeros((64, 64), dtype=torch.int16, device="cuda")
    dy = torch.zeros((4, 64), device="cuda")
    assert pkg.gemm_noalloc(view, dw, dy) == pkg.EINVAL
    # host memory is refused as well
    host = np.zeros(64 * 64, dtype=np.float32)
    assert L.sdv_gemm_noalloc(host.ctypes.data - host.ctypes.data % 16 + 16, p, p, 4, 64, 64, None) == pkg.EINVAL
    assert len(L.sdv_strerror(pkg.ETOOBIG)) > 0
