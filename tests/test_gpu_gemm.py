"""The three contractions of a layer in isolation (through lp_gemm_bf16) against their
definition, C = A.B in float64 on the same bf16 operands.  Sizes span several 128-wide
tiles with ragged tails, single-tile cases, and the degenerate small extents of the
workloads (N = 10, K = 784, M = 32)."""
import numpy as np
import pytest

from gpu_common import rel_l2

pytestmark = pytest.mark.gpu

SHAPES = [(128, 128, 64), (256, 384, 512), (32, 10, 784), (300, 200, 520), (1, 8, 8), (129, 65, 72),
          (512, 1000, 256), (64, 2056, 136)]


def _operands(which, M, N, K, seed):
    import torch
    g = torch.Generator(device="cpu").manual_seed(seed)
    pad8 = lambda v: (v + 7) // 8 * 8
    if which == 0:
        A = torch.randn(M, pad8(K), generator=g)
        B = torch.randn(N, pad8(K), generator=g)
    elif which == 1:
        A = torch.randn(M, pad8(K), generator=g)
        B = torch.randn(K, pad8(N), generator=g)
    else:
        A = torch.randn(K, pad8(M), generator=g)
        B = torch.randn(K, pad8(N), generator=g)
    return A.bfloat16(), B.bfloat16()


def _reference(which, M, N, K, A, B):
    a = A.double().numpy()
    b = B.double().numpy()
    if which == 0:
        return a[:, :K] @ b[:, :K].T
    if which == 1:
        return a[:, :K] @ b[:K, :N]
    return a[:K, :M].T @ b[:K, :N]


@pytest.mark.parametrize("tile_n", [0, 64, 256, 512, 448])      # 512 / 448 = 256 x 256 / 256 x 224 tile on an SM pair (cta_group::2)
@pytest.mark.parametrize("which", [0, 1, 2])
def test_contraction_matches_definition(which, tile_n):
    import torch
    from paper_2108_06629_b200 import binding as lpb
    lpb.lp_set_tuning(tile_n, 0)
    try:
        for i, (M, N, K) in enumerate(SHAPES):
            A, B = _operands(which, M, N, K, 100 * which + i)
            ref = _reference(which, M, N, K, A, B)
            ldc = (N + 3) // 4 * 4
            Cd = torch.full((M, ldc), 7.0, device="cuda")
            lpb.lp_gemm_bf16(which, M, N, K, A.cuda(), A.shape[1], B.cuda(), B.shape[1], Cd, ldc)
            torch.cuda.synchronize()
            got = Cd.cpu().numpy()
            assert rel_l2(got[:, :N], ref) < 1e-6 + 2e-7 * np.sqrt(K), (which, M, N, K)   # fp32 accumulation over K terms
            assert np.all(got[:, N:] == 0.0)          # pad lanes of the last 16-byte group are zeroed
    finally:
        lpb.lp_set_tuning(0, 0)


def test_deep_pipeline_and_two_stage_pipeline_agree():
    import torch
    from paper_2108_06629_b200 import binding as lpb
    M, N, K = 256, 256, 4096
    A, B = _operands(0, M, N, K, 7)
    outs = []
    for stages in (2, 6):
        lpb.lp_set_tuning(128, stages)
        Cd = torch.empty((M, N), device="cuda")
        lpb.lp_gemm_bf16(0, M, N, K, A.cuda(), K, B.cuda(), K, Cd, N)
        torch.cuda.synchronize()
        outs.append(Cd.cpu().numpy())
    lpb.lp_set_tuning(0, 0)
    assert np.array_equal(outs[0], outs[1])
    assert rel_l2(outs[0], _reference(0, M, N, K, A, B)) < 1e-6 + 2e-7 * np.sqrt(K)


def test_status_word_is_clear_after_ordinary_launches():
    import torch
    from paper_2108_06629_b200 import binding as lpb
    A, B = _operands(0, 256, 384, 512, 3)
    Cd = torch.empty((256, 384), device="cuda")
    lpb.lp_gemm_bf16(0, 256, 384, 512, A.cuda(), 512, B.cuda(), 512, Cd, 384)
    rc, word = lpb.lp_gemm_status()
    assert (rc, word) == (lpb.LP_OK, 0)


def test_bounded_wait_runs_out_reports_and_leaves_the_device_usable():
    """Every barrier wait in the kernels is bounded.  Here one is made to run out in the harmless
    way the library offers for it: the producer skips the last k-block, the MMA issuer waits for it
    for 2e6 cycles (about a millisecond) and gives up.  The kernel must return by itself, the
    status word must say so, and the next ordinary launch must be exact and leave the word clear."""
    import torch
    from paper_2108_06629_b200 import binding as lpb
    M, N, K = 256, 384, 512
    A, B = _operands(0, M, N, K, 11)
    Ad, Bd = A.cuda(), B.cuda()
    Cd = torch.zeros((M, N), device="cuda")
    assert lpb.lp_gemm_status() == (lpb.LP_OK, 0)
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    lpb.lp_debug_gemm_starved(M, N, K, Ad, K, Bd, K, Cd, N, 2_000_000)
    t1.record()
    rc, word = lpb.lp_gemm_status()            # waits for the device
    assert rc == lpb.LP_ERR_TIMEOUT and word in (2, 3), (rc, word)
    assert b"bounded" in lpb.lib().lp_last_error(None)
    assert t0.elapsed_time(t1) < 500.0         # gave up after the short limit, not after seconds
    # what did arrive was contracted: the result is the product over the first K - 64 columns (if the
    # epilogue's own wait had not run out first, in which case C was left alone)
    if word == 2:
        ref = A.double().numpy()[:, :K - 64] @ B.double().numpy()[:, :K - 64].T
        assert rel_l2(Cd.cpu().numpy(), ref) < 1e-5
    assert lpb.lp_gemm_status() == (lpb.LP_OK, 0)          # reading the word cleared it
    lpb.lp_gemm_bf16(0, M, N, K, Ad, K, Bd, K, Cd, N)
    assert lpb.lp_gemm_status() == (lpb.LP_OK, 0)
    assert rel_l2(Cd.cpu().numpy(), _reference(0, M, N, K, A, B)) < 1e-6 + 2e-7 * np.sqrt(K)
    # argument checks of the verification call
    lib = lpb.lib()
    assert lib.lp_debug_gemm_starved(M, N, 64, None, K, None, K, None, N, 2_000_000, None) == lpb.LP_ERR_INVALID_ARG
    assert lib.lp_debug_gemm_starved(M, N, K, Ad.data_ptr(), K, Bd.data_ptr(), K, Cd.data_ptr(), N, 5, None) == lpb.LP_ERR_INVALID_ARG
