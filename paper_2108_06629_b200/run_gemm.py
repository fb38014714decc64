"""Run one of the three contractions of a layer on random operands a few times.

    python -m paper_2108_06629_b200.run_gemm WHICH M N K REPS [TILE_N [STAGES]]

WHICH = 0 forward (A[M][K] . B[N][K]^T), 1 delta (A[M][K] . B[K][N]), 2 G (A[K][M]^T . B[K][N]);
bf16 operands, fp32 result, through lp_gemm_bf16.  Prints the event-timed duration and
TFLOP/s; meant to be wrapped by a profiler as well.
"""
import sys


def main(argv):
    import torch
    from . import binding as lpb
    which, M, N, K, reps = (int(v) for v in argv[:5])
    lpb.lp_set_tuning(int(argv[5]) if len(argv) > 5 else 0, int(argv[6]) if len(argv) > 6 else 0, 1)
    g = torch.Generator(device="cuda").manual_seed(0)
    shapes = {0: ((M, K), (N, K)), 1: ((M, K), (K, N)), 2: ((K, M), (K, N))}[which]
    A = torch.randn(shapes[0], device="cuda", generator=g).bfloat16()
    B = torch.randn(shapes[1], device="cuda", generator=g).bfloat16()
    C = torch.empty((M, N), device="cuda")
    lpb.lp_gemm_bf16(which, M, N, K, A, A.shape[1], B, B.shape[1], C, N)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        lpb.lp_gemm_bf16(which, M, N, K, A, A.shape[1], B, B.shape[1], C, N)
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / reps
    print("which=%d M=%d N=%d K=%d: %.1f us per launch, %.1f TFLOP/s" % (which, M, N, K, us, 2.0 * M * N * K / us / 1e6))


if __name__ == "__main__":
    main(sys.argv[1:])
