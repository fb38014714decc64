// Warp-specialised tcgen05 GEMM for sm_100a: D[M][N] = A . B with bf16 operands staged
// in shared memory by TMA (128-byte swizzle), fp32 accumulators in tensor memory, and a
// fused epilogue.  One 128 x BN output tile per CTA.
//
//   warp 0      TMA producer (one elected lane)
//   warp 1      tensor-memory allocation + MMA issue (one elected lane)
//   warps 2-5   epilogue: tcgen05.ld -> registers -> bias / activation / f' -> global
//
// Operand "major" follows the tensor-core convention: K-major = the contraction index is
// contiguous in memory, MN-major = the M (or N) index is contiguous.  With W stored
// [out][in] and activations [batch][features] the three contractions of a layer are
//   forward (Eq. 1)  A = a      K-major,  B = W      K-major
//   delta   (Eq. 4)  A = delta  K-major,  B = W      MN-major
//   G       (Eq. 5)  A = delta  MN-major, B = a      MN-major
// so one copy of each tensor serves all three.
#pragma once
#include <cuda_bf16.h>

#include "ptx.cuh"

namespace lp {

constexpr int GEMM_BM = 128;
constexpr int GEMM_BK = 64;          // 64 bf16 = one 128-byte swizzle row
constexpr int GEMM_THREADS = 192;
constexpr int GEMM_A_BYTES = GEMM_BM * GEMM_BK * 2;   // 16 KiB
constexpr int GEMM_MAX_STAGES = 8;

enum { EPI_STORE_F32 = 0, EPI_FPROP = 1, EPI_DGRAD = 2 };
enum { ACT_NONE = 0, ACT_RELU = 1, ACT_GELU = 2 };

struct GemmArgs {
  int M, N, K;
  int num_stages;
  int mode;                 // EPI_*
  int act;                  // ACT_*  (FPROP: f of this layer; DGRAD: f' of the previous layer)
  void* out;                // STORE_F32: float [M][ld_out]; FPROP: bf16 a^l (may be null); DGRAD: bf16 delta^{l-1}
  int ld_out;
  void* out2;               // FPROP: bf16 stored z^l (GELU) or fp32 z^L (last layer); else null
  int ld_out2;
  int out2_is_f32;
  const float* bias;        // FPROP: fp32 [N] or null
  const __nv_bfloat16* aux; // DGRAD: what f' is evaluated on (stored z for GELU, a for ReLU)
  int ld_aux;
  int* status;              // device status word: set non-zero if a bounded wait expires
};

__device__ __forceinline__ float gelu_fwd(float z) {
  return 0.5f * z * (1.0f + erff(z * 0.70710678118654752f));
}
__device__ __forceinline__ float gelu_grad(float z) {
  const float Phi = 0.5f * (1.0f + erff(z * 0.70710678118654752f));
  const float phi = __expf(-0.5f * z * z) * 0.39894228040143268f;
  return Phi + z * phi;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }

template <int BN>
struct GemmSmem {
  static constexpr int B_BYTES = BN * GEMM_BK * 2;
  static constexpr int STAGE_BYTES = GEMM_A_BYTES + B_BYTES;
  static constexpr size_t bytes(int stages) { return size_t(stages) * STAGE_BYTES + 1024 /*align slack*/ + 256; }
};

template <int BN, bool A_MN, bool B_MN>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const GemmArgs p) {
  using SM = GemmSmem<BN>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int S = p.num_stages;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + size_t(S) * SM::STAGE_BYTES);
  uint64_t* empty_bar = full_bar + GEMM_MAX_STAGES;
  uint64_t* acc_bar = empty_bar + GEMM_MAX_STAGES;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_bar + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int m0 = blockIdx.x * GEMM_BM;
  const int n0 = blockIdx.y * BN;
  const int num_kb = (p.K + GEMM_BK - 1) / GEMM_BK;

  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
    for (int s = 0; s < S; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    mbar_init(acc_bar, 1);
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, BN);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      bool ok = true;
      int issued = 0;
      for (int kb = 0; kb < num_kb && ok; ++kb) {
        const int s = kb % S;
        const uint32_t ph = (kb / S) & 1;
        ok = mbar_wait(&empty_bar[s], ph ^ 1u);
        if (!ok) break;
        uint8_t* sa = smem + size_t(s) * SM::STAGE_BYTES;
        uint8_t* sb = sa + GEMM_A_BYTES;
        mbar_arrive_expect_tx(&full_bar[s], SM::STAGE_BYTES);
        const int k0 = kb * GEMM_BK;
        if (A_MN) {
#pragma unroll
          for (int c = 0; c < GEMM_BM / 64; ++c) tma_load_2d(sa + c * 8192, &tmA, &full_bar[s], m0 + c * 64, k0);
        } else {
          tma_load_2d(sa, &tmA, &full_bar[s], k0, m0);
        }
        if (B_MN) {
#pragma unroll
          for (int c = 0; c < BN / 64; ++c) tma_load_2d(sb + c * 8192, &tmB, &full_bar[s], n0 + c * 64, k0);
        } else {
          tma_load_2d(sb, &tmB, &full_bar[s], k0, n0);
        }
        issued = kb + 1;
      }
      if (!ok) {
        atomicExch(p.status, 1);
        // let copies already in flight land before the CTA's shared memory is released
        for (int kb = max(0, issued - S); kb < issued; ++kb) mbar_wait(&full_bar[kb % S], (kb / S) & 1);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(GEMM_BM, BN, A_MN, B_MN);
      bool ok = true;
      for (int kb = 0; kb < num_kb; ++kb) {
        const int s = kb % S;
        const uint32_t ph = (kb / S) & 1;
        ok = mbar_wait(&full_bar[s], ph);
        if (!ok) break;
        tc_fence_after();
        const uint32_t sa = smem_u32(smem + size_t(s) * SM::STAGE_BYTES);
        const uint32_t sb = sa + GEMM_A_BYTES;
#pragma unroll
        for (int j = 0; j < GEMM_BK / 16; ++j) {
          const uint64_t da = A_MN ? make_smem_desc(sa + j * 2048, 8192, 1024) : make_smem_desc(sa + j * 32, 16, 1024);
          const uint64_t db = B_MN ? make_smem_desc(sb + j * 2048, 8192, 1024) : make_smem_desc(sb + j * 32, 16, 1024);
          umma_f16(tmem_base, da, db, idesc, (kb | j) != 0 ? 1u : 0u);
        }
        umma_commit(&empty_bar[s]);   // frees the stage once these MMAs have read it
      }
      if (!ok) atomicExch(p.status, 2);
      umma_commit(acc_bar);           // accumulator complete (also releases the epilogue on error)
    }
  } else {
    // ------------------------------------------------------------ epilogue
    const int q = warp & 3;           // tensor-memory lane quarter this warp may read
    const int row = m0 + q * 32 + lane;
    // stores go out in 16-byte groups; the lanes of the last group past N are written as zeros
    const int n_pad4 = (p.N + 3) & ~3, n_pad8 = (p.N + 7) & ~7;
    bool ok = mbar_wait(acc_bar, 0);
    ok = __all_sync(0xffffffffu, ok);      // warp-uniform: tcgen05.ld below is warp-collective
    if (!ok && lane == 0) atomicExch(p.status, 3);
    tc_fence_after();
    if (ok) {
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t r[32];
        __syncwarp();
        tmem_ld_32x32(tmem_base + (uint32_t(q * 32) << 16) + uint32_t(c * 32), r);
        tmem_ld_wait();
        const int nb = n0 + c * 32;
        if (row >= p.M) {
          // rows past M hold zeros (TMA zero fill); nothing to store
        } else if (p.mode == EPI_STORE_F32) {
          float* o = reinterpret_cast<float*>(p.out) + size_t(row) * p.ld_out;
#pragma unroll
          for (int g = 0; g < 8; ++g) {
            const int n = nb + g * 4;
            if (n >= n_pad4) break;
            float4 v;
            v.x = (n + 0 < p.N) ? __uint_as_float(r[g * 4 + 0]) : 0.f;
            v.y = (n + 1 < p.N) ? __uint_as_float(r[g * 4 + 1]) : 0.f;
            v.z = (n + 2 < p.N) ? __uint_as_float(r[g * 4 + 2]) : 0.f;
            v.w = (n + 3 < p.N) ? __uint_as_float(r[g * 4 + 3]) : 0.f;
            *reinterpret_cast<float4*>(o + n) = v;
          }
        } else if (p.mode == EPI_FPROP) {
          float z[32];
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const int n = nb + j;
            float b = 0.f;
            if (p.bias != nullptr && n < p.N) b = __ldg(p.bias + n);
            z[j] = (n < p.N) ? __uint_as_float(r[j]) + b : 0.f;
          }
          if (p.out2 != nullptr) {
            if (p.out2_is_f32) {
              float* o = reinterpret_cast<float*>(p.out2) + size_t(row) * p.ld_out2;
#pragma unroll
              for (int g = 0; g < 8; ++g) {
                const int n = nb + g * 4;
                if (n >= n_pad4) break;
                *reinterpret_cast<float4*>(o + n) = make_float4(z[g * 4], z[g * 4 + 1], z[g * 4 + 2], z[g * 4 + 3]);
              }
            } else {
              __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(p.out2) + size_t(row) * p.ld_out2;
#pragma unroll
              for (int g = 0; g < 4; ++g) {
                const int n = nb + g * 8;
                if (n >= n_pad8) break;
                uint4 v;
                v.x = pack_bf16x2(z[g * 8 + 0], z[g * 8 + 1]);
                v.y = pack_bf16x2(z[g * 8 + 2], z[g * 8 + 3]);
                v.z = pack_bf16x2(z[g * 8 + 4], z[g * 8 + 5]);
                v.w = pack_bf16x2(z[g * 8 + 6], z[g * 8 + 7]);
                *reinterpret_cast<uint4*>(o + n) = v;
              }
            }
          }
          if (p.out != nullptr) {
            if (p.act == ACT_RELU) {
#pragma unroll
              for (int j = 0; j < 32; ++j) z[j] = fmaxf(z[j], 0.f);
            } else if (p.act == ACT_GELU) {
#pragma unroll
              for (int j = 0; j < 32; ++j) z[j] = gelu_fwd(z[j]);
            }
            __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(p.out) + size_t(row) * p.ld_out;
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              const int n = nb + g * 8;
              if (n >= n_pad8) break;
              uint4 v;
              v.x = pack_bf16x2(z[g * 8 + 0], z[g * 8 + 1]);
              v.y = pack_bf16x2(z[g * 8 + 2], z[g * 8 + 3]);
              v.z = pack_bf16x2(z[g * 8 + 4], z[g * 8 + 5]);
              v.w = pack_bf16x2(z[g * 8 + 6], z[g * 8 + 7]);
              *reinterpret_cast<uint4*>(o + n) = v;
            }
          }
        } else {  // EPI_DGRAD: delta^{l-1} = (delta^l W) (.) f'(z^{l-1}), one rounding
          const __nv_bfloat16* a = p.aux + size_t(row) * p.ld_aux;
          __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(p.out) + size_t(row) * p.ld_out;
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            const int n = nb + g * 8;
            if (n >= n_pad8) break;
            float d[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) d[j] = (n + j < p.N) ? __uint_as_float(r[g * 8 + j]) : 0.f;
            if (p.act != ACT_NONE) {
              const uint4 av = *reinterpret_cast<const uint4*>(a + n);
              const uint32_t aw[4] = {av.x, av.y, av.z, av.w};
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const float z0 = bf16_lo(aw[j]), z1 = bf16_hi(aw[j]);
                if (p.act == ACT_RELU) {
                  d[2 * j] = z0 > 0.f ? d[2 * j] : 0.f;
                  d[2 * j + 1] = z1 > 0.f ? d[2 * j + 1] : 0.f;
                } else {
                  d[2 * j] *= gelu_grad(z0);
                  d[2 * j + 1] *= gelu_grad(z1);
                }
              }
            }
            uint4 v;
            v.x = pack_bf16x2(d[0], d[1]);
            v.y = pack_bf16x2(d[2], d[3]);
            v.z = pack_bf16x2(d[4], d[5]);
            v.w = pack_bf16x2(d[6], d[7]);
            *reinterpret_cast<uint4*>(o + n) = v;
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, BN);
  }
}

}  // namespace lp
