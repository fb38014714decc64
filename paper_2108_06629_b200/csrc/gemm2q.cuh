// Persistent SM-pair kernel for the forward (Eqs. 1-2) and delta (Eqs. 3-4) contractions: the form the
// pair kernel takes when a pair CTA has its SM to itself (TMEM_PAIR_ALONE, networks that mix pair and
// single-CTA kernels).  Alone on the SM, a one-tile CTA has nothing that hides its epilogue; here one
// CTA pair per SM pair walks the 256 x 256 tiles pair_id, pair_id + pairs, ... with the accumulator
// double-buffered in tensor memory (2 x 256 columns = all 512, which is why it must be alone), so the
// epilogue of tile i (activation / f' multiply / un-pooling, bf16 stores) runs under the main loop
// of tile i + 1:
//   warp 0     operand producer (TMA, ring of S stages of 32 KiB, runs on across tile boundaries)
//   warp 1     MMA issuer (leader CTA)
//   warps 2-5  epilogue of both CTAs, each on its own 128 rows
// Tiles are numbered rows first, so the pairs that run at the same time read the same columns of the
// weights and different rows of the activations.
// Barriers: full[s] (leader; both CTAs' loads complete on it), empty[s] (each CTA; tcgen05.commit
// multicast), accf[b] (each CTA; accumulator b complete), acce[b] (leader; eight arrivals: the four
// epilogue warps of each CTA have read accumulator b out).  Every wait is bounded.
#pragma once
#include "gemm2p.cuh"

namespace lp {

constexpr int GEMM2Q_THREADS = 192;
constexpr int GEMM2Q_STAGES = 5;
constexpr int GEMM2Q_STAGE = 32 * 1024;
constexpr int GEMM2Q_SMEM_BYTES = GEMM2Q_STAGES * GEMM2Q_STAGE + EPI_TILE_BYTES + 1024 + 1024;   // 181 KiB: no other allocating kernel fits beside it

template <bool B_MN, int MODE, int BN2 = GEMM2_BN>
__global__ void __launch_bounds__(GEMM2Q_THREADS, 1)
gemm2q_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const GemmArgs p,
              const int tiles_m, const int tiles_n) {
  constexpr int STAGE = GEMM2Q_STAGE, S = GEMM2Q_STAGES;
  static_assert(BN2 % 32 == 0 && BN2 >= 64 && BN2 <= 256, "pair tile width");
  constexpr uint32_t kLoadBytes = GEMM_A_BYTES + (B_MN ? 2 * 8192 : (BN2 / 2) * GEMM_BK * 2);
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  float* epi_tile = reinterpret_cast<float*>(smem + S * STAGE);
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + S * STAGE + EPI_TILE_BYTES);
  uint64_t* empty_bar = full_bar + S;
  uint64_t* accf_bar = empty_bar + S;     // [2]
  uint64_t* acce_bar = accf_bar + 2;      // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acce_bar + 2);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int num_kb = (p.K + GEMM_BK - 1) / GEMM_BK;
  const int total = tiles_m * tiles_n;
  const int pair_id = int(blockIdx.x >> 1), pairs = int(gridDim.x >> 1);
  const bool pix = (p.g.kind == GEOM_PIX_M);

  // this CTA's part of tile t
  auto tile_map = [&](int t) {
    TileMap tm;
    const int tmi = t % tiles_m, tni = t / tiles_m;
    tm.m0 = tmi * 256 + int(rank) * 128;
    tm.n0 = p.n_begin + tni * BN2;
    tm.nlim = p.N;
    tm.pn0 = tm.ph0 = tm.pw0 = 0;
    if (pix) {
      const int bx = tmi * 2 + int(rank);
      const int tw = bx % p.g.tiles_w, th = (bx / p.g.tiles_w) % p.g.tiles_h, tn = bx / (p.g.tiles_w * p.g.tiles_h);
      tm.pw0 = tw << p.g.lw;
      tm.ph0 = th << p.g.lh;
      tm.pn0 = tn * (GEMM_BM >> (p.g.lw + p.g.lh));
    }
    return tm;
  };

  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
    for (int s = 0; s < S; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&accf_bar[b], 1);
      mbar_init(&acce_bar[b], 8);
    }
    fence_barrier_init();
  }
  if (warp == 1) {
    if (lane == 0) tmem_note_enter(TK_PAIR_FD);
    tmem_alloc2(tmem_slot, 512);
    if (lane == 0) tmem_note_got(TK_PAIR_FD, 512);
    tmem_relinquish2();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ operand producer (both CTAs)
    if (lane == 0) {
      bool ok = true;
      long long issued = 0;
      const uint32_t smem0 = smem_u32(smem);
      const uint32_t full0 = smem_u32(full_bar), empty0 = smem_u32(empty_bar);
      uint32_t s = 0, ph = 0;
      for (int t = pair_id; t < total && ok; t += pairs) {
        const TileMap tm = tile_map(t);
        const int nb0 = tm.n0 + int(rank) * (BN2 / 2);        // the half of B this CTA stages
        int k0 = 0, c_tap = 0, c_chunk = 0;
        for (int kb = 0; kb < num_kb; ++kb, k0 += GEMM_BK) {
          ok = mbar_wait_addr(empty0 + 8u * s, ph ^ 1u, p.wait_limit);
          if (!ok) break;
          const uint32_t sa = smem0 + s * uint32_t(STAGE);
          const uint32_t sb = sa + GEMM_A_BYTES;
          const uint32_t fb = map_to_cta(full0 + 8u * s, 0);          // the leader's barrier
          if (rank == 0) mbar_arrive_expect_tx_addr(full0 + 8u * s, 2u * kLoadBytes);
          if (pix) {
            // (stride-1 layers: the tap's shift is the whole coordinate arithmetic)
            const int r = c_tap / p.g.S, sft = c_tap % p.g.S;
            const int sh = p.g.flip ? p.g.pad - r : r - p.g.pad;
            const int sw = p.g.flip ? p.g.pad - sft : sft - p.g.pad;
            tma2_load_4d_addr(sa, &tmA, fb, c_chunk * 64, tm.pw0 + sw, tm.ph0 + sh, tm.pn0);
            if (B_MN) {   // delta: B[k = (tap, co)][n = ci]
#pragma unroll
              for (int c = 0; c < 2; ++c) tma2_load_2d_addr(sb + c * 8192, &tmB, fb, c_tap * p.g.tap_pitch + nb0 + c * 64, c_chunk * 64);
            } else {      // forward: B[n = co][k = (tap, ci)]
              tma2_load_2d_addr(sb, &tmB, fb, c_tap * p.g.tap_pitch + c_chunk * 64, nb0);
            }
            if (++c_chunk == p.g.chunks_per_tap) { c_chunk = 0; ++c_tap; }
          } else {
            tma2_load_2d_addr(sa, &tmA, fb, k0, tm.m0);
            if (B_MN) {
#pragma unroll
              for (int c = 0; c < 2; ++c) tma2_load_2d_addr(sb + c * 8192, &tmB, fb, nb0 + c * 64, k0);
            } else {
              tma2_load_2d_addr(sb, &tmB, fb, k0, nb0);
            }
          }
          ++issued;
          if (++s == uint32_t(S)) { s = 0; ph ^= 1u; }
        }
      }
      if (!ok) {
        atomicExch(p.status, 24);
        // let copies already in flight land before the CTA's shared memory is released
        if (rank == 0)
          for (long long i = (issued > S ? issued - S : 0); i < issued; ++i) mbar_wait(&full_bar[i % S], uint32_t(i / S) & 1u, p.wait_limit);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (leader only)
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(256, BN2, false, B_MN);
      const uint64_t dA = make_smem_desc(smem_u32(smem), 16, 1024);
      const uint64_t dB = B_MN ? make_smem_desc(smem_u32(smem) + GEMM_A_BYTES, 8192, 1024)
                               : make_smem_desc(smem_u32(smem) + GEMM_A_BYTES, 16, 1024);
      const uint32_t dA_hi = uint32_t(dA >> 32), dB_hi = uint32_t(dB >> 32);
      constexpr uint32_t stepA = 32 >> 4, stepB = (B_MN ? 2048 : 32) >> 4;
      const uint32_t full0 = smem_u32(full_bar), empty0 = smem_u32(empty_bar);
      const uint32_t accf0 = smem_u32(accf_bar), acce0 = smem_u32(acce_bar);
      uint32_t s = 0, ph = 0, it = 0;
      uint32_t dA_lo = uint32_t(dA), dB_lo = uint32_t(dB);
      bool ok = true;
      for (int t = pair_id; t < total && ok; t += pairs, ++it) {
        const uint32_t buf = it & 1u;
        // both CTAs' epilogues must have read this accumulator out (tile it - 2)
        ok = mbar_wait_addr(acce0 + 8u * buf, ((it >> 1) & 1u) ^ 1u, p.wait_limit);
        if (!ok) break;
        tc_fence_after();
        const uint32_t tacc = tmem_base + buf * 256u;
        uint32_t acc = 0;
        for (int kb = 0; kb < num_kb; ++kb) {
          ok = mbar_wait_addr(full0 + 8u * s, ph, p.wait_limit);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int j = 0; j < GEMM_BK / 16; ++j) {
            umma2_f16_lohi(tacc, dA_lo + j * stepA, dA_hi, dB_lo + j * stepB, dB_hi, idesc, acc);
            acc = 1;
          }
          umma2_commit_both(empty0 + 8u * s);
          dA_lo += uint32_t(STAGE >> 4);
          dB_lo += uint32_t(STAGE >> 4);
          if (++s == uint32_t(S)) {
            s = 0;
            ph ^= 1u;
            dA_lo = uint32_t(dA);
            dB_lo = uint32_t(dB);
          }
        }
        umma2_commit_both(accf0 + 8u * buf);      // accumulator complete in both CTAs (also releases the epilogues on error)
      }
      if (!ok) atomicExch(p.status, 25);
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2-5 of both CTAs, own 128 rows)
    const int q = warp & 3;                                     // tensor-memory lane quarter this warp may read
    float* tile = epi_tile + q * (32 * EPI_PITCH);
    const int sub_row = lane >> 3;
    const int sub_col = (lane & 7) * 4;
    const uint32_t accf0 = smem_u32(accf_bar);
    const uint32_t acce_leader = map_to_cta(smem_u32(acce_bar), 0);
    bool good = true;
    uint32_t it = 0;
    for (int t = pair_id; t < total && good; t += pairs, ++it) {
      const TileMap tm = tile_map(t);
      const uint32_t buf = it & 1u;
      const uint32_t tacc = tmem_base + buf * 256u;
      good = mbar_wait_addr(accf0 + 8u * buf, (it >> 1) & 1u, p.wait_limit);
      good = __all_sync(0xffffffffu, good);
      if (!good) {
        if (lane == 0) atomicExch(p.status, 26);
        break;
      }
      tc_fence_after();
#pragma unroll 1
      for (int c = 0; c < BN2 / 32; ++c) {
        uint32_t r[32];
        __syncwarp();
        tmem_ld_32x32(tacc + (uint32_t(q * 32) << 16) + uint32_t(c * 32), r);
        tmem_ld_wait();
        if (c == BN2 / 32 - 1) {
          // last read of this accumulator: hand it back to the MMA issuer (in the leader CTA)
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(acce_leader + 8u * buf);
        }
#pragma unroll
        for (int g = 0; g < 8; ++g)
          *reinterpret_cast<uint4*>(tile + lane * EPI_PITCH + g * 4) = make_uint4(r[4 * g], r[4 * g + 1], r[4 * g + 2], r[4 * g + 3]);
        __syncwarp();
        epilogue_rows8<MODE>(p, tm, tile, q, sub_row, sub_col, tm.n0 + c * 32 + sub_col);
      }
    }
  }
  // neither CTA may release shared or tensor memory while its partner can still touch it
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc2(tmem_base, 512);
    if (lane == 0) tmem_note_freed(TK_PAIR_FD, 512);
  }
}

}  // namespace lp
