// Two-CTA variant of the tcgen05 GEMM for tensor-bound shapes: a cluster of two CTAs (an SM
// pair) computes one 256 x 256 output tile with tcgen05.mma.cta_group::2.  Each CTA stages its
// own 128 rows of A and only HALF of the B tile (128 of the 256 columns); the tensor cores of
// both SMs read both halves.  Per k-block an SM therefore loads 32 KiB for 128 x 256 x 64 MACs
// (64 B/clk at full tensor rate) instead of the 48 KiB (96 B/clk) a 128 x 256 single-CTA tile
// needs -- the difference between being fed by L2 and starving.
//
//   rank 0 ("leader"): TMA producer, MMA issuer for BOTH CTAs, epilogue of its 128 rows
//   rank 1           : TMA producer (its loads signal the leader's barrier), epilogue of its rows
//
// Hand-offs: TMA loads of both CTAs complete on the leader's "full" barrier (the leader arms it
// with the byte count of both); tcgen05.commit multicasts the "empty" and "accumulator ready"
// arrivals to the same barrier in both CTAs.  Every TMA load has a single destination CTA.
// Plain matrices, and the forward / delta contractions of 3x3 convolutions (GEOM_PIX_M: each
// CTA's 128 rows are a box of 128 pixels fetched through the 4-D NHWC map, shifted by the
// filter tap; one k-block = one tap x 64 channels); no split-K; epilogues as in gemm.cuh.
#pragma once
#include "gemm.cuh"

namespace lp {

constexpr int GEMM2_BN = 256;
// shared::cluster address of the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_alloc2(uint32_t* smem_result, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish2() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc2(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// 2-D tiled load whose completion is counted on the LEADER's barrier
__device__ __forceinline__ void tma2_load_2d_addr(uint32_t smem_dst, const CUtensorMap* m, uint32_t leader_bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, "
      "%4}], [%2];" ::"r"(smem_dst),
      "l"(reinterpret_cast<uint64_t>(m)), "r"(leader_bar), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void tma2_load_4d_addr(uint32_t smem_dst, const CUtensorMap* m, uint32_t leader_bar, int c0, int c1,
                                                  int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, "
      "%4, %5, %6}], [%2];" ::"r"(smem_dst),
      "l"(reinterpret_cast<uint64_t>(m)), "r"(leader_bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ void umma2_f16_lohi(uint32_t tmem_d, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                               uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "mov.b64 da, {%1, %2};\n\t"
      "mov.b64 db, {%3, %4};\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %5, p;\n\t}" ::"r"(tmem_d),
      "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrive on the barrier at this shared-memory offset in BOTH CTAs once all MMAs issued so far are done
__device__ __forceinline__ void umma2_commit_both(uint32_t bar) {
  asm volatile(
      "{\n\t.reg .b16 m;\n\tmov.b16 m, 3;\n\t"
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], m;\n\t}" ::"r"(bar)
      : "memory");
}

__device__ __forceinline__ void phase_mark(const GemmArgs& p, int k) {
  if (p.phase != nullptr) atomicAdd(p.phase + k, 1);
}

// UTMA (EPI_WGRAD_UPDATE only): Eq. 6 on the accumulator tile with the fp32 master / momentum tile
// streamed by TMA through the operand ring once the tile's k-blocks have passed -- each CTA fills
// "chunks" of its own 128 rows x 32 columns (16 KiB + 16 KiB, one stage), its epilogue updates them in
// place in shared memory and TMA stores write master, momentum and the bf16 ring image back.  A
// chunk fill completes on the CTA's own barrier ufull[stage] (the operand fills of both CTAs
// complete on the leader's full[stage]); both kinds of use release the stage through empty[stage],
// so the ring position, and with it the phase of empty[], stays uniform in both CTAs.
// BN2: columns of the pair's tile, 256 or a smaller multiple of 32 (each CTA stages BN2 / 2 of them).
// A narrower tile is chosen where it makes the number of tiles a whole multiple of the SM pairs:
// 2048 x 8192 outputs are 256 tiles of 256 columns -- 3.46 per SM pair, so some pairs run four and
// the tensor pipes of the others idle 13 % of the time -- but 296 = 4 x 74 tiles of 224 columns.
template <bool A_MN, bool B_MN, int MODE, bool UTMA = false, int BN2 = GEMM2_BN>
__global__ void __launch_bounds__(GEMM_THREADS, 2)
gemm2_tcgen05_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                     const __grid_constant__ UpdMaps um, const GemmArgs p) {
  static_assert(!UTMA || MODE == EPI_WGRAD_UPDATE, "the streamed update belongs to the G contraction");
  constexpr int STAGE_BYTES = GEMM_A_BYTES + 128 * GEMM_BK * 2;      // A rows + half of the B tile: 32 KiB
  static_assert(BN2 % 32 == 0 && BN2 >= 64 && BN2 <= 256 && (!UTMA || BN2 == 256), "pair tile width");
  constexpr int kChunks = BN2 / 32;
  // bytes one CTA's loads bring per k-block: its 128 rows of A and its half of the B tile (MN-major B comes in whole
  // 64-column boxes: the second box may reach past the half)
  constexpr uint32_t kLoadBytes = GEMM_A_BYTES + (B_MN ? 2 * 8192 : (BN2 / 2) * GEMM_BK * 2);
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int S = p.num_stages;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + size_t(S) * STAGE_BYTES);
  uint64_t* empty_bar = full_bar + GEMM_MAX_STAGES;
  uint64_t* acc_bar = empty_bar + GEMM_MAX_STAGES;
  uint64_t* ufull_bar = acc_bar + 1;                                   // [GEMM_MAX_STAGES] chunk fills (UTMA)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ufull_bar + GEMM_MAX_STAGES);
  float* epi_tile = reinterpret_cast<float*>(smem);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int num_kb = (p.K + GEMM_BK - 1) / GEMM_BK;
  const bool pix = (p.g.kind == GEOM_PIX_M);

  TileMap tm;
  tm.m0 = (blockIdx.x >> 1) * 256 + int(rank) * 128;    // this CTA's 128 rows
  tm.n0 = p.n_begin + blockIdx.y * BN2;                 // the pair's columns
  tm.nlim = p.N;
  tm.pn0 = tm.ph0 = tm.pw0 = 0;
  if (pix) {                                            // this CTA's box of 128 pixels
    const int bx = (blockIdx.x >> 1) * 2 + int(rank);
    const int tw = bx % p.g.tiles_w, th = (bx / p.g.tiles_w) % p.g.tiles_h, tn = bx / (p.g.tiles_w * p.g.tiles_h);
    tm.pw0 = tw << p.g.lw;
    tm.ph0 = th << p.g.lh;
    tm.pn0 = tn * (GEMM_BM >> (p.g.lw + p.g.lh));
  }
  const int nb0 = tm.n0 + int(rank) * (BN2 / 2);        // the half of B this CTA stages

  if (threadIdx.x == 0) {
    phase_mark(p, 0);
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
    if (UTMA) {
      tma_prefetch_desc(&um.W);
      if (p.mW != nullptr) tma_prefetch_desc(&um.M);
      tma_prefetch_desc(&um.R);
    }
    for (int s = 0; s < S; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
      mbar_init(&ufull_bar[s], 1);
    }
    mbar_init(acc_bar, 1);
    fence_barrier_init();
  }
  if (warp == 1) {
    const long long t_alloc = p.phase != nullptr ? clock64() : 0;
    if (lane == 0) tmem_note_enter(TK_PAIR);
    tmem_alloc2(tmem_slot, GEMM2_BN);
    if (lane == 0) tmem_note_got(TK_PAIR, GEMM2_BN);
    if (lane == 0) phase_mark(p, 1);
    if (p.phase != nullptr && lane == 0 && clock64() - t_alloc > 20000) atomicAdd(p.phase + 10, 1);
    tmem_relinquish2();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();          // the peer's barriers exist before anything arrives on them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  if (threadIdx.x == 0) phase_mark(p, 2);

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      bool ok = true;
      int issued = 0;
      const uint32_t smem0 = smem_u32(smem);
      const uint32_t full0 = smem_u32(full_bar), empty0 = smem_u32(empty_bar);
      uint32_t s = 0, ph = 0;
      int k0 = 0;
      int c_tap = 0, c_chunk = 0;                      // convolution: filter tap and 64-channel chunk of this k-block
      for (int kb = 0; kb < num_kb - p.starve_kb; ++kb, k0 += GEMM_BK) {
        ok = mbar_wait_addr(empty0 + 8u * s, ph ^ 1u, p.wait_limit);
        if (!ok) break;
        const uint32_t sa = smem0 + s * uint32_t(STAGE_BYTES);
        const uint32_t sb = sa + GEMM_A_BYTES;
        const uint32_t fb = map_to_cta(full0 + 8u * s, 0);          // the leader's barrier
        if (rank == 0) mbar_arrive_expect_tx_addr(full0 + 8u * s, 2u * kLoadBytes);
        if (pix) {
          // (this kernel serves stride-1 layers: the tap's shift is the whole coordinate arithmetic)
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
        } else if (A_MN) {
#pragma unroll
          for (int c = 0; c < 2; ++c) tma2_load_2d_addr(sa + c * 8192, &tmA, fb, tm.m0 + c * 64, k0);
        } else {
          tma2_load_2d_addr(sa, &tmA, fb, k0, tm.m0);
        }
        if (pix) {
          // (B was loaded with the tap's coordinates above)
        } else if (B_MN) {
#pragma unroll
          for (int c = 0; c < 2; ++c) tma2_load_2d_addr(sb + c * 8192, &tmB, fb, nb0 + c * 64, k0);
        } else {
          tma2_load_2d_addr(sb, &tmB, fb, k0, nb0);
        }
        issued = kb + 1;
        if (++s == uint32_t(S)) { s = 0; ph ^= 1u; }
      }
      int chunks_issued = 0;
      if constexpr (UTMA) {
        if (ok) {
          // one fill = one stage = 32 KiB: master + momentum of a 32-column chunk, or (no momentum)
          // the master of two neighbouring chunks -- the epilogue is bound by bytes in flight
          const int per = p.mW != nullptr ? 1 : 2;
          const uint32_t ufull0 = smem_u32(ufull_bar);
          for (int f = 0; f < kChunks / per; ++f) {
            ok = mbar_wait_addr(empty0 + 8u * s, ph ^ 1u, p.wait_limit);
            if (!ok) break;
            const uint32_t sa = smem0 + s * uint32_t(STAGE_BYTES);
            const uint32_t ub = ufull0 + 8u * s;
            mbar_arrive_expect_tx_addr(ub, 2u * UPD_CHUNK_BYTES);
            const int n = tm.n0 + f * per * 32;
            tma_load_2d_addr(sa, &um.W, ub, n, tm.m0);
            if (p.mW != nullptr) tma_load_2d_addr(sa + UPD_CHUNK_BYTES, &um.M, ub, n, tm.m0);
            else                 tma_load_2d_addr(sa + UPD_CHUNK_BYTES, &um.W, ub, n + 32, tm.m0);
            chunks_issued = f + 1;
            if (++s == uint32_t(S)) { s = 0; ph ^= 1u; }
          }
        }
      }
      if (!ok) {
        atomicExch(p.status, 11);
        // let copies already in flight land before the CTA's shared memory is released
        if (rank == 0)
          for (int kb = max(0, issued - S); kb < issued; ++kb) mbar_wait(&full_bar[kb % S], (kb / S) & 1, p.wait_limit);
        for (int f = max(0, chunks_issued - S); f < chunks_issued; ++f)
          mbar_wait(&ufull_bar[(num_kb + f) % S], uint32_t(f / S) & 1u, p.wait_limit);
      }
      phase_mark(p, 3);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (leader only)
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(256, BN2, A_MN, B_MN);
      const uint64_t dA = A_MN ? make_smem_desc(smem_u32(smem), 8192, 1024) : make_smem_desc(smem_u32(smem), 16, 1024);
      const uint64_t dB = B_MN ? make_smem_desc(smem_u32(smem) + GEMM_A_BYTES, 8192, 1024)
                               : make_smem_desc(smem_u32(smem) + GEMM_A_BYTES, 16, 1024);
      const uint32_t dA_hi = uint32_t(dA >> 32), dB_hi = uint32_t(dB >> 32);
      constexpr uint32_t stepA = (A_MN ? 2048 : 32) >> 4, stepB = (B_MN ? 2048 : 32) >> 4;
      const uint32_t full0 = smem_u32(full_bar), empty0 = smem_u32(empty_bar);
      uint32_t s = 0, ph = 0, acc = 0;
      uint32_t dA_lo = uint32_t(dA), dB_lo = uint32_t(dB);
      bool ok = true;
      for (int kb = 0; kb < num_kb; ++kb) {
        ok = mbar_wait_addr(full0 + 8u * s, ph, p.wait_limit);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int j = 0; j < GEMM_BK / 16; ++j) {
          umma2_f16_lohi(tmem_base, dA_lo + j * stepA, dA_hi, dB_lo + j * stepB, dB_hi, idesc, acc);
          acc = 1;
        }
        umma2_commit_both(empty0 + 8u * s);
        dA_lo += uint32_t(STAGE_BYTES >> 4);
        dB_lo += uint32_t(STAGE_BYTES >> 4);
        if (++s == uint32_t(S)) {
          s = 0;
          ph ^= 1u;
          dA_lo = uint32_t(dA);
          dB_lo = uint32_t(dB);
        }
      }
      if (!ok) atomicExch(p.status, 12);
      umma2_commit_both(smem_u32(acc_bar));
      phase_mark(p, 4);
    }
  } else {
    // ------------------------------------------------------------ epilogue (both CTAs, own rows)
    const int q = warp & 3;
    float* tile = epi_tile + q * (32 * EPI_PITCH);
    const int sub_row = lane >> 3;
    const int sub_col = (lane & 7) * 4;
    const int row0 = tm.m0 + q * 32;
    constexpr bool upd = (MODE == EPI_WGRAD_UPDATE);
    if constexpr (UTMA) {
      // Every one of the 128 epilogue threads runs the same number of named barriers whatever
      // happens: after a wait that ran out, the remaining chunks only keep the barrier count.
      const uint32_t smem0 = smem_u32(smem), empty0 = smem_u32(empty_bar), ufull0 = smem_u32(ufull_bar);
      const uint32_t ringbuf = smem_u32(full_bar) + 1024u;      // bf16 image of the chunk (8 KiB, 64-byte swizzle)
      const int trow = q * 32 + lane;                           // row of this CTA's half tile = tensor-memory lane
      bool good = mbar_wait(acc_bar, 0, p.wait_limit);
      good = __all_sync(0xffffffffu, good);
      if (!good && lane == 0) atomicExch(p.status, 13);
      tc_fence_after();
      const int per = p.mW != nullptr ? 1 : 2;                  // 32-column chunks per stage fill
      uint32_t us = uint32_t(num_kb % S), pending_stage = 0;
      bool pending = false, pending_release = false;
#pragma unroll 1
      for (int c = 0; c < kChunks; ++c) {
        const int f = c / per, sub = c % per;
        const uint32_t sW = smem0 + us * uint32_t(STAGE_BYTES) + (per == 2 ? uint32_t(sub) * UPD_CHUNK_BYTES : 0u);
        const uint32_t sM = sW + UPD_CHUNK_BYTES;                // (momentum form only)
        if (good && sub == 0) {
          good = mbar_wait_addr(ufull0 + 8u * us, uint32_t(f / S) & 1u, p.wait_limit);
          good = __all_sync(0xffffffffu, good);
          if (!good && lane == 0) atomicExch(p.status, 14);
        }
        uint32_t packed[16];
        if (good) {
          uint32_t r[32];
          tmem_ld_32x32(tmem_base + (uint32_t(q * 32) << 16) + uint32_t(c * 32), r);
          tmem_ld_wait();
          const uint32_t rowoff = uint32_t(trow) * 128u;
          const uint32_t swz = uint32_t(trow & 7);
          const int grow = tm.m0 + trow;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint32_t off = rowoff + ((uint32_t(j) ^ swz) << 4);
            float g[4] = {__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]), __uint_as_float(r[4 * j + 2]),
                          __uint_as_float(r[4 * j + 3])};
            const int n = tm.n0 + c * 32 + 4 * j;
            if (p.out != nullptr && grow < p.M && n < tm.nlim) {
              float* dst = reinterpret_cast<float*>(p.out) + size_t(grow) * p.ld_out + n;
              if (n + 3 < tm.nlim) {
                __stcs(reinterpret_cast<float4*>(dst), make_float4(g[0], g[1], g[2], g[3]));
              } else {
                for (int e = 0; e < 4; ++e) if (n + e < tm.nlim) dst[e] = g[e];
              }
            }
            float m[4] = {g[0], g[1], g[2], g[3]};
            if (p.mW != nullptr) {
              float4 mm;
              asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(mm.x), "=f"(mm.y), "=f"(mm.z), "=f"(mm.w) : "r"(sM + off));
              m[0] = p.mu * mm.x + g[0]; m[1] = p.mu * mm.y + g[1];
              m[2] = p.mu * mm.z + g[2]; m[3] = p.mu * mm.w + g[3];
              asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(sM + off), "f"(m[0]), "f"(m[1]), "f"(m[2]), "f"(m[3]) : "memory");
            }
            float4 w;
            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(w.x), "=f"(w.y), "=f"(w.z), "=f"(w.w) : "r"(sW + off));
            w.x -= p.lr * m[0]; w.y -= p.lr * m[1]; w.z -= p.lr * m[2]; w.w -= p.lr * m[3];
            asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(sW + off), "f"(w.x), "f"(w.y), "f"(w.z), "f"(w.w) : "memory");
            packed[2 * j] = pack_bf16x2(w.x, w.y);
            packed[2 * j + 1] = pack_bf16x2(w.z, w.w);
          }
        }
        // the bf16 staging tile is free once the previous chunk's stores have read it; the same
        // wait releases that chunk's stage to the producer when it was the stage's last chunk
        if (threadIdx.x == 64 && pending) {
          tma_store_wait_read0();
          if (pending_release) mbar_arrive_addr(empty0 + 8u * pending_stage);
          pending = false;
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (good) {
          const uint32_t roff = ringbuf + uint32_t(trow) * 64u;
          const uint32_t rs = uint32_t(trow >> 1) & 3u;
#pragma unroll
          for (int u = 0; u < 4; ++u)
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(roff + ((uint32_t(u) ^ rs) << 4)), "r"(packed[4 * u]),
                         "r"(packed[4 * u + 1]), "r"(packed[4 * u + 2]), "r"(packed[4 * u + 3])
                         : "memory");
        }
        fence_proxy_async_smem();
        asm volatile("bar.sync 1, 128;" ::: "memory");
        const bool last_of_stage = (sub == per - 1);
        if (threadIdx.x == 64) {
          if (good) {
            const int n = tm.n0 + c * 32;
            tma_store_2d_addr(&um.W, sW, n, tm.m0);
            if (p.mW != nullptr) tma_store_2d_addr(&um.M, sM, n, tm.m0);
            tma_store_2d_addr(&um.R, ringbuf, n, tm.m0);
            tma_store_commit();
            pending = true;
            pending_release = last_of_stage;
            pending_stage = us;
          } else if (last_of_stage) {
            mbar_arrive_addr(empty0 + 8u * us);      // keep the producer's bounded waits short
          }
        }
        if (last_of_stage && ++us == uint32_t(S)) us = 0;
      }
      if (pending) tma_store_wait_read0();           // (thread 64 only) shared memory must outlive the last stores' reads
    } else {
    WmRegs cur;
    if constexpr (upd) load_wm(p, row0, tm.n0 + sub_col, tm.nlim, sub_row, cur);
    bool ok = mbar_wait(acc_bar, 0, p.wait_limit);
    ok = __all_sync(0xffffffffu, ok);
    if (!ok && lane == 0) atomicExch(p.status, 13);
    tc_fence_after();
    if (ok) {
#pragma unroll 1
      for (int c = 0; c < BN2 / 32; ++c) {
        uint32_t r[32];
        __syncwarp();
        tmem_ld_32x32(tmem_base + (uint32_t(q * 32) << 16) + uint32_t(c * 32), r);
        tmem_ld_wait();
#pragma unroll
        for (int g = 0; g < 8; ++g)
          *reinterpret_cast<uint4*>(tile + lane * EPI_PITCH + g * 4) = make_uint4(r[4 * g], r[4 * g + 1], r[4 * g + 2], r[4 * g + 3]);
        __syncwarp();
        const int n = tm.n0 + c * 32 + sub_col;
        if constexpr (upd) {
          WmRegs nxt;
          if (c + 1 < BN2 / 32) load_wm(p, row0, n + 32, tm.nlim, sub_row, nxt);
          apply_update(p, row0, n, tm.nlim, sub_row, tile, sub_col, cur);
          cur = nxt;
        } else {
          epilogue_rows8<MODE>(p, tm, tile, q, sub_row, sub_col, n);
        }
      }
    }
    }
  }
  // neither CTA may release shared or tensor memory while its partner can still touch it
  if (threadIdx.x == 64) phase_mark(p, 5);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (threadIdx.x == 0) phase_mark(p, 6);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc2(tmem_base, GEMM2_BN);
    if (lane == 0) tmem_note_freed(TK_PAIR, GEMM2_BN);
    if (lane == 0) phase_mark(p, 7);
  }
}

}  // namespace lp
