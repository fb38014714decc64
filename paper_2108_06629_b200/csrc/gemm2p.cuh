// Persistent form of the SM-pair G kernel (Eq. 5 with Eq. 6 in its epilogue) for contractions with
// many short tiles: G of a fully connected layer contracts over the minibatch, so a tile of the
// 8192 x 8192 gradient at batch 2048 is only 32 k-blocks long and a one-tile CTA spends a third of
// its life outside the main loop (launch, tensor-memory allocation, pipeline ramp, update epilogue).
//
// One CTA pair per SM pair walks tiles pair_id, pair_id + pairs, ...:
//   warp 0     operand producer (TMA, ring of SO stages, runs on across tile boundaries)
//   warp 1     MMA issuer (leader CTA), accumulators double-buffered in tensor memory (2 x 256 columns)
//   warps 2-5  epilogue: Eq. 6 on the accumulator against master / momentum chunks in shared memory
//   warp 6     update-tile producer: streams the fp32 master (and momentum) of the tiles, one 128 x 32
//              chunk per fill, through chunk slots of its own (64 KiB: four slots, or two with
//              momentum), independent of the operand ring and as far ahead as the slots allow
//   warp 7     store issuer: sends every updated chunk (master, momentum, bf16 image) back with TMA
//              stores and frees its slot as soon as the stores have read it
// so the update of tile i (an HBM stream) runs under the main loop of tile i + 1.
//
// Barriers.  full[s] (leader; both CTAs' operand loads complete on it), empty[s] (each CTA; released by
// tcgen05.commit multicast), accf[b] (each CTA; accumulator b complete, commit multicast), acce[b]
// (leader; eight arrivals: the four epilogue warps of each CTA have read accumulator b out of tensor
// memory), ufull[u] / uempty[u] (each CTA's own chunk slots), staged[k] / sfree[k] (the two bf16 staging
// tiles between the epilogue warps and the store issuer).  Every wait is bounded.
#pragma once
#include "gemm2.cuh"

namespace lp {

constexpr int GEMM2P_THREADS = 256;
constexpr int GEMM2P_STAGE = 32 * 1024;
constexpr int GEMM2P_POOL = 6 * GEMM2P_STAGE;        // operand stages (32 KiB each) + chunk slots (16 KiB, 32 KiB with momentum) share 192 KiB
constexpr int GEMM2P_MAX_SO = 6, GEMM2P_MAX_SC = 8;
constexpr int GEMM2P_SMEM_BYTES = GEMM2P_POOL + 2 * UPD_RING_BYTES + 1024 + 1024;

__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}

template <int kInstance = 0>
__global__ void __launch_bounds__(GEMM2P_THREADS, 1)
gemm2p_g_update_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                       const __grid_constant__ UpdMaps um, const GemmArgs p, const int tiles_m, const int tiles_n) {
  constexpr int STAGE = GEMM2P_STAGE, SC_MAX = GEMM2P_MAX_SC, SO_MAX = GEMM2P_MAX_SO;
  const int SO = p.num_stages;                             // operand stages; the rest of the pool holds chunk slots
  constexpr int kChunks = GEMM2_BN / 32;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* chunk_mem = smem + SO * STAGE;
  uint8_t* ring_mem = smem + GEMM2P_POOL;                             // two bf16 staging tiles (8 KiB each)
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(ring_mem + 2 * UPD_RING_BYTES);
  uint64_t* empty_bar = full_bar + SO_MAX;
  uint64_t* accf_bar = empty_bar + SO_MAX;    // [2]
  uint64_t* acce_bar = accf_bar + 2;          // [2]
  uint64_t* ufull_bar = acce_bar + 2;         // [SC]
  uint64_t* uempty_bar = ufull_bar + SC_MAX;  // [SC]
  uint64_t* staged_bar = uempty_bar + SC_MAX; // [2] a staging tile (and its chunk slot) is ready to be stored
  uint64_t* sfree_bar = staged_bar + 2;       // [2] a staging tile may be written again
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sfree_bar + 2);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int num_kb = (p.K + GEMM_BK - 1) / GEMM_BK;
  const int total = tiles_m * tiles_n;                     // 256 x 256 tiles
  const int pair_id = int(blockIdx.x >> 1), pairs = int(gridDim.x >> 1);
  const bool mom = p.mW != nullptr;
  const uint32_t slot_bytes = mom ? 2u * UPD_CHUNK_BYTES : uint32_t(UPD_CHUNK_BYTES);
  const int SC = min(SC_MAX, int((GEMM2P_POOL - SO * STAGE) / slot_bytes));      // chunk slots

  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
    tma_prefetch_desc(&um.W);
    if (p.mW != nullptr) tma_prefetch_desc(&um.M);
    tma_prefetch_desc(&um.R);
    for (int s = 0; s < SO; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&accf_bar[b], 1);
      mbar_init(&acce_bar[b], 8);
    }
    for (int u = 0; u < SC_MAX; ++u) {
      mbar_init(&ufull_bar[u], 1);
      mbar_init(&uempty_bar[u], 1);
    }
    for (int k = 0; k < 2; ++k) {
      mbar_init(&staged_bar[k], 128);
      mbar_init(&sfree_bar[k], 1);
    }
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc2(tmem_slot, 512);
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
        const int m0 = (t % tiles_m) * 256 + int(rank) * 128;        // this CTA's 128 rows of A
        const int nb0 = (t / tiles_m) * GEMM2_BN + int(rank) * 128;  // the half of B this CTA stages
        int k0 = 0;
        for (int kb = 0; kb < num_kb; ++kb, k0 += GEMM_BK) {
          ok = mbar_wait_addr(empty0 + 8u * s, ph ^ 1u, p.wait_limit);
          if (!ok) break;
          const uint32_t sa = smem0 + s * uint32_t(STAGE);
          const uint32_t sb = sa + GEMM_A_BYTES;
          const uint32_t fb = map_to_cta(full0 + 8u * s, 0);          // the leader's barrier
          if (rank == 0) mbar_arrive_expect_tx_addr(full0 + 8u * s, 2 * STAGE);
#pragma unroll
          for (int c = 0; c < 2; ++c) tma2_load_2d_addr(sa + c * 8192, &tmA, fb, m0 + c * 64, k0);
#pragma unroll
          for (int c = 0; c < 2; ++c) tma2_load_2d_addr(sb + c * 8192, &tmB, fb, nb0 + c * 64, k0);
          ++issued;
          if (++s == uint32_t(SO)) { s = 0; ph ^= 1u; }
        }
      }
      if (!ok) {
        atomicExch(p.status, 15);
        // let copies already in flight land before the CTA's shared memory is released
        if (rank == 0)
          for (long long i = (issued > SO ? issued - SO : 0); i < issued; ++i) mbar_wait(&full_bar[i % SO], uint32_t(i / SO) & 1u, p.wait_limit);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (leader only)
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(256, GEMM2_BN, true, true);
      const uint64_t dA = make_smem_desc(smem_u32(smem), 8192, 1024);
      const uint64_t dB = make_smem_desc(smem_u32(smem) + GEMM_A_BYTES, 8192, 1024);
      const uint32_t dA_hi = uint32_t(dA >> 32), dB_hi = uint32_t(dB >> 32);
      constexpr uint32_t step = 2048 >> 4;
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
        const uint32_t tacc = tmem_base + buf * uint32_t(GEMM2_BN);
        uint32_t acc = 0;
        for (int kb = 0; kb < num_kb; ++kb) {
          ok = mbar_wait_addr(full0 + 8u * s, ph, p.wait_limit);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int j = 0; j < GEMM_BK / 16; ++j) {
            umma2_f16_lohi(tacc, dA_lo + j * step, dA_hi, dB_lo + j * step, dB_hi, idesc, acc);
            acc = 1;
          }
          umma2_commit_both(empty0 + 8u * s);
          dA_lo += uint32_t(STAGE >> 4);
          dB_lo += uint32_t(STAGE >> 4);
          if (++s == uint32_t(SO)) {
            s = 0;
            ph ^= 1u;
            dA_lo = uint32_t(dA);
            dB_lo = uint32_t(dB);
          }
        }
        umma2_commit_both(accf0 + 8u * buf);      // accumulator complete in both CTAs (also releases the epilogues on error)
      }
      if (!ok) atomicExch(p.status, 16);
    }
  } else if (warp == 6) {
    // ------------------------------------------------------------ update-tile producer (both CTAs)
    if (lane == 0) {
      bool ok = true;
      long long issued = 0;
      const uint32_t chunk0 = smem_u32(chunk_mem);
      const uint32_t ufull0 = smem_u32(ufull_bar), uempty0 = smem_u32(uempty_bar);
      uint32_t u = 0, uph = 0;
      for (int t = pair_id; t < total && ok; t += pairs) {
        const int m0 = (t % tiles_m) * 256 + int(rank) * 128;
        const int n0 = (t / tiles_m) * GEMM2_BN;
        for (int c = 0; c < kChunks; ++c) {
          ok = mbar_wait_addr(uempty0 + 8u * u, uph ^ 1u, p.wait_limit);
          if (!ok) break;
          const uint32_t dst = chunk0 + u * slot_bytes;
          const uint32_t ub = ufull0 + 8u * u;
          mbar_arrive_expect_tx_addr(ub, slot_bytes);
          tma_load_2d_addr(dst, &um.W, ub, n0 + c * 32, m0);
          if (mom) tma_load_2d_addr(dst + UPD_CHUNK_BYTES, &um.M, ub, n0 + c * 32, m0);
          ++issued;
          if (++u == uint32_t(SC)) { u = 0; uph ^= 1u; }
        }
      }
      if (!ok) {
        atomicExch(p.status, 17);
        for (long long i = (issued > SC ? issued - SC : 0); i < issued; ++i) mbar_wait(&ufull_bar[i % SC], uint32_t(i / SC) & 1u, p.wait_limit);
      }
    }
  } else if (warp == 7) {
    // ------------------------------------------------------------ store issuer (both CTAs)
    if (lane == 0) {
      bool ok = true;
      const uint32_t chunk0 = smem_u32(chunk_mem), ring0 = smem_u32(ring_mem);
      const uint32_t staged0 = smem_u32(staged_bar), sfree0 = smem_u32(sfree_bar), uempty0 = smem_u32(uempty_bar);
      uint32_t u = 0, gc = 0, prev_u = 0;
      for (int t = pair_id; t < total && ok; t += pairs) {
        const int m0 = (t % tiles_m) * 256 + int(rank) * 128;
        const int n0 = (t / tiles_m) * GEMM2_BN;
        for (int c = 0; c < kChunks; ++c, ++gc) {
          const uint32_t k = gc & 1u;
          ok = mbar_wait_addr(staged0 + 8u * k, (gc >> 1) & 1u, p.wait_limit);
          if (!ok) break;
          const uint32_t sW = chunk0 + u * slot_bytes;
          const int n = n0 + c * 32;
          tma_store_2d_addr(&um.W, sW, n, m0);
          if (mom) tma_store_2d_addr(&um.M, sW + UPD_CHUNK_BYTES, n, m0);
          tma_store_2d_addr(&um.R, ring0 + k * uint32_t(UPD_RING_BYTES), n, m0);
          tma_store_commit();
          // one group may stay in flight: the stores of the PREVIOUS chunk have read shared memory, so its
          // chunk slot and its staging tile are free
          asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
          if (gc > 0) {
            mbar_arrive_addr(uempty0 + 8u * prev_u);
            mbar_arrive_addr(sfree0 + 8u * (k ^ 1u));
          }
          prev_u = u;
          if (++u == uint32_t(SC)) u = 0;
        }
      }
      tma_store_wait_read0();
      if (ok && gc > 0) {                                // (the last chunk's slot: nobody waits for it any more, kept for symmetry)
        mbar_arrive_addr(uempty0 + 8u * prev_u);
        mbar_arrive_addr(sfree0 + 8u * ((gc - 1) & 1u));
      }
      if (!ok) atomicExch(p.status, 20);
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2-5 of both CTAs, own 128 rows)
    const int q = warp & 3;                                     // tensor-memory lane quarter this warp may read
    const int trow = q * 32 + lane;                             // row of this CTA's half tile = tensor-memory lane
    const uint32_t chunk0 = smem_u32(chunk_mem), ring0 = smem_u32(ring_mem);
    const uint32_t accf0 = smem_u32(accf_bar), ufull0 = smem_u32(ufull_bar);
    const uint32_t staged0 = smem_u32(staged_bar), sfree0 = smem_u32(sfree_bar);
    const uint32_t acce_leader = map_to_cta(smem_u32(acce_bar), 0);
    bool good = true;
    uint32_t it = 0, u = 0, uph = 0, gc = 0;                    // tile count, chunk slot / phase, running chunk count
    for (int t = pair_id; t < total && good; t += pairs, ++it) {
      const int m0 = (t % tiles_m) * 256 + int(rank) * 128;
      const int n0 = (t / tiles_m) * GEMM2_BN;
      const uint32_t buf = it & 1u;
      const uint32_t tacc = tmem_base + buf * uint32_t(GEMM2_BN);
      good = mbar_wait_addr(accf0 + 8u * buf, (it >> 1) & 1u, p.wait_limit);
      good = __all_sync(0xffffffffu, good);
      if (!good) {
        if (lane == 0) atomicExch(p.status, 18);
        break;
      }
      tc_fence_after();
#pragma unroll 1
      for (int c = 0; c < kChunks; ++c, ++gc) {
        const uint32_t k = gc & 1u;
        const uint32_t sW = chunk0 + u * slot_bytes;
        const uint32_t sM = sW + UPD_CHUNK_BYTES;               // (momentum form only)
        const uint32_t ringbuf = ring0 + k * uint32_t(UPD_RING_BYTES);
        // the chunk's master (and momentum) have landed, and the staging tile of two chunks ago has been stored
        good = mbar_wait_addr(ufull0 + 8u * u, uph, p.wait_limit) && mbar_wait_addr(sfree0 + 8u * k, ((gc >> 1) & 1u) ^ 1u, p.wait_limit);
        good = __all_sync(0xffffffffu, good);
        if (!good) {
          if (lane == 0) atomicExch(p.status, 19);
          break;
        }
        uint32_t r[32];
        tmem_ld_32x32(tacc + (uint32_t(q * 32) << 16) + uint32_t(c * 32), r);
        tmem_ld_wait();
        if (c == kChunks - 1) {
          // last read of this accumulator: hand it back to the MMA issuer (in the leader CTA)
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(acce_leader + 8u * buf);
        }
        const uint32_t rowoff = uint32_t(trow) * 128u;
        const uint32_t swz = uint32_t(trow & 7);
        const int grow = m0 + trow;
        uint32_t packed[16];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const uint32_t off = rowoff + ((uint32_t(j) ^ swz) << 4);
          float g[4] = {__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]), __uint_as_float(r[4 * j + 2]),
                        __uint_as_float(r[4 * j + 3])};
          const int n = n0 + c * 32 + 4 * j;
          if (p.out != nullptr && grow < p.M && n < p.N) {
            float* dst = reinterpret_cast<float*>(p.out) + size_t(grow) * p.ld_out + n;
            if (n + 3 < p.N) {
              __stcs(reinterpret_cast<float4*>(dst), make_float4(g[0], g[1], g[2], g[3]));
            } else {
              for (int e = 0; e < 4; ++e) if (n + e < p.N) dst[e] = g[e];
            }
          }
          float m[4] = {g[0], g[1], g[2], g[3]};
          if (mom) {
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
        {
          const uint32_t roff = ringbuf + uint32_t(trow) * 64u;
          const uint32_t rs = uint32_t(trow >> 1) & 3u;
#pragma unroll
          for (int v = 0; v < 4; ++v)
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(roff + ((uint32_t(v) ^ rs) << 4)), "r"(packed[4 * v]),
                         "r"(packed[4 * v + 1]), "r"(packed[4 * v + 2]), "r"(packed[4 * v + 3])
                         : "memory");
        }
        // this thread's part of the chunk is in shared memory: make it visible to the copy engine and
        // tell the store issuer (128 arrivals complete the chunk)
        fence_proxy_async_smem();
        mbar_arrive_addr(staged0 + 8u * k);
        if (++u == uint32_t(SC)) { u = 0; uph ^= 1u; }
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
  }
}

}  // namespace lp
