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
// so the update of tile i (an HBM stream) runs under the main loop of tile i + 1.  An epilogue lane
// owns one row of the chunk: it reads its 128 bytes of master (and momentum) from the slot, applies
// Eq. 6 to its accumulator row and writes master, momentum and the bf16 image straight to global
// memory with 32-byte stores -- the results do not pass through shared memory again.  (The SM-pair
// main loop already uses most of the shared-memory bandwidth: 48 KiB read by the tensor core and
// 32 KiB written by TMA per k-block; an update staged in shared memory and sent back with TMA stores
// added 25 % to that traffic and the same 25 % to the kernel's time.)
//
// Barriers.  full[s] (leader; both CTAs' operand loads complete on it), empty[s] (each CTA; released by
// tcgen05.commit multicast), accf[b] (each CTA; accumulator b complete, commit multicast), acce[b]
// (leader; eight arrivals: the four epilogue warps of each CTA have read accumulator b out of tensor
// memory), ufull[u] / uempty[u] (each CTA's own chunk slots; 128 arrivals free a slot).  Every wait is bounded.
#pragma once
#include "gemm2.cuh"

namespace lp {

constexpr int GEMM2P_THREADS = 224;
constexpr int GEMM2P_STAGE = 32 * 1024;
constexpr int GEMM2P_POOL = 6 * GEMM2P_STAGE;        // operand stages (32 KiB each) + chunk slots (16 KiB, 32 KiB with momentum) share 192 KiB
constexpr int GEMM2P_MAX_SO = 6, GEMM2P_MAX_SC = 8;
constexpr int GEMM2P_SMEM_BYTES = GEMM2P_POOL + 1024 + 1024;

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
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + GEMM2P_POOL);
  uint64_t* empty_bar = full_bar + SO_MAX;
  uint64_t* accf_bar = empty_bar + SO_MAX;    // [2]
  uint64_t* acce_bar = accf_bar + 2;          // [2]
  uint64_t* ufull_bar = acce_bar + 2;         // [SC]
  uint64_t* uempty_bar = ufull_bar + SC_MAX;  // [SC]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(uempty_bar + SC_MAX);

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
      mbar_init(&uempty_bar[u], 128);     // every epilogue thread has read its row of the slot
    }
    fence_barrier_init();
  }
  if (warp == 1) {
    if (lane == 0) tmem_note_enter(TK_PAIR_G);
    tmem_alloc2(tmem_slot, 512);
    if (lane == 0) tmem_note_got(TK_PAIR_G, 512);
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
  } else {
    // ------------------------------------------------------------ epilogue (warps 2-5 of both CTAs, own 128 rows)
    const int q = warp & 3;                                     // tensor-memory lane quarter this warp may read
    const int trow = q * 32 + lane;                             // row of this CTA's half tile = tensor-memory lane
    const uint32_t chunk0 = smem_u32(chunk_mem);
    const uint32_t accf0 = smem_u32(accf_bar), ufull0 = smem_u32(ufull_bar), uempty0 = smem_u32(uempty_bar);
    const uint32_t acce_leader = map_to_cta(smem_u32(acce_bar), 0);
    const bool ring32 = (p.ld_out & 15) == 0;                   // rows of the bf16 image start on 32-byte boundaries
    bool good = true;
    uint32_t it = 0, u = 0, uph = 0;                            // tile count, chunk slot / phase
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
      const int grow = m0 + trow;
      const bool row_ok = grow < p.M;
      const size_t rowbase = size_t(row_ok ? grow : 0) * p.ld_out;
#pragma unroll 1
      for (int c = 0; c < kChunks; ++c) {
        const uint32_t sW = chunk0 + u * slot_bytes;
        const uint32_t sM = sW + UPD_CHUNK_BYTES;               // (momentum form only)
        good = mbar_wait_addr(ufull0 + 8u * u, uph, p.wait_limit);
        good = __all_sync(0xffffffffu, good);
        if (!good) {
          if (lane == 0) atomicExch(p.status, 19);
          break;
        }
        uint32_t r[32];
        tmem_ld_32x32(tacc + (uint32_t(q * 32) << 16) + uint32_t(c * 32), r);
        // this lane's row of the chunk: 128 bytes of master (and momentum), 128-byte swizzle
        const uint32_t rowoff = uint32_t(trow) * 128u;
        const uint32_t swz = uint32_t(trow & 7);
        float4 w[8], mm[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const uint32_t off = rowoff + ((uint32_t(j) ^ swz) << 4);
          asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(w[j].x), "=f"(w[j].y), "=f"(w[j].z), "=f"(w[j].w) : "r"(sW + off));
          if (mom)
            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(mm[j].x), "=f"(mm[j].y), "=f"(mm[j].z), "=f"(mm[j].w) : "r"(sM + off));
        }
        tmem_ld_wait();
        if (c == kChunks - 1) {
          // last read of this accumulator: hand it back to the MMA issuer (in the leader CTA)
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(acce_leader + 8u * buf);
        }
        const int nc = n0 + c * 32;
        uint32_t packed[16];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float g[4] = {__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]), __uint_as_float(r[4 * j + 2]),
                              __uint_as_float(r[4 * j + 3])};
          float m[4] = {g[0], g[1], g[2], g[3]};
          if (mom) {
            m[0] = p.mu * mm[j].x + g[0]; m[1] = p.mu * mm[j].y + g[1];
            m[2] = p.mu * mm[j].z + g[2]; m[3] = p.mu * mm[j].w + g[3];
            mm[j] = make_float4(m[0], m[1], m[2], m[3]);
          }
          w[j].x -= p.lr * m[0]; w[j].y -= p.lr * m[1]; w[j].z -= p.lr * m[2]; w[j].w -= p.lr * m[3];
          packed[2 * j] = pack_bf16x2(w[j].x, w[j].y);
          packed[2 * j + 1] = pack_bf16x2(w[j].z, w[j].w);
        }
        // The slot is handed back only here, after the arithmetic above has consumed every value read from it:
        // an arrive issued right behind the ld.shared instructions let the refill overwrite, now and then,
        // the last 16-byte units before those loads had read them (free-running runs differed from
        // serialised ones in a few float4 per million).
        mbar_arrive_addr(uempty0 + 8u * u);
        if (row_ok) {
          // 32-byte stores: eight fp32 (or sixteen bf16) of this lane's row per instruction, whole sectors
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int n = nc + 8 * j;
            if (n >= p.N) continue;                      // (columns up to the padded pitch exist and stay zero)
            if (p.out != nullptr) {
              float* dst = reinterpret_cast<float*>(p.out) + rowbase + n;
              asm volatile("st.global.cs.v8.f32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "f"(__uint_as_float(r[8 * j])),
                           "f"(__uint_as_float(r[8 * j + 1])), "f"(__uint_as_float(r[8 * j + 2])), "f"(__uint_as_float(r[8 * j + 3])),
                           "f"(__uint_as_float(r[8 * j + 4])), "f"(__uint_as_float(r[8 * j + 5])), "f"(__uint_as_float(r[8 * j + 6])),
                           "f"(__uint_as_float(r[8 * j + 7]))
                           : "memory");
            }
            asm volatile("st.global.cs.v8.f32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p.W + rowbase + n), "f"(w[2 * j].x),
                         "f"(w[2 * j].y), "f"(w[2 * j].z), "f"(w[2 * j].w), "f"(w[2 * j + 1].x), "f"(w[2 * j + 1].y), "f"(w[2 * j + 1].z),
                         "f"(w[2 * j + 1].w)
                         : "memory");
            if (mom)
              asm volatile("st.global.cs.v8.f32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p.mW + rowbase + n), "f"(mm[2 * j].x),
                           "f"(mm[2 * j].y), "f"(mm[2 * j].z), "f"(mm[2 * j].w), "f"(mm[2 * j + 1].x), "f"(mm[2 * j + 1].y),
                           "f"(mm[2 * j + 1].z), "f"(mm[2 * j + 1].w)
                           : "memory");
          }
          __nv_bfloat16* rdst = p.ring + rowbase + nc;
          if (ring32) {
#pragma unroll
            for (int j = 0; j < 2; ++j)
              if (nc + 16 * j < p.N)
                asm volatile("st.global.cs.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(rdst + 16 * j), "r"(packed[8 * j]),
                             "r"(packed[8 * j + 1]), "r"(packed[8 * j + 2]), "r"(packed[8 * j + 3]), "r"(packed[8 * j + 4]),
                             "r"(packed[8 * j + 5]), "r"(packed[8 * j + 6]), "r"(packed[8 * j + 7])
                             : "memory");
          } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
              if (nc + 8 * j < p.N)
                *reinterpret_cast<uint4*>(rdst + 8 * j) = make_uint4(packed[4 * j], packed[4 * j + 1], packed[4 * j + 2], packed[4 * j + 3]);
          }
        }
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
    if (lane == 0) tmem_note_freed(TK_PAIR_G, 512);
  }
}

}  // namespace lp
