// 3x3 convolution contractions over few channels (at most 64 on both sides): forward
// (Eqs. 1-2) and delta (Eqs. 3-4) as an implicit GEMM whose activation operand is fetched ONCE
// per tile.
//
// The general kernel loads a 128-pixel x 64-channel box per filter tap, i.e. nine shifted copies
// of nearly the same pixels; with only 64 output columns per tile the tensor cores then wait on
// the ~64 B/clk one SM can pull from L2.  Here a tile is 8 x 16 pixels of one image; its
// 10 x 18 halo box (the pixels the nine taps touch) lands in shared memory once (22.5 KiB), and
// the operand of tap (r, s) is a VIEW of it: the matrix descriptor starts r * 10 + s pixel rows
// into the box, eight consecutive pixels of an image row form one 8-row swizzle group and the
// next group is one box row (10 pixels = 1280 bytes) further.  The
// 128-byte swizzle is a function of the absolute shared-memory address for TMA and for the
// tensor core alike, so a view that starts at any 128-byte row of the box needs nothing else
// (checked tap by tap with one-hot weights: exact with the descriptor's base-offset field left
// zero, chunk-permuted when it is set to the start row).  All nine 64 x 64 weight taps stay resident in shared memory (72 KiB) for the whole
// persistent CTA.  Per tile the SM now reads 22.5 KiB instead of 216 KiB; four boxes are in flight.
//
// The same pipeline also runs the forward GEMM of a layer whose whole contraction fits one
// k-block and whose output is at most 64 columns wide (plain geometry: the patch-matrix form of
// a first convolution layer): one weight "tap", tiles of 128 consecutive rows fetched through a
// 2-D map, the output tile stored through a 2-D map.  Such a layer is 25 000 tiles of a single
// k-block each, and what it needs is this kernel's epilogue.
#pragma once
#include "gemm.cuh"

namespace lp {

constexpr int HALO_W = 10, HALO_H = 18;                       // box: pixels per row (pitch) x rows
constexpr int HALO_STAGES = 4;
constexpr int HALO_BYTES = HALO_W * HALO_H * 128;             // 64 bf16 channels per pixel
constexpr int HALO_TAP_BYTES = 64 * 64 * 2;                   // one weight tap: 64 x 64 bf16
constexpr int HALO_OUT_BYTES = GEMM_BM * 128;                 // forward: one output tile, 128 pixels x 64 bf16 channels
constexpr int HALO_THREADS = 320;                             // producer warp, MMA warp, eight epilogue warps
constexpr int HALO_EPI_BYTES = 2 * EPI_TILE_BYTES;            // forward: two output tiles (32 KiB); delta: eight transposition tiles (36 KiB)
static_assert(HALO_EPI_BYTES >= 2 * HALO_OUT_BYTES, "the epilogue area holds two output tiles");
constexpr int HALO_SMEM_BYTES = 9 * HALO_TAP_BYTES + HALO_STAGES * HALO_BYTES + HALO_EPI_BYTES + 256 + 1024;
static_assert((HALO_STAGES * HALO_BYTES) % 1024 == 0, "the buffers behind the halo boxes stay 1 KiB aligned");

template <bool B_MN, int MODE>
__global__ void __launch_bounds__(HALO_THREADS, 1)
conv_halo_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                 const __grid_constant__ CUtensorMap tmO, const GemmArgs p, const int tiles_total) {
  constexpr int BN = 64;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sB = smem;                                   // [9][64 x 64] weight taps
  uint8_t* sA = smem + 9 * HALO_TAP_BYTES;              // [HALO_STAGES] halo boxes
  uint8_t* sO = sA + HALO_STAGES * HALO_BYTES;                    // forward: [2] output tiles (TMA store sources)
  float* epi_tile = reinterpret_cast<float*>(sO);                 // delta: one transposition tile per epilogue warp (same area)
  uint64_t* bars = reinterpret_cast<uint64_t*>(sO + HALO_EPI_BYTES);
  uint64_t* wfull = bars;          // weights resident
  uint64_t* afull = bars + 1;                       // [HALO_STAGES] halo box landed
  uint64_t* aempty = afull + HALO_STAGES;           // [HALO_STAGES] halo box consumed
  uint64_t* accf = aempty + HALO_STAGES;            // [2] accumulator complete
  uint64_t* acce = accf + 2;                        // [2] accumulator drained
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acce + 2);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
    if (MODE == EPI_FPROP) tma_prefetch_desc(&tmO);
    mbar_init(wfull, 1);
    for (int b = 0; b < HALO_STAGES; ++b) {
      mbar_init(&afull[b], 1);
      mbar_init(&aempty[b], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&accf[b], 1);
      mbar_init(&acce[b], 8);      // one arrival per epilogue warp
    }
    fence_barrier_init();
  }
  if (warp == 1) {
    if (lane == 0) tmem_note_enter(TK_HALO);
    tmem_alloc(tmem_slot, 2 * BN);
    if (lane == 0) tmem_note_got(TK_HALO, 2 * BN);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // CTA b works through the contiguous tile range [t_begin, t_end): neighbouring tiles share halo
  // pixels in L2, and the tile coordinates advance without divisions.
  const bool plain = (p.g.kind == GEOM_PLAIN);          // one tap, 128 consecutive rows per tile
  const int ntaps = plain ? 1 : 9;
  const int tiles_per_image = plain ? 1 : p.g.tiles_w * p.g.tiles_h;
  const int per_cta = (tiles_total + int(gridDim.x) - 1) / int(gridDim.x);
  const int t_begin = min(int(blockIdx.x) * per_cta, tiles_total);
  const int t_end = min(t_begin + per_cta, tiles_total);
  const int tw_begin = plain ? 0 : t_begin % p.g.tiles_w, th_begin = plain ? 0 : (t_begin / p.g.tiles_w) % p.g.tiles_h;
  const int tn_begin = t_begin / tiles_per_image;

  if (warp == 0) {
    if (lane == 0) {
      bool ok = true;
      int issued = 0;
      mbar_arrive_expect_tx(wfull, uint32_t(ntaps) * HALO_TAP_BYTES);
      for (int tap = 0; tap < ntaps; ++tap) tma_load_2d(sB + tap * HALO_TAP_BYTES, &tmB, wfull, tap * p.g.tap_pitch, 0);
      uint32_t st = 0, sph = 0;
      int tw = tw_begin, th = th_begin, n = tn_begin;
      for (int t = t_begin; t < t_end; ++t) {
        ok = mbar_wait(&aempty[st], sph ^ 1u);
        if (!ok) break;
        if (plain) {
          mbar_arrive_expect_tx(&afull[st], GEMM_A_BYTES);
          tma_load_2d(sA + st * HALO_BYTES, &tmA, &afull[st], 0, t * GEMM_BM);
        } else {
          mbar_arrive_expect_tx(&afull[st], HALO_BYTES);
          // the box starts one pixel left of and above the tile; pixels outside the image read zero (= the padding)
          tma_load_4d(sA + st * HALO_BYTES, &tmA, &afull[st], 0, tw * 8 - 1, th * 16 - 1, n);
          if (++tw == p.g.tiles_w) { tw = 0; if (++th == p.g.tiles_h) { th = 0; ++n; } }
        }
        ++issued;
        if (++st == uint32_t(HALO_STAGES)) { st = 0; sph ^= 1u; }
      }
      if (!ok) {
        atomicExch(p.status, 1);
        mbar_wait(wfull, 0);
        for (int i = (issued > HALO_STAGES ? issued - HALO_STAGES : 0); i < issued; ++i)
          mbar_wait(&afull[i % HALO_STAGES], uint32_t(i / HALO_STAGES) & 1u);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(GEMM_BM, BN, false, B_MN);
      constexpr uint32_t stepB = (B_MN ? 2048 : 32) >> 4;
      // One thread issues 36 MMAs per tile, so everything that can be is computed once: the
      // descriptors of box 0 / tap 0, and per tap the start-address offset of its view (the
      // address field counts 16-byte units and never carries out of the low word).
      const uint64_t dA = make_smem_desc(smem_u32(sA), 16, plain ? 1024 : HALO_W * 128);
      const uint64_t dB = B_MN ? make_smem_desc(smem_u32(sB), 8192, 1024) : make_smem_desc(smem_u32(sB), 16, 1024);
      const uint32_t dA_lo0 = uint32_t(dA), dA_hi = uint32_t(dA >> 32), dB_lo0 = uint32_t(dB), dB_hi = uint32_t(dB >> 32);
      uint32_t tap_off[9];
#pragma unroll
      for (int tap = 0; tap < 9; ++tap) {
        int r = tap / 3, s = tap % 3;
        if (p.g.flip) { r = 2 - r; s = 2 - s; }        // delta: the tap's shift is mirrored
        tap_off[tap] = uint32_t(r * HALO_W + s) * (128u >> 4);
      }
      bool ok = mbar_wait(wfull, 0);
      uint32_t it = 0, st = 0, sph = 0;
      for (int t = t_begin; t < t_end && ok; ++t, ++it) {
        const uint32_t buf = it & 1u;
        ok = mbar_wait(&acce[buf], ((it >> 1) & 1u) ^ 1u);
        if (!ok) break;
        ok = mbar_wait(&afull[st], sph);
        if (!ok) break;
        tc_fence_after();
        const uint32_t tacc = tmem_base + buf * uint32_t(BN);
        const uint32_t a_lo = dA_lo0 + st * uint32_t(HALO_BYTES >> 4);
        uint32_t acc = 0;
#pragma unroll
        for (int tap = 0; tap < 9; ++tap) {
          if (tap >= ntaps) break;
#pragma unroll
          for (int j = 0; j < GEMM_BK / 16; ++j) {
            umma_f16_lohi(tacc, a_lo + tap_off[tap] + uint32_t(j * 2), dA_hi,
                          dB_lo0 + uint32_t(tap) * uint32_t(HALO_TAP_BYTES >> 4) + uint32_t(j) * stepB, dB_hi, idesc, acc);
            acc = 1;
          }
        }
        umma_commit(&aempty[st]);
        umma_commit(&accf[buf]);
        if (++st == uint32_t(HALO_STAGES)) { st = 0; sph ^= 1u; }
      }
      if (!ok) atomicExch(p.status, 2);
    }
  } else {
    // Eight warps: warp w reads tensor-memory lanes 32 * (w % 4) (the rows of its quarter of the
    // tile) and takes columns 32 * half .. + 32.  With one warp per scheduler there is nothing to
    // hide an instruction's latency behind, so the epilogue is spread as wide as the tile allows.
    const int q = warp & 3;
    const int half = (warp - 2) >> 2;
    float* tile = epi_tile + (warp - 2) * (32 * EPI_PITCH);
    const int sub_row = lane >> 3;
    const int sub_col = (lane & 7) * 4;
    uint32_t it = 0;
    bool dead = false;      // a wait ran out: keep the named-barrier count, touch nothing else
    // the bias of this warp's 32 output channels does not depend on the tile (rows are padded to 8 with zeros)
    float4 bias4[8];
#pragma unroll
    for (int g = 0; g < 8; ++g) {
      const int n = half * 32 + 4 * g;
      bias4[g] = (MODE == EPI_FPROP && p.bias != nullptr && n < p.N) ? __ldg(reinterpret_cast<const float4*>(p.bias + n))
                                                                     : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    int tw = tw_begin - 1, th = th_begin, tn = tn_begin;
    for (int t = t_begin; t < t_end; ++t, ++it) {
      const uint32_t buf = it & 1u;
      if (!plain && ++tw == p.g.tiles_w) { tw = 0; if (++th == p.g.tiles_h) { th = 0; ++tn; } }
      TileMap tm;
      tm.m0 = t * GEMM_BM;            // (plain geometry)
      tm.n0 = 0;
      tm.nlim = p.N;
      tm.pw0 = tw * 8;
      tm.ph0 = th * 16;
      tm.pn0 = tn;
      if (!dead) {
        bool ok = mbar_wait(&accf[buf], (it >> 1) & 1u);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) {
          if (lane == 0) atomicExch(p.status, 3);
          dead = true;
        }
      }
      if (dead && MODE != EPI_FPROP) break;      // only the forward epilogue has CTA-wide barriers
      tc_fence_after();
      const uint32_t tacc = tmem_base + buf * uint32_t(BN);
      if constexpr (MODE == EPI_FPROP) {
        // Forward: a lane keeps its accumulator row (one pixel), adds the bias, applies f, and
        // writes the 64 bf16 channels as one 128-byte swizzled row of a shared-memory tile that a
        // TMA store sends to the NHWC output (8 x 16 pixel box) -- no transposition, no address
        // arithmetic per element, and the global writes are whole lines.
        const int trow = q * 32 + lane;
        const uint32_t so = smem_u32(sO) + buf * uint32_t(HALO_OUT_BYTES) + uint32_t(trow) * 128u;
        const uint32_t swz = uint32_t(trow & 7);
        uint32_t packed[16];
        if (!dead) {
          uint32_t r[32];
          tmem_ld_32x32(tacc + (uint32_t(q * 32) << 16) + uint32_t(half * 32), r);
          tmem_ld_wait();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&acce[buf]);
#pragma unroll
          for (int g = 0; g < 8; ++g) {
            const int n = half * 32 + 4 * g;
            float v[4] = {__uint_as_float(r[4 * g]) + bias4[g].x, __uint_as_float(r[4 * g + 1]) + bias4[g].y,
                          __uint_as_float(r[4 * g + 2]) + bias4[g].z, __uint_as_float(r[4 * g + 3]) + bias4[g].w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              if (n + e >= p.N) v[e] = 0.f;
              else if (p.act == ACT_RELU) v[e] = fmaxf(v[e], 0.f);
            }
            packed[2 * g] = pack_bf16x2(v[0], v[1]);
            packed[2 * g + 1] = pack_bf16x2(v[2], v[3]);
          }
        }
        // the staging tile of two tiles ago must have been read by its store
        if (threadIdx.x == 64) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (!dead) {
#pragma unroll
          for (int u = 0; u < 4; ++u)
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(so + ((uint32_t(half * 4 + u) ^ swz) << 4)), "r"(packed[4 * u]),
                         "r"(packed[4 * u + 1]), "r"(packed[4 * u + 2]), "r"(packed[4 * u + 3])
                         : "memory");
        }
        fence_proxy_async_smem();
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (threadIdx.x == 64 && !dead) {
          if (plain) {
            tma_store_2d_addr(&tmO, smem_u32(sO) + buf * uint32_t(HALO_OUT_BYTES), 0, tm.m0);
          } else {
            asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4, %5}], [%1];" ::"l"(
                             reinterpret_cast<uint64_t>(&tmO)),
                         "r"(smem_u32(sO) + buf * uint32_t(HALO_OUT_BYTES)), "r"(0), "r"(tm.pw0), "r"(tm.ph0), "r"(tm.pn0)
                         : "memory");
          }
          tma_store_commit();
        }
        continue;
      }
      {
        const int c = half;
        uint32_t r[32];
        __syncwarp();
        tmem_ld_32x32(tacc + (uint32_t(q * 32) << 16) + uint32_t(c * 32), r);
        tmem_ld_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&acce[buf]);
#pragma unroll
        for (int g = 0; g < 8; ++g)
          *reinterpret_cast<uint4*>(tile + lane * EPI_PITCH + g * 4) = make_uint4(r[4 * g], r[4 * g + 1], r[4 * g + 2], r[4 * g + 3]);
        __syncwarp();
        const int n = c * 32 + sub_col;
        epilogue_rows8<MODE>(p, tm, tile, q, sub_row, sub_col, n);
      }
    }
  }
  if (MODE == EPI_FPROP && threadIdx.x == 64) tma_store_wait_read0();   // shared memory must outlive the stores' reads
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 2 * BN);
    if (lane == 0) tmem_note_freed(TK_HALO, 2 * BN);
  }
}

// ---------------------------------------------------------------------------------------------
// G (Eq. 5) of the same layers: G[co][tap][ci] = sum over pixels of delta[px][co] a[px + tap][ci].
//
// The general kernel gives every (tap, 64-pixel k-block) its own pair of TMA loads, so the nine
// taps re-read delta and the activations nine times through L2, and with 64 output channels
// only half of each 128-row MMA is used.  Here the contraction runs over 8 x 16 pixel tiles:
// per tile one delta box (128 pixels x 64 channels, 16 KiB) and one activation halo box
// (22.5 KiB) are fetched, and the TRANSPOSED gradient is accumulated,
//   D[m = (tap pair half, ci)][n = co] += sum_px  A[px][m] B[px][n],
// with A = two shifted views of the halo box side by side (the descriptor's leading-dimension
// stride, the distance between the two 64-wide halves of M, is the distance between the two
// taps: one pixel = 128 bytes, or 1024 bytes from tap (r, 2) to tap (r + 1, 0)) and B = the delta
// box.  Nine taps = four pairs and a single: five accumulators of 64 columns stay in tensor
// memory over ALL tiles of the CTA; at the end each CTA writes its 5 x 128 x 64 partial sums and
// a second small kernel adds the CTAs' partials in CTA order and applies Eq. 6.  A layer with
// 128 output channels takes two such passes (64 channels each).
constexpr int HALOG_STAGES = 5;                                 // 201 KiB: this CTA takes all 512 tensor-memory columns, so no other kernel that allocates any may fit beside it
constexpr int HALOG_D_OFF = 24576;                              // delta box behind the halo box (1 KiB aligned)
constexpr int HALOG_STAGE_BYTES = HALOG_D_OFF + GEMM_A_BYTES;   // 40 KiB
constexpr int HALOG_SMEM_BYTES = HALOG_STAGES * HALOG_STAGE_BYTES + 256 + 1024;
constexpr int HALOG_GROUPS = 5;
constexpr int HALOG_PART_FLOATS = HALOG_GROUPS * GEMM_BM * 64;  // partial sums of one CTA

template <int kInstance = 0>   // (a template only so that the header may be included by several translation units)
__global__ void __launch_bounds__(GEMM_THREADS, 1)
conv_halo_g_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmD, const ConvGeom g,
                   const int tiles_total, const int co0, float* __restrict__ partial, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + HALOG_STAGES * HALOG_STAGE_BYTES);
  uint64_t* full = bars;
  uint64_t* empty = bars + HALOG_STAGES;
  uint64_t* accf = empty + HALOG_STAGES;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(accf + 1);
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tmX);
    tma_prefetch_desc(&tmD);
    for (int b = 0; b < HALOG_STAGES; ++b) {
      mbar_init(&full[b], 1);
      mbar_init(&empty[b], 1);
    }
    mbar_init(accf, 1);
    fence_barrier_init();
  }
  if (warp == 1) {
    if (lane == 0) tmem_note_enter(TK_HALO_G);
    tmem_alloc(tmem_slot, 512);
    if (lane == 0) tmem_note_got(TK_HALO_G, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int per_cta = (tiles_total + int(gridDim.x) - 1) / int(gridDim.x);
  const int t_begin = min(int(blockIdx.x) * per_cta, tiles_total);
  const int t_end = min(t_begin + per_cta, tiles_total);

  if (warp == 0) {
    if (lane == 0) {
      bool ok = true;
      int issued = 0;
      uint32_t st = 0, sph = 0;
      int tw = t_begin % g.tiles_w, th = (t_begin / g.tiles_w) % g.tiles_h, n = t_begin / (g.tiles_w * g.tiles_h);
      for (int t = t_begin; t < t_end; ++t) {
        ok = mbar_wait(&empty[st], sph ^ 1u);
        if (!ok) break;
        uint8_t* base = smem + st * HALOG_STAGE_BYTES;
        mbar_arrive_expect_tx(&full[st], HALO_BYTES + GEMM_A_BYTES);
        tma_load_4d(base, &tmX, &full[st], 0, tw * 8 - 1, th * 16 - 1, n);
        tma_load_4d(base + HALOG_D_OFF, &tmD, &full[st], co0, tw * 8, th * 16, n);   // 64 output channels from co0
        ++issued;
        if (++st == uint32_t(HALOG_STAGES)) { st = 0; sph ^= 1u; }
        if (++tw == g.tiles_w) { tw = 0; if (++th == g.tiles_h) { th = 0; ++n; } }
      }
      if (!ok) {
        atomicExch(status, 21);
        for (int i = (issued > HALOG_STAGES ? issued - HALOG_STAGES : 0); i < issued; ++i)
          mbar_wait(&full[i % HALOG_STAGES], uint32_t(i / HALOG_STAGES) & 1u);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(GEMM_BM, 64, true, true);
      // tap groups: first tap of the group as a halo row offset, and the distance to its partner
      const uint32_t first_row[HALOG_GROUPS] = {0u, 2u, uint32_t(HALO_W + 1), uint32_t(2 * HALO_W), uint32_t(2 * HALO_W + 2)};
      const uint32_t lbo[HALOG_GROUPS] = {128u, uint32_t((HALO_W - 2) * 128), 128u, 128u, 0u};
      uint32_t dA_lo[HALOG_GROUPS], dA_hi[HALOG_GROUPS];
#pragma unroll
      for (int q = 0; q < HALOG_GROUPS; ++q) {
        const uint64_t d = make_smem_desc(smem_u32(smem) + first_row[q] * 128u, lbo[q], HALO_W * 128);
        dA_lo[q] = uint32_t(d);
        dA_hi[q] = uint32_t(d >> 32);
      }
      const uint64_t dB = make_smem_desc(smem_u32(smem) + HALOG_D_OFF, 8192, 1024);
      const uint32_t dB_lo0 = uint32_t(dB), dB_hi = uint32_t(dB >> 32);
      bool ok = true;
      uint32_t st = 0, sph = 0, acc = 0;
      for (int t = t_begin; t < t_end; ++t) {
        ok = mbar_wait(&full[st], sph);
        if (!ok) break;
        tc_fence_after();
        const uint32_t soff = st * uint32_t(HALOG_STAGE_BYTES >> 4);
#pragma unroll
        for (int k = 0; k < 8; ++k) {            // 16 pixels per MMA: two image rows of the tile
#pragma unroll
          for (int q = 0; q < HALOG_GROUPS; ++q)
            umma_f16_lohi(tmem_base + uint32_t(q * 64), dA_lo[q] + soff + uint32_t(k) * uint32_t((2 * HALO_W * 128) >> 4), dA_hi[q],
                          dB_lo0 + soff + uint32_t(k) * (2048u >> 4), dB_hi, idesc, acc);
          acc = 1;
        }
        umma_commit(&empty[st]);
        if (++st == uint32_t(HALOG_STAGES)) { st = 0; sph ^= 1u; }
      }
      if (!ok) atomicExch(status, 22);
      umma_commit(accf);
    }
  } else {
    const int q = warp & 3;
    bool ok = mbar_wait(accf, 0);
    ok = __all_sync(0xffffffffu, ok);
    if (!ok && lane == 0) atomicExch(status, 23);
    tc_fence_after();
    float* dst = partial + size_t(blockIdx.x) * HALOG_PART_FLOATS;
    const bool any = t_end > t_begin;          // a CTA without tiles contributes zeros
    for (int grp = 0; grp < HALOG_GROUPS; ++grp) {
#pragma unroll 1
      for (int c = 0; c < 2; ++c) {
        uint32_t r[32];
        if (ok && any) {
          tmem_ld_32x32(tmem_base + (uint32_t(q * 32) << 16) + uint32_t(grp * 64 + c * 32), r);
          tmem_ld_wait();
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j) r[j] = 0u;
        }
        float4* o = reinterpret_cast<float4*>(dst + (size_t(grp) * GEMM_BM + q * 32 + lane) * 64 + c * 32);
#pragma unroll
        for (int j = 0; j < 8; ++j)
          o[j] = make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]), __uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3]));
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
    if (lane == 0) tmem_note_freed(TK_HALO_G, 512);
  }
}

// Adds the CTAs' partial sums in CTA order and applies Eq. 6 (or only stores G when W is null).
// One thread per element of the transposed accumulators, n (= output channel) fastest, so the
// partial sums are read coalesced; the 64 x 9 x 64 weight elements themselves are scattered.
struct HaloGUpdate {
  const float* partial;
  int n_ctas;
  int co0;                        // first output channel of this pass (layers with more than 64 take several)
  int n_out, n_in, ld_w;          // weight matrix [n_out][9 * tap_pitch], pitch ld_w
  int tap_pitch;
  float* G;                       // may be null
  float* W;                       // null: store G only
  float* mW;                      // may be null
  __nv_bfloat16* ring;
  float lr, mu;
};
template <int kInstance = 0>
__global__ void __launch_bounds__(256) conv_halo_g_update_kernel(const HaloGUpdate a) {
  const int e = blockIdx.x * 256 + threadIdx.x;
  if (e >= HALOG_PART_FLOATS) return;
  const int co = a.co0 + (e & 63), m = (e >> 6) & 127, grp = e >> 13;
  const int half = m >> 6, ci = m & 63;
  const int tap = (grp < 4) ? 2 * grp + half : (half == 0 ? 8 : -1);
  if (tap < 0 || ci >= a.n_in || co >= a.n_out) return;
  float g = 0.f;
  const float* src = a.partial + e;
#pragma unroll 8
  for (int c = 0; c < a.n_ctas; ++c) g += __ldcg(src + size_t(c) * HALOG_PART_FLOATS);
  const size_t off = size_t(co) * a.ld_w + size_t(tap) * a.tap_pitch + ci;
  if (a.G != nullptr) a.G[off] = g;
  if (a.W == nullptr) return;
  float mm = g;
  if (a.mW != nullptr) {
    mm = a.mu * a.mW[off] + g;
    a.mW[off] = mm;
  }
  const float w = a.W[off] - a.lr * mm;
  a.W[off] = w;
  a.ring[off] = __float2bfloat16_rn(w);
}

}  // namespace lp
