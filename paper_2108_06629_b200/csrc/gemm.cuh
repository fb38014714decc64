// Warp-specialised tcgen05 GEMM for sm_100a: D[M][N] = A . B with bf16 operands staged
// in shared memory by TMA (128-byte swizzle), fp32 accumulators in tensor memory, and a
// fused epilogue.  One 128 x BN output tile per CTA.
//
//   warp 0      TMA producer (one elected lane)
//   warp 1      tensor-memory allocation + MMA issue (one elected lane)
//   warps 2-5   epilogue: tcgen05.ld -> shared-memory transpose -> bias / activation / f' /
//               update -> coalesced global accesses
//
// Operand "major" follows the tensor-core convention: K-major = the contraction index is
// contiguous in memory, MN-major = the M (or N) index is contiguous.  With W stored
// [out][in] and activations [batch][features] the three contractions of a layer are
//   forward (Eq. 1)  A = a      K-major,  B = W      K-major
//   delta   (Eq. 4)  A = delta  K-major,  B = W      MN-major
//   G       (Eq. 5)  A = delta  MN-major, B = a      MN-major
// so one copy of each tensor serves all three.
//
// Convolutions (3x3, stride 1, zero padding 1, NHWC activations, weights [Cout][R][S][Cin]) run
// through the same kernel as implicit GEMMs: the producer addresses the activation tensor
// through a 4-D tensor map and shifts the pixel box by the filter tap; coordinates outside
// the image are zero-filled by TMA, which is the padding.  See ConvGeom.
#pragma once
#include <cuda_bf16.h>

#include "ptx.cuh"

namespace lp {

constexpr int GEMM_BM = 128;
constexpr int GEMM_BK = 64;          // 64 bf16 = one 128-byte swizzle row
constexpr int GEMM_THREADS = 192;
constexpr int GEMM_A_BYTES = GEMM_BM * GEMM_BK * 2;   // 16 KiB
constexpr int GEMM_MAX_STAGES = 8;
// SM-pair kernels (cta_group::2 tensor-memory allocations) and single-CTA kernels (cta_group::1) are not
// run side by side by one handle: where they alternated on the same SMs a pair CTA was found, about once
// in 10^6, waiting in tcgen05.alloc for ever on an otherwise idle GPU (every other CTA of its launch
// had its columns, no bounded wait had expired); handles with one kind only never showed it.  The
// handle picks the kind (lp_api.cu, shape_layers).  TMEM_PAIR_ALONE is the measurement mode in which
// a convolutional network runs its wide layers on pairs all the same: a pair CTA then takes 181 - 193
// KiB of shared memory, so that no single-CTA kernel's allocation shares its SM.
enum { TMEM_DEFAULT = 0, TMEM_PAIR_ALONE = 1 };

enum { EPI_STORE_F32 = 0, EPI_FPROP = 1, EPI_DGRAD = 2, EPI_WGRAD_UPDATE = 3, EPI_DGRAD_UNPOOL = 4 };
enum { ACT_NONE = 0, ACT_RELU = 1, ACT_GELU = 2 };

// How the GEMM indices map onto image pixels.
//   GEOM_PLAIN   ordinary matrices.
//   GEOM_PIX_M   forward / delta of a convolution: the 128 rows of a tile are a box of
//                bw x bh x bn pixels (w fastest) of an NHWC tensor; the contraction runs over
//                (filter tap, 64-channel chunk); the A box is shifted by the tap.
//   GEOM_PIX_K   G of a convolution: rows = output channels, columns = (tap, input channel),
//                the contraction runs over boxes of 64 pixels; the B box (activations) is
//                shifted by the tap of the column tile.
enum { GEOM_PLAIN = 0, GEOM_PIX_M = 1, GEOM_PIX_K = 2 };
struct ConvGeom {
  int kind;
  int H, W;              // PIX_M: size of the tensor the tile rows index (the output of the contraction);
                         // PIX_K: size of the pixel grid the contraction runs over (the layer's output grid)
  int lw, lh;            // log2 of the box width / height; images per box = box pixels >> (lw + lh)
  int tiles_w, tiles_h;  // boxes per row / column of the grid the boxes tile
  int S, pad;            // filter width (tap = r*S + s) and padding
  int flip;              // 0: forward / G (input pixel = output pixel * stride + tap - pad); 1: delta
  int chunks_per_tap;    // PIX_M: 64-channel chunks of the A tensor per tap
  int tap_pitch;         // elements between taps inside a row of the weight matrix (padded Cin)
  int n_per_tap;         // PIX_K: column tiles per tap
  // General filters and strides.  stride: the convolution's stride (forward and G fetch the input
  // through a tensor map that steps `stride` pixels; start coordinate = box origin * stride + shift).
  // Delta of a strided layer runs once per residue class (roff_h, roff_w) of the input pixel
  // modulo the stride: the tile rows are the pixels (h*rs + roff_h, w*rs + roff_w) of the H x W
  // tensor, rs = stride, and only the taps r = tap_r0 + tap_step*i, s = tap_s0 + tap_step*j
  // (j < tap_ns) reach such a pixel, from delta pixel (h + (roff_h + pad - r)/stride, ...).
  int stride;            // >= 1
  int rs, roff_h, roff_w;
  int tap_r0, tap_s0, tap_step, tap_ns;   // enumeration of the taps of this launch: k-th tap = (r0 + step*(k / ns), s0 + step*(k % ns))
};

struct GemmArgs {
  int M, N, K;
  int n_begin;              // first output column of this launch (a multiple of the tile width; columns [n_begin, N) are
                            // computed): one piece of a contraction split by output columns (Section III-B, delta' / delta'')
  int num_stages;
  int mode;                 // EPI_*
  int act;                  // ACT_*  (FPROP: f of this layer; DGRAD: f' of the previous layer)
  void* out;                // STORE_F32 / WGRAD_UPDATE: float [M][ld_out]; FPROP: bf16 a^l (may be null); DGRAD: bf16 delta^{l-1}
  int ld_out;
  void* out2;               // FPROP: bf16 stored z^l (GELU) or fp32 z^L (last layer); else null
  int ld_out2;
  int out2_is_f32;
  const float* bias;        // FPROP: fp32 [N] or null
  const __nv_bfloat16* aux; // DGRAD: what f' is evaluated on (stored z for GELU, a for ReLU)
  int ld_aux;
  // EPI_WGRAD_UPDATE: fp32 master / momentum (may be null) / bf16 ring slot, all [M][ld_out];
  // `out` (may be null) additionally receives G
  float* W;
  float* mW;
  __nv_bfloat16* ring;
  float lr, mu;
  // EPI_DGRAD_UNPOOL: the layer below ended in a 2x2 max pool.  Element (row, col) of the product
  // belongs to pooled pixel row * pool_ppr + col / pool_C, channel col % pool_C; it is routed to
  // the window position recorded in pool_idx (and gated by the pooled activation in `aux`),
  // the other three positions of the window receive zero.
  const unsigned char* pool_idx;
  int pool_C, pool_ppr, pool_Hp, pool_Wp;
  // split-K (splits > 1): blockIdx.z owns k-blocks [z*kb_per_split, (z+1)*kb_per_split); every CTA
  // writes its fp32 partial tile to `partial`, the last CTA of a tile to arrive (tile_counter)
  // adds the partials in split order -- a fixed order, so results do not depend on timing --
  // and runs the epilogue.
  int splits, kb_per_split;
  float* partial;           // [tiles][splits][128][BN]
  unsigned* tile_counter;   // [tiles], zero between launches
  ConvGeom g;
  int persistent;           // CTAs loop over tiles (grid sized to the machine) instead of one tile each
  int l2_ahead;             // plain GEMM: k-blocks of the B operand to pull into L2 ahead of the pipeline (0 = off)
  int upd_tma;              // EPI_WGRAD_UPDATE: master / momentum / ring tiles move by TMA through the stage ring
  // EPI_WGRAD_UPDATE with the TMA update: the bias gradient (column sums of delta^l over the batch)
  // and the bias update of Eq. 6, done by the CTAs of the first column tile (bdelta null = off)
  const __nv_bfloat16* bdelta;   // delta^l [brows][bld]
  int bld, brows;
  float *bb, *bmb, *bdb, *bbring;   // bias master, momentum (may be null), gradient, destination ring slot
  int* status;              // device status word: set non-zero if a bounded wait expires
  long long wait_limit;     // SM cycles after which a wait on a barrier gives up (0 at the call = the default, about 2 s)
  int tmem_policy;          // host side only, see TMEM_* below
  int* phase;               // diagnosis of a stall (LP_TRACE_TASKS): eight counters of CTAs past each phase of the pair kernel, or null
  int starve_kb;            // verification of the bounded waits only: the TMA producer skips the last starve_kb k-blocks of
                            // every tile, so the MMA issuer's wait for them must run out (plain GEMM, one tile per CTA)
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

constexpr int EPI_PITCH = 36;                       // floats; 32 + 4 keeps 128-bit accesses conflict-free
constexpr int EPI_TILE_BYTES = 4 * 32 * EPI_PITCH * 4;   // one 32 x 32 staging tile per epilogue warp (18 KiB)
static_assert(EPI_TILE_BYTES <= GEMM_A_BYTES + 64 * GEMM_BK * 2, "staging tiles must fit in one pipeline stage");

// Where a tile's rows and columns live in the output.
struct TileMap {
  int m0, n0;         // first global row / column (plain)
  int nlim;           // columns >= nlim do not exist
  int pn0, ph0, pw0;  // GEOM_PIX_M: first image / row / column of the pixel box
};
// Global row index of tile row `tr` (0..127), or -1 if the row does not exist.
__device__ __forceinline__ int tile_row(const GemmArgs& p, const TileMap& t, int tr) {
  if (p.g.kind != GEOM_PIX_M) {
    const int row = t.m0 + tr;
    return row < p.M ? row : -1;
  }
  // (pixel boxes tile their grid exactly: every row of a tile exists)
  const int w = t.pw0 + (tr & ((1 << p.g.lw) - 1));
  const int h = t.ph0 + ((tr >> p.g.lw) & ((1 << p.g.lh) - 1));
  const int n = t.pn0 + (tr >> (p.g.lw + p.g.lh));
  return (n * p.g.H + h * p.g.rs + p.g.roff_h) * p.g.W + w * p.g.rs + p.g.roff_w;
}

// Bias of four consecutive output columns (zero where there is none).
__device__ __forceinline__ void load_bias4(const GemmArgs& p, int n, int N, float b[4]) {
#pragma unroll
  for (int j = 0; j < 4; ++j) b[j] = (p.bias != nullptr && n + j < N) ? __ldg(p.bias + n + j) : 0.f;
}
// Forward epilogue for columns n..n+3 of one row: z = acc + b; z^L / stored z; a = f(z).
__device__ __forceinline__ void fprop_store4(const GemmArgs& p, int row, int n, int N, const float acc[4], const float b[4]) {
  const int n_pad4 = (N + 3) & ~3;
  float v[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) v[j] = acc[j] + b[j];
  if (p.out2 != nullptr) {
    if (p.out2_is_f32) {
      if (n < n_pad4)
        *reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out2) + size_t(row) * p.ld_out2 + n) = make_float4(v[0], v[1], v[2], v[3]);
    } else {
      *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(p.out2) + size_t(row) * p.ld_out2 + n) =
          make_uint2(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]));
    }
  }
  if (p.out != nullptr) {
    if (p.act == ACT_RELU) {
#pragma unroll
      for (int j = 0; j < 4; ++j) v[j] = fmaxf(v[j], 0.f);
    } else if (p.act == ACT_GELU) {
#pragma unroll
      for (int j = 0; j < 4; ++j) v[j] = gelu_fwd(v[j]);
    }
    *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(p.out) + size_t(row) * p.ld_out + n) =
        make_uint2(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]));
  }
}
// Delta epilogue: delta^{l-1} = (delta^l W) (.) f'(z^{l-1}), one rounding; av = the four stored
// values of z^{l-1} (GELU) or a^{l-1} (ReLU: a > 0 <=> z > 0) at this position.
__device__ __forceinline__ void dgrad_store4(const GemmArgs& p, int row, int n, const float acc[4], uint2 av) {
  float v[4] = {acc[0], acc[1], acc[2], acc[3]};
  if (p.act != ACT_NONE) {
    const float z[4] = {bf16_lo(av.x), bf16_hi(av.x), bf16_lo(av.y), bf16_hi(av.y)};
#pragma unroll
    for (int j = 0; j < 4; ++j) v[j] = (p.act == ACT_RELU) ? (z[j] > 0.f ? v[j] : 0.f) : v[j] * gelu_grad(z[j]);
  }
  *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(p.out) + size_t(row) * p.ld_out + n) =
      make_uint2(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]));
}

// The layer below ended in ReLU + 2x2 max pool: output row `row`, column n of the delta product
// lives on the pooled grid; pooled pixel pp, channel c, and the 2x2 window it came from.
struct UnpoolPos {
  int pp, c, pn, ph, pw;
};
__device__ __forceinline__ UnpoolPos unpool_pos(const GemmArgs& p, int row, int n) {
  UnpoolPos u;
  const int C = p.pool_C;
  u.pp = row * p.pool_ppr + n / C;
  u.c = n % C;
  u.pw = u.pp % p.pool_Wp;
  u.ph = (u.pp / p.pool_Wp) % p.pool_Hp;
  u.pn = u.pp / (p.pool_Wp * p.pool_Hp);
  return u;
}
// Routes four channels of the gradient to the recorded maximum of the window (idx: one byte per
// channel, 0..3), gated by the pooled activation av (ReLU); the three other positions get zeros.
__device__ __forceinline__ void unpool_store4(const GemmArgs& p, const UnpoolPos& u, const float v[4], uint32_t idx, uint2 av) {
  const float a[4] = {bf16_lo(av.x), bf16_hi(av.x), bf16_lo(av.y), bf16_hi(av.y)};
  __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(p.out);
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int oh = 2 * u.ph + (k >> 1), ow = 2 * u.pw + (k & 1);
    float d[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) d[j] = (((idx >> (8 * j)) & 0xFFu) == uint32_t(k) && a[j] > 0.f) ? v[j] : 0.f;
    const size_t off = (size_t(u.pn * 2 * p.pool_Hp + oh) * (2 * p.pool_Wp) + ow) * p.ld_out + u.c;
    *reinterpret_cast<uint2*>(o + off) = make_uint2(pack_bf16x2(d[0], d[1]), pack_bf16x2(d[2], d[3]));
  }
}

// Epilogue for 4 consecutive columns n..n+3 of output row `row`.  Lanes past the column limit
// inside the last 16-byte (fp32) / 8-element (bf16) group are written as zeros; groups that
// start beyond that are skipped.
template <int MODE>
__device__ __forceinline__ void epilogue_store4(const GemmArgs& p, int row, int n, int N, float4 acc) {
  float v[4] = {n + 0 < N ? acc.x : 0.f, n + 1 < N ? acc.y : 0.f, n + 2 < N ? acc.z : 0.f, n + 3 < N ? acc.w : 0.f};
  const int n_pad4 = (N + 3) & ~3, n_pad8 = (N + 7) & ~7;
  if (MODE == EPI_STORE_F32) {
    if (n >= n_pad4) return;
    *reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) + size_t(row) * p.ld_out + n) = make_float4(v[0], v[1], v[2], v[3]);
  } else if (MODE == EPI_FPROP) {
    if (n >= n_pad8) return;
    float b[4];
    load_bias4(p, n, N, b);
    fprop_store4(p, row, n, N, v, b);
  } else if (MODE == EPI_DGRAD) {
    if (n >= n_pad8) return;
    uint2 av = make_uint2(0u, 0u);
    if (p.act != ACT_NONE) av = *reinterpret_cast<const uint2*>(p.aux + size_t(row) * p.ld_aux + n);
    dgrad_store4(p, row, n, v, av);
  } else if (MODE == EPI_DGRAD_UNPOOL) {
    if (n >= N) return;
    const UnpoolPos u = unpool_pos(p, row, n);
    const uint32_t idx = *reinterpret_cast<const uint32_t*>(p.pool_idx + size_t(u.pp) * p.pool_C + u.c);
    const uint2 av = *reinterpret_cast<const uint2*>(p.aux + size_t(u.pp) * p.ld_aux + u.c);
    unpool_store4(p, u, v, idx, av);
  } else {  // EPI_WGRAD_UPDATE (plain form, used after a split-K reduction)
    if (n >= n_pad8) return;
    const size_t off = size_t(row) * p.ld_out + n;
    if (p.out != nullptr) __stcs(reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) + off), make_float4(v[0], v[1], v[2], v[3]));
    float4 w = __ldcs(reinterpret_cast<const float4*>(p.W + off));
    float m[4] = {v[0], v[1], v[2], v[3]};
    if (p.mW != nullptr) {
      const float4 pm = __ldcs(reinterpret_cast<const float4*>(p.mW + off));
      m[0] = p.mu * pm.x + v[0]; m[1] = p.mu * pm.y + v[1]; m[2] = p.mu * pm.z + v[2]; m[3] = p.mu * pm.w + v[3];
      __stcs(reinterpret_cast<float4*>(p.mW + off), make_float4(m[0], m[1], m[2], m[3]));
    }
    w.x -= p.lr * m[0]; w.y -= p.lr * m[1]; w.z -= p.lr * m[2]; w.w -= p.lr * m[3];
    __stcs(reinterpret_cast<float4*>(p.W + off), w);
    *reinterpret_cast<uint2*>(p.ring + off) = make_uint2(pack_bf16x2(w.x, w.y), pack_bf16x2(w.z, w.w));
  }
}

// One lane's share of a transposed 32 x 32 chunk: columns n..n+3 of the eight tile rows
// q*32 + i*4 + sub_row.  The four epilogue warps of a CTA are all the latency hiding there is,
// so what does not depend on the row is fetched once (the bias) and what does is fetched for
// all eight rows before the first store (f' operands): a store may alias a later load as far as
// the compiler knows, and would otherwise serialise eight global round trips.
template <int MODE>
__device__ __forceinline__ void epilogue_rows8(const GemmArgs& p, const TileMap& tm, const float* tile, int q,
                                               int sub_row, int sub_col, int n) {
  int rows[8];
#pragma unroll
  for (int i8 = 0; i8 < 8; ++i8) rows[i8] = tile_row(p, tm, q * 32 + i8 * 4 + sub_row);
  const int N = tm.nlim;
  const int n_pad8 = (N + 7) & ~7;
  if constexpr (MODE == EPI_FPROP) {
    if (n >= n_pad8) return;
    float b[4];
    load_bias4(p, n, N, b);
#pragma unroll
    for (int i8 = 0; i8 < 8; ++i8) {
      if (rows[i8] < 0) continue;
      const float4 a = *reinterpret_cast<const float4*>(tile + (i8 * 4 + sub_row) * EPI_PITCH + sub_col);
      const float v[4] = {n + 0 < N ? a.x : 0.f, n + 1 < N ? a.y : 0.f, n + 2 < N ? a.z : 0.f, n + 3 < N ? a.w : 0.f};
      fprop_store4(p, rows[i8], n, N, v, b);
    }
  } else if constexpr (MODE == EPI_DGRAD) {
    if (n >= n_pad8) return;
    uint2 av[8];
#pragma unroll
    for (int i8 = 0; i8 < 8; ++i8)
      av[i8] = (p.act != ACT_NONE && rows[i8] >= 0) ? *reinterpret_cast<const uint2*>(p.aux + size_t(rows[i8]) * p.ld_aux + n)
                                                    : make_uint2(0u, 0u);
#pragma unroll
    for (int i8 = 0; i8 < 8; ++i8) {
      if (rows[i8] < 0) continue;
      const float4 a = *reinterpret_cast<const float4*>(tile + (i8 * 4 + sub_row) * EPI_PITCH + sub_col);
      const float v[4] = {n + 0 < N ? a.x : 0.f, n + 1 < N ? a.y : 0.f, n + 2 < N ? a.z : 0.f, n + 3 < N ? a.w : 0.f};
      dgrad_store4(p, rows[i8], n, v, av[i8]);
    }
  } else if constexpr (MODE == EPI_DGRAD_UNPOOL) {
    if (n >= N) return;
    UnpoolPos u[8];
    uint32_t idx[8];
    uint2 av[8];
#pragma unroll
    for (int i8 = 0; i8 < 8; ++i8) {
      if (rows[i8] < 0) continue;
      u[i8] = unpool_pos(p, rows[i8], n);
      idx[i8] = *reinterpret_cast<const uint32_t*>(p.pool_idx + size_t(u[i8].pp) * p.pool_C + u[i8].c);
      av[i8] = *reinterpret_cast<const uint2*>(p.aux + size_t(u[i8].pp) * p.ld_aux + u[i8].c);
    }
#pragma unroll
    for (int i8 = 0; i8 < 8; ++i8) {
      if (rows[i8] < 0) continue;
      const float4 a = *reinterpret_cast<const float4*>(tile + (i8 * 4 + sub_row) * EPI_PITCH + sub_col);
      const float v[4] = {n + 0 < N ? a.x : 0.f, n + 1 < N ? a.y : 0.f, n + 2 < N ? a.z : 0.f, n + 3 < N ? a.w : 0.f};
      unpool_store4(p, u[i8], v, idx[i8], av[i8]);
    }
  } else {
#pragma unroll
    for (int i8 = 0; i8 < 8; ++i8) {
      const float4 a = *reinterpret_cast<const float4*>(tile + (i8 * 4 + sub_row) * EPI_PITCH + sub_col);
      if (rows[i8] >= 0) epilogue_store4<MODE>(p, rows[i8], n, N, a);
    }
  }
}

// ---- fused G + update epilogue (EPI_WGRAD_UPDATE, no split-K) -------------------------------
// The accumulator chunk is G; the epilogue streams the fp32 master (and momentum) tile through
// registers: m <- mu m + G; W <- W - eta m; ring <- RN(W).  It is an HBM-streaming loop with
// few warps, so the loads of the NEXT 32 x 32 chunk are issued before the current chunk is
// processed (and those of the first chunk before the accumulator is even complete).
struct WmRegs {
  float4 w[8];
  float4 m[8];
};
__device__ __forceinline__ void load_wm(const GemmArgs& p, int row0, int n, int nlim, int sub_row, WmRegs& r) {
  const bool col_ok = n < ((nlim + 7) & ~7);
#pragma unroll
  for (int it = 0; it < 8; ++it) {
    const int row = row0 + it * 4 + sub_row;
    const bool ok = col_ok && row < p.M;
    const size_t off = size_t(row) * p.ld_out + n;
    r.w[it] = ok ? __ldcs(reinterpret_cast<const float4*>(p.W + off)) : make_float4(0.f, 0.f, 0.f, 0.f);
    if (p.mW != nullptr) r.m[it] = ok ? __ldcs(reinterpret_cast<const float4*>(p.mW + off)) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
}
__device__ __forceinline__ void apply_update(const GemmArgs& p, int row0, int n, int nlim, int sub_row,
                                             const float* tile, int sub_col, const WmRegs& r) {
  if (n >= ((nlim + 7) & ~7)) return;
#pragma unroll
  for (int it = 0; it < 8; ++it) {
    const int rr = it * 4 + sub_row;
    const int row = row0 + rr;
    if (row >= p.M) continue;
    const float4 acc = *reinterpret_cast<const float4*>(tile + rr * EPI_PITCH + sub_col);
    float g[4] = {n + 0 < nlim ? acc.x : 0.f, n + 1 < nlim ? acc.y : 0.f, n + 2 < nlim ? acc.z : 0.f, n + 3 < nlim ? acc.w : 0.f};
    const size_t off = size_t(row) * p.ld_out + n;
    if (p.out != nullptr) __stcs(reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) + off), make_float4(g[0], g[1], g[2], g[3]));
    float m[4] = {g[0], g[1], g[2], g[3]};
    if (p.mW != nullptr) {
      m[0] = p.mu * r.m[it].x + g[0]; m[1] = p.mu * r.m[it].y + g[1];
      m[2] = p.mu * r.m[it].z + g[2]; m[3] = p.mu * r.m[it].w + g[3];
      __stcs(reinterpret_cast<float4*>(p.mW + off), make_float4(m[0], m[1], m[2], m[3]));
    }
    float4 w = r.w[it];
    w.x -= p.lr * m[0]; w.y -= p.lr * m[1]; w.z -= p.lr * m[2]; w.w -= p.lr * m[3];
    __stcs(reinterpret_cast<float4*>(p.W + off), w);
    *reinterpret_cast<uint2*>(p.ring + off) = make_uint2(pack_bf16x2(w.x, w.y), pack_bf16x2(w.z, w.w));
  }
}

// Tensor maps of the fused update's streamed tiles: fp32 master and momentum (boxes of 32
// columns x 128 rows, 128-byte swizzle) and the bf16 ring slot being written (same box,
// 64-byte swizzle).
struct UpdMaps {
  CUtensorMap W, M, R;
};
constexpr int UPD_CHUNK_BYTES = GEMM_BM * 32 * 4;     // one fp32 chunk: 128 rows x 32 columns (16 KiB)
constexpr int UPD_RING_BYTES = GEMM_BM * 32 * 2;      // its bf16 image (8 KiB)

template <int BN>
struct GemmSmem {
  static constexpr int B_BYTES = BN * GEMM_BK * 2;
  static constexpr int STAGE_BYTES = GEMM_A_BYTES + B_BYTES;
  // pipeline stages; then a block of barriers followed by either the epilogue's transposition
  // tiles (persistent CTAs; a one-tile CTA reuses stage 0) or, 1 KiB in, the bf16 staging tile
  // of the TMA update path; alignment slack
  static constexpr size_t bytes(int stages, bool persistent, bool upd_tma = false) {
    const size_t tail = upd_tma ? size_t(1024 + UPD_RING_BYTES) : size_t(256 + (persistent ? EPI_TILE_BYTES : 0));
    return size_t(stages) * STAGE_BYTES + tail + 1024;
  }
};

// One output tile (and, with split-K, one slice of its contraction) of the launch.
struct TileCtx {
  TileMap tm;
  int tap, col0;        // GEOM_PIX_K: filter tap and first input channel of the column tile
  int kb_begin, num_kb; // k-blocks of this work item
  int tile_id, z;       // output tile index and split index
};

template <int BN>
__device__ __forceinline__ TileCtx decode_tile(const GemmArgs& p, int t, int tiles_m, int tiles_n) {
  TileCtx c;
  const int tiles = tiles_m * tiles_n;
  c.z = t / tiles;
  c.tile_id = t - c.z * tiles;
  const int bx = c.tile_id % tiles_m, by = c.tile_id / tiles_m;     // row tiles fastest: neighbours share the B tile
  const int num_kb_total = (p.K + GEMM_BK - 1) / GEMM_BK;
  c.kb_begin = (p.splits > 1) ? c.z * p.kb_per_split : 0;
  c.num_kb = (p.splits > 1) ? max(0, min(num_kb_total, c.kb_begin + p.kb_per_split) - c.kb_begin) : num_kb_total;
  c.tm.m0 = bx * GEMM_BM;
  c.tm.n0 = p.n_begin + by * BN;
  c.tm.nlim = p.N;
  c.tm.pn0 = c.tm.ph0 = c.tm.pw0 = 0;
  c.tap = 0;
  c.col0 = c.tm.n0;
  if (p.g.kind == GEOM_PIX_M) {
    const int tw = bx % p.g.tiles_w, th = (bx / p.g.tiles_w) % p.g.tiles_h, tn = bx / (p.g.tiles_w * p.g.tiles_h);
    c.tm.pw0 = tw << p.g.lw;
    c.tm.ph0 = th << p.g.lh;
    c.tm.pn0 = tn * (GEMM_BM >> (p.g.lw + p.g.lh));
  } else if (p.g.kind == GEOM_PIX_K) {
    c.tap = by / p.g.n_per_tap;
    c.col0 = (by % p.g.n_per_tap) * BN;
    c.tm.n0 = c.tap * p.g.tap_pitch + c.col0;
    c.tm.nlim = c.tap * p.g.tap_pitch + p.g.tap_pitch;     // columns of the next tap belong to another tile
  }
  return c;
}

// Persistent kernel: the grid is sized to the machine (gridDim.x CTAs), CTA b works through
// tiles b, b + gridDim.x, ...  The accumulator is double-buffered in tensor memory (2 x BN
// columns) so that the epilogue of one tile overlaps the main loop of the next, and the
// shared-memory pipeline runs on across tile boundaries.
template <int BN, bool A_MN, bool B_MN, int MODE, bool SPLITK, bool PERSIST, bool UTMA = false>
__global__ void __launch_bounds__(GEMM_THREADS, BN <= 128 ? 2 : 1)
gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const __grid_constant__ UpdMaps um, const GemmArgs p, const int tiles_m, const int tiles_n,
                    const int total_work) {
  using SM = GemmSmem<BN>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int S = p.num_stages;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + size_t(S) * SM::STAGE_BYTES);
  uint64_t* empty_bar = full_bar + GEMM_MAX_STAGES;
  uint64_t* accf_bar = empty_bar + GEMM_MAX_STAGES;     // [2] accumulator buffer full  (MMA -> epilogue)
  uint64_t* acce_bar = accf_bar + 2;                    // [2] accumulator buffer empty (epilogue -> MMA)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acce_bar + 2);
  // Staging tiles of the epilogue.  With one tile per CTA they reuse pipeline stage 0 (by the time
  // the accumulator barrier fires every load has landed and every MMA has read its operands);
  // a CTA that loops over tiles keeps loading while the epilogue runs and needs its own space.
  float* epi_tile = PERSIST ? reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(full_bar) + 256)
                            : reinterpret_cast<float*>(smem);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  // Fused update by TMA (one tile = its k-blocks followed by BN / 32 "chunk fills" of the same
  // stage ring: 128 x 32 fp32 of the master and of the momentum).  The epilogue updates a chunk
  // in place in shared memory and a TMA store writes it back, so the HBM stream of Eq. 6 is
  // queued by the copy engine, many chunks deep, instead of by the registers of four warps.
  // (UTMA is a template parameter, not a flag: the register-path update keeps 128 registers of
  // prefetched tiles per thread, and a kernel that contains both forms is allocated for the larger --
  // two resident CTAs then own the whole register file and no other stream's block fits beside them.)
  static_assert(!UTMA || ((MODE == EPI_WGRAD_UPDATE) && !SPLITK && BN >= 128 && (BN * GEMM_BK * 2 >= UPD_CHUNK_BYTES)),
                "the TMA update needs an unsplit update tile at least 128 columns wide");
  constexpr bool kUpdTmaOk = UTMA;
  constexpr bool upd_tma = UTMA;
  constexpr int kChunks = BN / 32;

  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
    if (upd_tma) {
      tma_prefetch_desc(&um.W);
      if (p.mW != nullptr) tma_prefetch_desc(&um.M);
      tma_prefetch_desc(&um.R);
    }
    for (int s = 0; s < S; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&accf_bar[b], 1);
      mbar_init(&acce_bar[b], 4);      // one arrival per epilogue warp
    }
    fence_barrier_init();
  }
  if (warp == 1) {
    const long long t_alloc = p.phase != nullptr ? clock64() : 0;
    if (lane == 0) tmem_note_enter(PERSIST ? TK_GEMM_PERSISTENT : TK_GEMM);
    tmem_alloc(tmem_slot, PERSIST ? 2 * BN : BN);     // a second accumulator only when tiles follow one another
    if (lane == 0) tmem_note_got(PERSIST ? TK_GEMM_PERSISTENT : TK_GEMM, PERSIST ? 2 * BN : BN);
    if (p.phase != nullptr && lane == 0) {            // (diagnosis: how many allocations had to wait for columns)
      atomicAdd(p.phase + 9, 1);
      if (clock64() - t_alloc > 20000) atomicAdd(p.phase + 8, 1);
    }
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    // One lane runs this loop; everything it needs per k-block is kept in registers as raw
    // 32-bit shared-memory addresses so that the instruction stream between two TMA issues
    // stays short (a single thread issues at a few cycles per instruction).
    if (lane == 0) {
      bool ok = true;
      long long issued = 0;
      const uint32_t smem0 = smem_u32(smem);
      const uint32_t full0 = smem_u32(full_bar), empty0 = smem_u32(empty_bar);
      uint32_t s = 0, ph = 0;
      for (int t = blockIdx.x; t < total_work && ok; t += (PERSIST ? int(gridDim.x) : total_work)) {
        const TileCtx tc = decode_tile<BN>(p, t, tiles_m, tiles_n);
        const TileMap& tm = tc.tm;
        // running position of the contraction
        int k0 = tc.kb_begin * GEMM_BK;                    // plain: element offset along K
        int c_tap = 0, c_chunk = 0;                        // PIX_M: filter tap, 64-channel chunk
        int bw0 = 0, bh0 = 0, bn0 = 0;                     // PIX_K: pixel box of this k-block
        int dh = 0, dw = 0;                                // PIX_K: pixel shift of this tile's tap
        if (p.g.kind == GEOM_PIX_M) {
          c_tap = tc.kb_begin / p.g.chunks_per_tap;
          c_chunk = tc.kb_begin % p.g.chunks_per_tap;
        } else if (p.g.kind == GEOM_PIX_K) {
          const int tw = tc.kb_begin % p.g.tiles_w, th = (tc.kb_begin / p.g.tiles_w) % p.g.tiles_h;
          bw0 = tw << p.g.lw;
          bh0 = th << p.g.lh;
          bn0 = (tc.kb_begin / (p.g.tiles_w * p.g.tiles_h)) * (GEMM_BK >> (p.g.lw + p.g.lh));
          dh = tc.tap / p.g.S - p.g.pad;
          dw = tc.tap % p.g.S - p.g.pad;
        }
        // Weight streaming (small batch): the shared-memory pipeline holds only S k-blocks, not
        // enough to cover an HBM round trip, so the B operand is additionally requested into L2
        // l2_ahead k-blocks early; the pipeline then runs at L2-hit latency.
        const int ahead = (p.g.kind == GEOM_PLAIN) ? p.l2_ahead : 0;
        for (int kb = 0; kb < min(ahead, tc.num_kb); ++kb) {
          const int kk = (tc.kb_begin + kb) * GEMM_BK;
          if (B_MN) {
#pragma unroll
            for (int c = 0; c < BN / 64; ++c) tma_prefetch_l2_2d(&tmB, tm.n0 + c * 64, kk);
          } else {
            tma_prefetch_l2_2d(&tmB, kk, tm.n0);
          }
        }
        for (int kb = 0; kb < tc.num_kb - p.starve_kb; ++kb) {
          if (ahead > 0 && kb + ahead < tc.num_kb) {
            const int kk = k0 + ahead * GEMM_BK;
            if (B_MN) {
#pragma unroll
              for (int c = 0; c < BN / 64; ++c) tma_prefetch_l2_2d(&tmB, tm.n0 + c * 64, kk);
            } else {
              tma_prefetch_l2_2d(&tmB, kk, tm.n0);
            }
          }
          ok = mbar_wait_addr(empty0 + 8u * s, ph ^ 1u, p.wait_limit);
          if (!ok) break;
          const uint32_t sa = smem0 + s * uint32_t(SM::STAGE_BYTES);
          const uint32_t sb = sa + GEMM_A_BYTES;
          const uint32_t fb = full0 + 8u * s;
          mbar_arrive_expect_tx_addr(fb, SM::STAGE_BYTES);
          if (p.g.kind == GEOM_PLAIN) {
            if (A_MN) {
#pragma unroll
              for (int c = 0; c < GEMM_BM / 64; ++c) tma_load_2d_addr(sa + c * 8192, &tmA, fb, tm.m0 + c * 64, k0);
            } else {
              tma_load_2d_addr(sa, &tmA, fb, k0, tm.m0);
            }
            if (B_MN) {
#pragma unroll
              for (int c = 0; c < BN / 64; ++c) tma_load_2d_addr(sb + c * 8192, &tmB, fb, tm.n0 + c * 64, k0);
            } else {
              tma_load_2d_addr(sb, &tmB, fb, k0, tm.n0);
            }
            k0 += GEMM_BK;
          } else if (p.g.kind == GEOM_PIX_M) {
            // A: 128 pixels x 64 channels of the activation / delta tensor, shifted by the tap
            const int r = p.g.tap_r0 + p.g.tap_step * (c_tap / p.g.tap_ns), sft = p.g.tap_s0 + p.g.tap_step * (c_tap % p.g.tap_ns);
            const int wtap = r * p.g.S + sft;         // position of this tap in a row of the weight matrix
            int cw, ch;
            if (p.g.flip) {   // delta: output pixel of the layer that reaches this input pixel through tap (r, s)
              cw = tm.pw0 + (p.g.roff_w + p.g.pad - sft) / p.g.stride;
              ch = tm.ph0 + (p.g.roff_h + p.g.pad - r) / p.g.stride;
            } else {          // forward: first input pixel of the box (the map steps `stride` pixels per element)
              cw = tm.pw0 * p.g.stride + sft - p.g.pad;
              ch = tm.ph0 * p.g.stride + r - p.g.pad;
            }
            tma_load_4d_addr(sa, &tmA, fb, c_chunk * 64, cw, ch, tm.pn0);
            if (B_MN) {   // delta: B[k = (tap, co)][n = ci]: rows co, columns tap*pitch + ci
#pragma unroll
              for (int c = 0; c < BN / 64; ++c)
                tma_load_2d_addr(sb + c * 8192, &tmB, fb, wtap * p.g.tap_pitch + tm.n0 + c * 64, c_chunk * 64);
            } else {      // forward: B[n = co][k = (tap, ci)]
              tma_load_2d_addr(sb, &tmB, fb, wtap * p.g.tap_pitch + c_chunk * 64, tm.n0);
            }
            if (++c_chunk == p.g.chunks_per_tap) { c_chunk = 0; ++c_tap; }
          } else {
            // G: A = delta (64 pixels x 128 output channels), B = activations shifted by the tap
#pragma unroll
            for (int c = 0; c < GEMM_BM / 64; ++c) tma_load_4d_addr(sa + c * 8192, &tmA, fb, tm.m0 + c * 64, bw0, bh0, bn0);
#pragma unroll
            for (int c = 0; c < BN / 64; ++c)
              tma_load_4d_addr(sb + c * 8192, &tmB, fb, tc.col0 + c * 64, bw0 * p.g.stride + dw, bh0 * p.g.stride + dh, bn0);
            bw0 += 1 << p.g.lw;
            if (bw0 >= p.g.W) {
              bw0 = 0;
              bh0 += 1 << p.g.lh;
              if (bh0 >= p.g.H) { bh0 = 0; bn0 += GEMM_BK >> (p.g.lw + p.g.lh); }
            }
          }
          ++issued;
          if (++s == uint32_t(S)) { s = 0; ph ^= 1u; }
        }
        if constexpr (kUpdTmaOk) {
          if (upd_tma && ok) {
            const uint32_t bytes = p.mW != nullptr ? 2u * UPD_CHUNK_BYTES : uint32_t(UPD_CHUNK_BYTES);
            for (int c = 0; c < kChunks; ++c) {
              ok = mbar_wait_addr(empty0 + 8u * s, ph ^ 1u, p.wait_limit);
              if (!ok) break;
              const uint32_t sa = smem0 + s * uint32_t(SM::STAGE_BYTES);
              const uint32_t fb = full0 + 8u * s;
              mbar_arrive_expect_tx_addr(fb, bytes);
              tma_load_2d_addr(sa, &um.W, fb, tm.n0 + c * 32, tm.m0);
              if (p.mW != nullptr) tma_load_2d_addr(sa + UPD_CHUNK_BYTES, &um.M, fb, tm.n0 + c * 32, tm.m0);
              ++issued;
              if (++s == uint32_t(S)) { s = 0; ph ^= 1u; }
            }
          }
        }
      }
      if (!ok) {
        atomicExch(p.status, 1);
        // let copies already in flight land before the CTA's shared memory is released
        for (long long i = (issued > S ? issued - S : 0); i < issued; ++i) mbar_wait(&full_bar[i % S], uint32_t(i / S) & 1u, p.wait_limit);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(GEMM_BM, BN, A_MN, B_MN);
      // descriptors of stage 0, k-slice 0; other stages / slices only move the 14-bit start
      // address field (units of 16 bytes), which cannot carry out of the low word
      const uint64_t dA = A_MN ? make_smem_desc(smem_u32(smem), 8192, 1024) : make_smem_desc(smem_u32(smem), 16, 1024);
      const uint64_t dB = B_MN ? make_smem_desc(smem_u32(smem) + GEMM_A_BYTES, 8192, 1024)
                               : make_smem_desc(smem_u32(smem) + GEMM_A_BYTES, 16, 1024);
      const uint32_t dA_hi = uint32_t(dA >> 32), dB_hi = uint32_t(dB >> 32);
      constexpr uint32_t stepA = (A_MN ? 2048 : 32) >> 4, stepB = (B_MN ? 2048 : 32) >> 4;
      const uint32_t full0 = smem_u32(full_bar), empty0 = smem_u32(empty_bar);
      const uint32_t accf0 = smem_u32(accf_bar), acce0 = smem_u32(acce_bar);
      uint32_t s = 0, ph = 0;
      uint32_t dA_lo = uint32_t(dA), dB_lo = uint32_t(dB);
      bool ok = true;
      uint32_t it = 0;     // tiles done by this CTA
      for (int t = blockIdx.x; t < total_work && ok; t += (PERSIST ? int(gridDim.x) : total_work), ++it) {
        const TileCtx tc = decode_tile<BN>(p, t, tiles_m, tiles_n);
        const uint32_t buf = PERSIST ? (it & 1u) : 0u;
        if (PERSIST) {
          // the epilogue must have drained this accumulator buffer (tile it - 2)
          ok = mbar_wait_addr(acce0 + 8u * buf, ((it >> 1) & 1u) ^ 1u, p.wait_limit);
          if (!ok) break;
          tc_fence_after();
        }
        const uint32_t tacc = tmem_base + buf * uint32_t(BN);
        uint32_t acc = 0;
        for (int kb = 0; kb < tc.num_kb; ++kb) {
          ok = mbar_wait_addr(full0 + 8u * s, ph, p.wait_limit);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int j = 0; j < GEMM_BK / 16; ++j) {
            umma_f16_lohi(tacc, dA_lo + j * stepA, dA_hi, dB_lo + j * stepB, dB_hi, idesc, acc);
            acc = 1;
          }
          umma_commit_addr(empty0 + 8u * s);   // frees the stage once these MMAs have read it
          dA_lo += uint32_t(SM::STAGE_BYTES >> 4);
          dB_lo += uint32_t(SM::STAGE_BYTES >> 4);
          if (++s == uint32_t(S)) {
            s = 0;
            ph ^= 1u;
            dA_lo = uint32_t(dA);
            dB_lo = uint32_t(dB);
          }
        }
        umma_commit_addr(accf0 + 8u * buf);    // accumulator complete (also releases the epilogue on error)
        if constexpr (kUpdTmaOk) {
          if (upd_tma) {
            // The tile's chunk fills pass through the ring without this warp.  A CTA that goes on
            // to another tile still has to SEE each of them complete: a parity wait only tells
            // adjacent phases apart, and a stage may not run two phases ahead of a waiter.
            for (int c = 0; c < kChunks; ++c) {
              if (PERSIST) {
                ok = mbar_wait_addr(full0 + 8u * s, ph, p.wait_limit);
                if (!ok) break;
              }
              dA_lo += uint32_t(SM::STAGE_BYTES >> 4);
              dB_lo += uint32_t(SM::STAGE_BYTES >> 4);
              if (++s == uint32_t(S)) {
                s = 0;
                ph ^= 1u;
                dA_lo = uint32_t(dA);
                dB_lo = uint32_t(dB);
              }
            }
          }
        }
      }
      if (!ok) atomicExch(p.status, 2);
    }
  } else {
    // ------------------------------------------------------------ epilogue
    // tcgen05.ld hands each lane one accumulator ROW (32 consecutive columns).  Storing from
    // that layout would touch 32 rows per instruction, so every 32 x 32 chunk is first
    // transposed through a padded per-warp shared-memory tile; afterwards a lane owns 4
    // consecutive columns of one row and a warp instruction covers 4 rows x 128 contiguous
    // bytes (fp32) -- fully used sectors for every load and store of the epilogue.
    const int q = warp & 3;           // tensor-memory lane quarter this warp may read
    float* tile = epi_tile + q * (32 * EPI_PITCH);
    const int sub_row = lane >> 3;        // 0..3
    const int sub_col = (lane & 7) * 4;   // 0,4,..,28
    constexpr bool split = SPLITK;
    constexpr bool upd = (MODE == EPI_WGRAD_UPDATE);
    const uint32_t accf0 = smem_u32(accf_bar), acce0 = smem_u32(acce_bar);
    bool ok = true;
    uint32_t it = 0;
    // TMA update path: position in the stage ring, and the store whose source has not been released yet
    uint32_t us = 0, uph = 0, pending_stage = 0;
    bool pending = false, good = true;
    for (int t = blockIdx.x; t < total_work && ok; t += (PERSIST ? int(gridDim.x) : total_work), ++it) {
      const TileCtx tc = decode_tile<BN>(p, t, tiles_m, tiles_n);
      const TileMap& tm = tc.tm;
      const uint32_t buf = PERSIST ? (it & 1u) : 0u;
      const uint32_t tacc = tmem_base + buf * uint32_t(BN);
      const int row0 = tm.m0 + q * 32;
      if constexpr (kUpdTmaOk) {
        if (upd_tma) {
          // Every one of the 128 epilogue threads runs the same number of named barriers whatever
          // happens: after a wait that ran out, the remaining chunks only keep the barrier count.
          const uint32_t smem0 = smem_u32(smem), full0 = smem_u32(full_bar), empty0 = smem_u32(empty_bar);
          const uint32_t ringbuf = full0 + 1024u;
          const int trow = q * 32 + lane;            // row of the tile this lane owns (tensor-memory lane)
          if (p.bdelta != nullptr && tm.n0 == 0 && tm.m0 + trow < p.M) {
            // Bias of output feature m = column sum of delta over the batch, then Eq. 6 -- while
            // the tile's main loop runs.  Same order of additions as the stand-alone update
            // kernel (four interleaved partial sums, combined in order), so both give the same bits.
            const int m = tm.m0 + trow;
            float part[4] = {0.f, 0.f, 0.f, 0.f};
            const __nv_bfloat16* src = p.bdelta + m;
            int r = 0;
#pragma unroll 4
            for (; r + 4 <= p.brows; r += 4) {
#pragma unroll
              for (int i = 0; i < 4; ++i) part[i] += __bfloat162float(src[size_t(r + i) * p.bld]);
            }
            for (int i = 0; r + i < p.brows; ++i) part[i] += __bfloat162float(src[size_t(r + i) * p.bld]);
            float g = 0.f;
#pragma unroll
            for (int i = 0; i < 4; ++i) g += part[i];
            p.bdb[m] = g;
            float mm = g;
            if (p.bmb != nullptr) {
              mm = p.mu * p.bmb[m] + g;
              p.bmb[m] = mm;
            }
            const float b = p.bb[m] - p.lr * mm;
            p.bb[m] = b;
            p.bbring[m] = b;
          }
          if (good) {
            good = mbar_wait_addr(accf0 + 8u * buf, (it >> 1) & 1u, p.wait_limit);
            good = __all_sync(0xffffffffu, good);
            if (!good && lane == 0) atomicExch(p.status, 3);
          }
          tc_fence_after();
          for (int kb = 0; kb < tc.num_kb; ++kb)       // the operand fills of this tile
            if (++us == uint32_t(S)) { us = 0; uph ^= 1u; }
#pragma unroll 1
          for (int c = 0; c < kChunks; ++c) {
            const uint32_t sW = smem0 + us * uint32_t(SM::STAGE_BYTES);
            const uint32_t sM = sW + UPD_CHUNK_BYTES;
            if (good) {
              good = mbar_wait_addr(full0 + 8u * us, uph, p.wait_limit);
              good = __all_sync(0xffffffffu, good);
              if (!good && lane == 0) atomicExch(p.status, 4);
            }
            uint32_t packed[16];
            if (good) {
              uint32_t r[32];
              if (tc.num_kb > 0) {
                tmem_ld_32x32(tacc + (uint32_t(q * 32) << 16) + uint32_t(c * 32), r);
                tmem_ld_wait();
              } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) r[j] = 0u;
              }
              if (PERSIST && c == kChunks - 1) {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&acce_bar[buf]);
              }
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
            // the bf16 staging tile is free once the previous chunk's stores have read it; the
            // same wait releases that chunk's stage to the producer
            if (threadIdx.x == 64 && pending) {
              tma_store_wait_read0();
              mbar_arrive_addr(empty0 + 8u * pending_stage);
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
            if (threadIdx.x == 64) {
              if (good) {
                const int n = tm.n0 + c * 32;
                tma_store_2d_addr(&um.W, sW, n, tm.m0);
                if (p.mW != nullptr) tma_store_2d_addr(&um.M, sM, n, tm.m0);
                tma_store_2d_addr(&um.R, ringbuf, n, tm.m0);
                tma_store_commit();
                pending = true;
                pending_stage = us;
                if (PERSIST && c == kChunks - 1) {
                  // A tile's last stage is released before the next tile is touched: the next
                  // accumulator can only complete if the producer gets this stage back, so
                  // deferring the release to the next tile's first chunk would be a cycle.
                  tma_store_wait_read0();
                  mbar_arrive_addr(empty0 + 8u * us);
                  pending = false;
                }
              } else {
                mbar_arrive_addr(empty0 + 8u * us);   // keep the producer's bounded waits short
              }
            }
            if (++us == uint32_t(S)) { us = 0; uph ^= 1u; }
          }
          continue;
        }
      }
      WmRegs cur;
      if constexpr (upd && !split && !UTMA) {
        // Pull this warp's 32 rows of the master (and momentum) tile into L2 while the main loop
        // runs: the register prefetch below only reaches one chunk ahead, and an L2 hit costs a
        // fraction of an HBM round trip.
        constexpr int SEGS = BN * 4 / 128;               // 128-byte lines per tile row
        for (int i = lane; i < 32 * SEGS; i += 32) {
          const int row = row0 + i / SEGS, col = tm.n0 + (i % SEGS) * 32;
          if (row < p.M && col < tm.nlim) {
            const size_t off = size_t(row) * p.ld_out + col;
            asm volatile("prefetch.global.L2 [%0];" ::"l"(p.W + off));
            if (p.mW != nullptr) asm volatile("prefetch.global.L2 [%0];" ::"l"(p.mW + off));
          }
        }
        load_wm(p, row0, tm.n0 + sub_col, tm.nlim, sub_row, cur);   // in flight while the main loop runs
      }
      ok = mbar_wait_addr(accf0 + 8u * buf, (it >> 1) & 1u, p.wait_limit);
      ok = __all_sync(0xffffffffu, ok);      // warp-uniform: tcgen05.ld below is warp-collective
      if (!ok) {
        if (lane == 0) atomicExch(p.status, 3);
        break;
      }
      tc_fence_after();
      float* part = split ? p.partial + (size_t(tc.tile_id) * p.splits + tc.z) * (size_t(GEMM_BM) * BN) : nullptr;
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t r[32];
        __syncwarp();
        if (tc.num_kb > 0) {
          tmem_ld_32x32(tacc + (uint32_t(q * 32) << 16) + uint32_t(c * 32), r);
          tmem_ld_wait();
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j) r[j] = 0u;     // a split without k-blocks contributes zero
        }
        if (PERSIST && c == BN / 32 - 1) {
          // last read of this accumulator buffer: hand it back to the MMA issuer
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&acce_bar[buf]);
        }
#pragma unroll
        for (int g = 0; g < 8; ++g)
          *reinterpret_cast<uint4*>(tile + lane * EPI_PITCH + g * 4) = make_uint4(r[4 * g], r[4 * g + 1], r[4 * g + 2], r[4 * g + 3]);
        __syncwarp();
        const int n = tm.n0 + c * 32 + sub_col;
        if constexpr (split) {
#pragma unroll
          for (int i8 = 0; i8 < 8; ++i8) {
            const int rr = i8 * 4 + sub_row;
            const float4 acc = *reinterpret_cast<const float4*>(tile + rr * EPI_PITCH + sub_col);
            __stcg(reinterpret_cast<float4*>(part + size_t(q * 32 + rr) * BN + c * 32 + sub_col), acc);
          }
        } else if constexpr (upd && !UTMA) {
          WmRegs nxt;
          if (c + 1 < BN / 32) load_wm(p, row0, n + 32, tm.nlim, sub_row, nxt);
          apply_update(p, row0, n, tm.nlim, sub_row, tile, sub_col, cur);
          cur = nxt;
        } else {
          epilogue_rows8<MODE>(p, tm, tile, q, sub_row, sub_col, n);
        }
      }
      if constexpr (split) {
        // all four epilogue warps have written their part of the partial tile: publish it, and
        // let the last CTA of this tile reduce the partials in split order
        volatile uint32_t* is_last = tmem_slot + 1;
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (threadIdx.x == 64) {
          __threadfence();
          const unsigned prev = atomicAdd(p.tile_counter + tc.tile_id, 1u);
          const bool last = (prev == unsigned(p.splits) - 1u);
          if (last) p.tile_counter[tc.tile_id] = 0u;          // ready for the next launch
          *is_last = last ? 1u : 0u;
          __threadfence();
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (*is_last != 0u) {
          const float* base = p.partial + size_t(tc.tile_id) * p.splits * (size_t(GEMM_BM) * BN);
          const size_t zstride = size_t(GEMM_BM) * BN;
#pragma unroll 1
          for (int c = 0; c < BN / 32; ++c) {
            const int n = tm.n0 + c * 32 + sub_col;
            // eight independent rows per lane: their loads are issued together for every split,
            // the additions keep split order
            float4 acc[8];
#pragma unroll
            for (int i8 = 0; i8 < 8; ++i8)
              acc[i8] = __ldcg(reinterpret_cast<const float4*>(base + size_t(q * 32 + i8 * 4 + sub_row) * BN + c * 32 + sub_col));
            for (int z = 1; z < p.splits; ++z) {
              float4 tt[8];
#pragma unroll
              for (int i8 = 0; i8 < 8; ++i8)
                tt[i8] = __ldcg(reinterpret_cast<const float4*>(base + z * zstride + size_t(q * 32 + i8 * 4 + sub_row) * BN + c * 32 + sub_col));
#pragma unroll
              for (int i8 = 0; i8 < 8; ++i8) {
                acc[i8].x += tt[i8].x; acc[i8].y += tt[i8].y; acc[i8].z += tt[i8].z; acc[i8].w += tt[i8].w;
              }
            }
#pragma unroll
            for (int i8 = 0; i8 < 8; ++i8) {
              const int row = tile_row(p, tm, q * 32 + i8 * 4 + sub_row);
              if (row >= 0) epilogue_store4<MODE>(p, row, n, tm.nlim, acc[i8]);
            }
          }
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");     // is_last is rewritten by the next tile
      }
    }
    if constexpr (kUpdTmaOk) {
      if (pending) {                       // (thread 64 only) shared memory must outlive the last stores' reads
        tma_store_wait_read0();
        mbar_arrive_addr(smem_u32(empty_bar) + 8u * pending_stage);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, PERSIST ? 2 * BN : BN);
    if (lane == 0) tmem_note_freed(PERSIST ? TK_GEMM_PERSISTENT : TK_GEMM, PERSIST ? 2 * BN : BN);
  }
}

}  // namespace lp
