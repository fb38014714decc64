// Host side of the tcgen05 GEMM: tensor-map encoding, tile selection, launch, and the
// stand-alone lp_gemm_bf16 entry point.
#include "gemm2q.cuh"
#include "conv_halo.cuh"

#include <algorithm>
#include <atomic>
#include <cstdlib>
#include <mutex>

#include "common.h"

namespace lp {

// ---------------------------------------------------------------------------
// cuTensorMapEncodeTiled is a driver API; fetch it through the runtime so the library has
// no link-time dependency on libcuda.
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn(std::string* err) {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  static std::string first_err;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q);
    if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || p == nullptr) {
      first_err = std::string("cuTensorMapEncodeTiled unavailable: ") + cudaGetErrorString(e);
    } else {
      fn = reinterpret_cast<EncodeTiledFn>(p);
    }
  });
  if (!fn && err) *err = first_err;
  return fn;
}

int make_tmap_bf16_2d(CUtensorMap* out, const void* base, uint64_t inner, uint64_t outer, uint64_t pitch_elems,
                      uint32_t box_inner, uint32_t box_outer, std::string* err) {
  EncodeTiledFn fn = get_encode_fn(err);
  if (!fn) return LP_ERR_CUDA;
  if ((reinterpret_cast<uintptr_t>(base) & 15) || (pitch_elems & 7) || box_inner != 64 || box_outer > 256) {
    if (err) *err = "tensor map: base must be 16-byte aligned, pitch a multiple of 8 elements, box <= 256";
    return LP_ERR_INVALID_ARG;
  }
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {pitch_elems * 2};
  cuuint32_t box[2] = {box_inner, box_outer};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    if (err) *err = "cuTensorMapEncodeTiled failed with CUresult " + std::to_string(int(r));
    return LP_ERR_CUDA;
  }
  return LP_OK;
}

// Row-major 2-D tensor of 4-byte (fp32) or 2-byte (bf16) elements moved in boxes of 32 columns:
// 128-byte rows with the 128-byte swizzle, or 64-byte rows with the 64-byte swizzle.
int make_tmap_rows32(CUtensorMap* out, const void* base, int elem_bytes, uint64_t inner, uint64_t outer,
                     uint64_t pitch_elems, uint32_t box_outer, std::string* err) {
  EncodeTiledFn fn = get_encode_fn(err);
  if (!fn) return LP_ERR_CUDA;
  if ((reinterpret_cast<uintptr_t>(base) & 15) || ((pitch_elems * elem_bytes) & 15) || box_outer > 256 ||
      (elem_bytes != 4 && elem_bytes != 2)) {
    if (err) *err = "tensor map: base and pitch must be 16-byte aligned, box <= 256";
    return LP_ERR_INVALID_ARG;
  }
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {pitch_elems * elem_bytes};
  cuuint32_t box[2] = {32, box_outer};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(out, elem_bytes == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                  const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  elem_bytes == 4 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    if (err) *err = "cuTensorMapEncodeTiled (update tile) failed with CUresult " + std::to_string(int(r));
    return LP_ERR_CUDA;
  }
  return LP_OK;
}

// NHWC bf16 tensor [N][H][W][C] with channel pitch `pitch_c` (multiple of 8): dimensions
// (C, W, H, N), box (64 channels, bw, bh, bn pixels).  Coordinates outside the tensor read zero.
int make_tmap_bf16_nhwc(CUtensorMap* out, const void* base, uint64_t C, uint64_t W, uint64_t H, uint64_t N,
                        uint64_t pitch_c, uint32_t bw, uint32_t bh, uint32_t bn, std::string* err, uint32_t step) {
  EncodeTiledFn fn = get_encode_fn(err);
  if (!fn) return LP_ERR_CUDA;
  if ((reinterpret_cast<uintptr_t>(base) & 15) || (pitch_c & 7) || step < 1 || bw * step > 256 || bh * step > 256 || bn > 256) {
    if (err) *err = "tensor map: base must be 16-byte aligned, channel pitch a multiple of 8, box <= 256";
    return LP_ERR_INVALID_ARG;
  }
  // step > 1: the box takes every step-th pixel in w and h (a strided convolution's input seen from a
  // box of its output pixels): the traversed extent is bw * step, of which ceil(. / step) = bw are loaded
  cuuint64_t dims[4] = {C, W, H, N};
  cuuint64_t strides[3] = {pitch_c * 2, W * pitch_c * 2, H * W * pitch_c * 2};
  cuuint32_t box[4] = {64, bw * step, bh * step, bn};
  cuuint32_t estr[4] = {1, step, step, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    if (err) *err = "cuTensorMapEncodeTiled (4-D) failed with CUresult " + std::to_string(int(r));
    return LP_ERR_CUDA;
  }
  return LP_OK;
}

// ---------------------------------------------------------------------------
static int g_force_bn = 0;
static int g_force_stages = 0;
static int g_force_splits = 0;
static int g_l2_ahead = 16;   // measured 0 / 8 / 16 / 32 / 64 k-blocks ahead: 47.0 / 46.2 / 45.2 / 47.0 / 50.8 us (256 x 4096 x 4096)
static int g_force_persistent = -1;   // -1 automatic, 0 one tile per CTA, 1 persistent CTAs
void gemm_set_tuning(int bn, int stages, int splits) {
  g_force_bn = bn;
  g_force_stages = stages;
  g_force_splits = splits >= 0 ? (splits & 0xFF) : 0;
  // bits 8-9 of the third tuning knob force the tile loop: 1 = one tile per CTA, 2 = persistent
  g_force_persistent = splits >= 0 ? ((splits >> 8) & 3) - 1 : -1;
  if (g_force_persistent > 1) g_force_persistent = -1;
}

static int sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1)
      n = 148;
  }
  return n;
}

// Split-K factor.  Measured on B200 (M = 256, N = K = 4096): the split main loop is shorter
// but writing and re-reading the fp32 partial tiles costs more than it saves (25 us unsplit,
// 28 / 35 / 52 us at 2 / 4 / 8 splits), and under the stage scheduler other kernels fill the
// idle SMs anyway.  So the automatic choice is "off" for such shapes; the path is covered by the
// tests through lp_set_tuning.
int gemm_pick_splits(int M, int N, int K, int bn) {
  const int num_kb = (K + GEMM_BK - 1) / GEMM_BK;
  // The exception: a handful of tiles with a very long contraction (64 x 4096 x 25088: 32 tiles of
  // 392 k-blocks, one CTA streaming 6.4 MB of weights each): 145 us unsplit, 95 / 74 / 89 us at
  // 2 / 4 / 8 splits.
  const long long tiles = (long long)((M + GEMM_BM - 1) / GEMM_BM) * ((N + bn - 1) / bn);
  // Fewer tiles with longer contractions take more splits: about one CTA per SM, never fewer than 64 k-blocks per
  // split (a single 10-column tile over 100352 inputs, the classifier behind an unpooled 28 x 28 x 128 image: 24 splits).
  const int automatic = (tiles <= 48 && num_kb >= 256) ? int(std::max<long long>(1, std::min<long long>(std::min<long long>(148 / tiles, num_kb / 64), 64))) : 1;
  int s = g_force_splits > 0 ? g_force_splits : automatic;
  s = std::max(1, std::min(s, num_kb));
  const int per = (num_kb + s - 1) / s;
  return (num_kb + per - 1) / per;      // no empty split
}

int gemm_pick_bn(int which, int M, int N, int K, bool allow_pair) {
  if (g_force_bn == 64 || g_force_bn == 128 || g_force_bn == 256 || g_force_bn == GEMM_BN_PAIR) return g_force_bn;
  if (g_force_bn == GEMM_BN_PAIR224) return which == 2 ? GEMM_BN_PAIR : GEMM_BN_PAIR224;
  if (N <= 64) return 64;
  // tensor-bound shapes: 256 x 256 tiles on SM pairs (code GEMM_BN_PAIR)
  if (allow_pair && M >= 1024 && N >= 1024 && K >= 1024) {
    // forward / delta: a 224-column tile where that fills the last round of SM pairs better (cost =
    // rounds of tiles over the pairs x tile width); G keeps 256 (its update streams 64-column fills)
    if (which != 2 && g_force_bn == 0) {
      const long long pairs = std::max(1, sm_count() / 2), tm = (M + 255) / 256;
      const long long t256 = tm * ((N + 255) / 256), t224 = tm * ((N + 223) / 224);
      if (((t224 + pairs - 1) / pairs) * 224 < ((t256 + pairs - 1) / pairs) * 256) return GEMM_BN_PAIR224;
    }
    return GEMM_BN_PAIR;
  }
  (void)which;
  // 128 x 256 tiles need 96 B/clk of operands per SM instead of 128 B/clk and measured 1250 vs
  // 1130 TFLOP/s on 2048 x 8192 x 8192; they only pay off when the contraction is long and
  // there are enough tiles to fill two CTAs on every SM
  const long long tiles256 = (long long)((M + GEMM_BM - 1) / GEMM_BM) * ((N + 255) / 256);
  if (K >= 1024 && tiles256 >= 2 * 148) return 256;
  // (Narrower tiles for small batches were tried: 128 x 64 tiles make a lone forward kernel
  // 35 % faster, but re-read the activations twice as often, and with every stage's kernels
  // sharing L2 and HBM the whole step got 5 % slower.)
  return 128;
}

void gemm_box_dims(int which, int bn, uint32_t boxA[2], uint32_t boxB[2]) {
  const bool a_mn = (which == 2), b_mn = (which != 0);
  boxA[0] = 64; boxA[1] = a_mn ? 64 : GEMM_BM;
  boxB[0] = 64; boxB[1] = b_mn ? 64 : uint32_t(gemm_is_pair(bn) ? gemm_tile_cols(bn) / 2 : bn);   // a pair CTA stages half of the tile's columns
}


template <int BN, bool A_MN, bool B_MN, int MODE>
static cudaError_t launch_one(const CUtensorMap& tmA, const CUtensorMap& tmB, GemmArgs a, cudaStream_t st,
                              const UpdMaps* um) {
  if (a.splits < 1 || a.partial == nullptr) a.splits = 1;
  if (a.wait_limit <= 0) a.wait_limit = LP_WAIT_LIMIT_CYCLES;
  const int num_kb = (a.K + GEMM_BK - 1) / GEMM_BK;
  a.kb_per_split = (num_kb + a.splits - 1) / a.splits;
  const int tiles_m = (a.M + GEMM_BM - 1) / GEMM_BM;
  int tiles_n = (a.N - a.n_begin + BN - 1) / BN;
  if (a.g.kind == GEOM_PIX_K) tiles_n = a.g.n_per_tap * (a.N / a.g.tap_pitch);   // (tap, channel block)
  const long long work = (long long)tiles_m * tiles_n * a.splits;
  // BN <= 128: two CTAs per SM (2 x 2 x BN tensor-memory columns); BN = 256: one.
  // Many short tiles (convolutions over large images: thousands of tiles of 9..72 k-blocks) are
  // run by persistent CTAs -- no per-tile launch, barrier and tensor-memory set-up, epilogue
  // overlapped with the next main loop: 64 -> 64 channels at 224 x 224 forward 891 -> 546 us.
  // Few or long tiles keep one tile per CTA with a deeper pipeline: measured on the 8 x 4096
  // workload the persistent form was slower there (step 1.08 vs 0.90 ms), because the fused
  // update epilogue dominates its tiles and a second resident CTA hides more of its latency.
  const int per_sm = BN <= 128 ? 2 : 1;
  const long long slots = (long long)sm_count() * per_sm;
  a.persistent = (work >= 4 * slots && a.kb_per_split <= 96) ? 1 : 0;
  if (g_force_persistent >= 0) a.persistent = g_force_persistent;
  if (a.starve_kb > 0) a.persistent = 0;      // (the starved producer only keeps its ring position for one tile)
  // fused update streamed by TMA: plain geometry, no split-K, tiles at least 128 columns wide
  static const UpdMaps no_maps{};
  a.upd_tma = (MODE == EPI_WGRAD_UPDATE && um != nullptr && a.splits == 1 && BN >= 128 && a.g.kind == GEOM_PLAIN) ? 1 : 0;
  if (!a.upd_tma) um = &no_maps;
  const int stage_bytes = GEMM_A_BYTES + BN * GEMM_BK * 2;
  const int tail = a.upd_tma ? 1024 + UPD_RING_BYTES : 256 + (a.persistent ? EPI_TILE_BYTES : 0);
  const int avail = (per_sm == 2 ? 113 : 227) * 1024 - 1024 - 512 - tail;
  int s = g_force_stages > 0 ? g_force_stages : avail / stage_bytes;
  s = std::max(2, std::min(s, GEMM_MAX_STAGES));
  if (!a.persistent) s = std::max(2, std::min(s, std::max(a.kb_per_split + (a.upd_tma ? BN / 32 : 0), 2)));
  while (s > 2 && size_t(s) * stage_bytes > size_t(227 * 1024 - 1024 - 512 - 1024 - EPI_TILE_BYTES)) --s;
  a.num_stages = s;
  const size_t smem = GemmSmem<BN>::bytes(s, a.persistent != 0, a.upd_tma != 0);
  const int grid = int(a.persistent ? std::min<long long>(work, slots) : work);
  // single-wave launches stream their weights once: request them into L2 well ahead of the pipeline
  a.l2_ahead = (a.g.kind == GEOM_PLAIN && work <= slots && a.kb_per_split >= 8) ? g_l2_ahead : 0;
#define LP_LAUNCH(SPL, PER) \
  gemm_tcgen05_kernel<BN, A_MN, B_MN, MODE, SPL, PER><<<grid, GEMM_THREADS, smem, st>>>(tmA, tmB, *um, a, tiles_m, tiles_n, int(work))
  if constexpr (MODE == EPI_WGRAD_UPDATE && BN >= 128) {
    if (a.upd_tma) {
      if (a.persistent)
        gemm_tcgen05_kernel<BN, A_MN, B_MN, MODE, false, true, true><<<grid, GEMM_THREADS, smem, st>>>(tmA, tmB, *um, a, tiles_m, tiles_n, int(work));
      else
        gemm_tcgen05_kernel<BN, A_MN, B_MN, MODE, false, false, true><<<grid, GEMM_THREADS, smem, st>>>(tmA, tmB, *um, a, tiles_m, tiles_n, int(work));
      return cudaGetLastError();
    }
  }
  if (a.splits > 1) { if (a.persistent) LP_LAUNCH(true, true); else LP_LAUNCH(true, false); }
  else              { if (a.persistent) LP_LAUNCH(false, true); else LP_LAUNCH(false, false); }
#undef LP_LAUNCH
  return cudaGetLastError();
}

template <int BN, bool A_MN, bool B_MN, int MODE>
static cudaError_t configure_one() {
  cudaError_t e;
#define LP_ATTR(SPL, PER)                                                                                   \
  if ((e = cudaFuncSetAttribute(gemm_tcgen05_kernel<BN, A_MN, B_MN, MODE, SPL, PER>,                          \
                                cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024)) != cudaSuccess)   \
    return e;
  LP_ATTR(false, false) LP_ATTR(false, true) LP_ATTR(true, false) LP_ATTR(true, true)
#undef LP_ATTR
  if constexpr (MODE == EPI_WGRAD_UPDATE && BN >= 128) {
    if ((e = cudaFuncSetAttribute(gemm_tcgen05_kernel<BN, A_MN, B_MN, MODE, false, false, true>,
                                  cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024)) != cudaSuccess)
      return e;
    if ((e = cudaFuncSetAttribute(gemm_tcgen05_kernel<BN, A_MN, B_MN, MODE, false, true, true>,
                                  cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024)) != cudaSuccess)
      return e;
  }
  return cudaSuccess;
}

// instantiated combinations: (operand majors of the contraction) x (epilogue)
#define LP_FOR_EACH_VARIANT(X, BN)           \
  X(BN, false, false, EPI_FPROP)             \
  X(BN, false, false, EPI_STORE_F32)         \
  X(BN, false, true, EPI_DGRAD)              \
  X(BN, false, true, EPI_DGRAD_UNPOOL)       \
  X(BN, false, true, EPI_STORE_F32)          \
  X(BN, true, true, EPI_STORE_F32)           \
  X(BN, true, true, EPI_WGRAD_UPDATE)

// ---- two-CTA (SM pair) kernel ---------------------------------------------------------------
template <bool A_MN, bool B_MN, int MODE, int BN2 = GEMM2_BN>
static cudaError_t launch_pair(const CUtensorMap& tmA, const CUtensorMap& tmB, GemmArgs a, cudaStream_t st, const UpdMaps* um) {
  a.splits = 1;
  if (a.wait_limit <= 0) a.wait_limit = LP_WAIT_LIMIT_CYCLES;
  static const UpdMaps no_maps{};
  a.upd_tma = (MODE == EPI_WGRAD_UPDATE && um != nullptr && a.g.kind == GEOM_PLAIN) ? 1 : 0;
  if (!a.upd_tma) um = &no_maps;
  const int stage_bytes = 32 * 1024;
  const int num_kb = (a.K + GEMM_BK - 1) / GEMM_BK;
  int s = g_force_stages > 0 ? g_force_stages : (a.tmem_policy == TMEM_PAIR_ALONE ? 6 : 3);   // 3 x 32 KiB: two CTAs per SM; 6: alone
  s = std::max(2, std::min(std::min(s, GEMM_MAX_STAGES), std::max(num_kb + (a.upd_tma ? GEMM2_BN / 64 : 0), 2)));
  const size_t tail = 1024 + 256 + (a.upd_tma ? 1024 + UPD_RING_BYTES : 0);   // alignment slack, barriers, bf16 staging tile
  while (s > 2 && size_t(s) * stage_bytes + tail > 227 * 1024) --s;
  a.num_stages = s;
  cudaLaunchConfig_t cfg = {};
  // (convolution geometry: M is a whole number of 128-pixel boxes, and an even one -- the caller checks)
  cfg.gridDim = dim3(2 * ((a.M + 255) / 256), (a.N - a.n_begin + BN2 - 1) / BN2, 1);
  cfg.blockDim = dim3(GEMM_THREADS, 1, 1);
  cfg.dynamicSmemBytes = size_t(s) * stage_bytes + tail;
  if (a.tmem_policy == TMEM_PAIR_ALONE)      // (also when a short contraction takes fewer stages)
    cfg.dynamicSmemBytes = std::max<size_t>(cfg.dynamicSmemBytes, size_t(6) * stage_bytes + tail);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if constexpr (MODE == EPI_WGRAD_UPDATE && BN2 == GEMM2_BN) {
    if (a.upd_tma) {
      // Many short tiles (G of a wide layer contracts over the minibatch only): one persistent CTA pair
      // per SM pair, update streamed under the next tile's main loop (8192 x 8192 x 2048: 255 -> 248 us).
      const int tiles_m = (a.M + 255) / 256, tiles_n = (a.N + GEMM2_BN - 1) / GEMM2_BN;
      const int pairs = std::max(1, sm_count() / 2);
      // (with momentum the one-tile form measured faster: 337 against 371 us on 8192 x 8192 x 2048)
      const bool persistent = g_force_persistent >= 0 ? g_force_persistent == 1
                                                      : (tiles_m * tiles_n >= 2 * pairs && num_kb <= 96 && a.mW == nullptr);
      if (persistent && a.starve_kb == 0) {
        cfg.gridDim = dim3(2 * std::min(tiles_m * tiles_n, pairs), 1, 1);
        cfg.blockDim = dim3(GEMM2P_THREADS, 1, 1);
        cfg.dynamicSmemBytes = GEMM2P_SMEM_BYTES;
        // 192 KiB of shared memory divided between operand stages and update-chunk slots
        // (chunk slots are 16 KiB, 32 KiB with momentum: four operand stages leave four / two of them, three leave six / three)
        a.num_stages = g_force_stages > 0 ? std::max(2, std::min(g_force_stages, 5)) : (a.mW != nullptr ? 3 : 4);
        return cudaLaunchKernelEx(&cfg, gemm2p_g_update_kernel<0>, tmA, tmB, *um, a, tiles_m, tiles_n);
      }
      return cudaLaunchKernelEx(&cfg, gemm2_tcgen05_kernel<A_MN, B_MN, MODE, true>, tmA, tmB, *um, a);
    }
  }
  if constexpr (!A_MN && (MODE == EPI_FPROP || MODE == EPI_DGRAD || MODE == EPI_DGRAD_UNPOOL)) {
    // A pair CTA that has its SM to itself walks the tiles with two accumulators (see gemm2q.cuh)
    const int tiles_m = (a.M + 255) / 256, tiles_n = (a.N - a.n_begin + BN2 - 1) / BN2;
    const int pairs = std::max(1, sm_count() / 2);
    // also for the delta contraction of wide fully connected layers (MN-major B: 211 -> 206 us on 2048 x 8192 x 8192
    // in a burst, 252 -> 246 us in a 300-step run; the forward contraction measures the same either way)
    const bool long_delta = (MODE == EPI_DGRAD || MODE == EPI_DGRAD_UNPOOL) && a.g.kind == GEOM_PLAIN &&
                            tiles_m * tiles_n >= 2 * pairs && num_kb >= 32;
    if ((a.tmem_policy == TMEM_PAIR_ALONE || g_force_persistent == 1 || long_delta) && a.starve_kb == 0 && g_force_persistent != 0 &&
        g_force_stages == 0) {
      cfg.gridDim = dim3(2 * std::min(tiles_m * tiles_n, pairs), 1, 1);
      cfg.blockDim = dim3(GEMM2Q_THREADS, 1, 1);
      cfg.dynamicSmemBytes = GEMM2Q_SMEM_BYTES;
      a.num_stages = GEMM2Q_STAGES;
      return cudaLaunchKernelEx(&cfg, gemm2q_kernel<B_MN, MODE, BN2>, tmA, tmB, a, tiles_m, tiles_n);
    }
  }
  return cudaLaunchKernelEx(&cfg, gemm2_tcgen05_kernel<A_MN, B_MN, MODE, false, BN2>, tmA, tmB, *um, a);
}
template <bool A_MN, bool B_MN, int MODE>
static cudaError_t configure_pair() {
  cudaError_t e = cudaFuncSetAttribute(gemm2_tcgen05_kernel<A_MN, B_MN, MODE, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       227 * 1024);
  if constexpr (MODE == EPI_WGRAD_UPDATE) {
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(gemm2_tcgen05_kernel<A_MN, B_MN, MODE, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  } else if constexpr (!A_MN) {      // forward / delta also exist with 224-column tiles
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(gemm2_tcgen05_kernel<A_MN, B_MN, MODE, false, 224>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if constexpr (MODE == EPI_FPROP || MODE == EPI_DGRAD || MODE == EPI_DGRAD_UNPOOL) {
      if (e == cudaSuccess)
        e = cudaFuncSetAttribute(gemm2q_kernel<B_MN, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM2Q_SMEM_BYTES);
      if (e == cudaSuccess)
        e = cudaFuncSetAttribute(gemm2q_kernel<B_MN, MODE, 224>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM2Q_SMEM_BYTES);
    }
  }
  return e;
}
#define LP_FOR_EACH_PAIR_VARIANT(X)   \
  X(false, false, EPI_FPROP)          \
  X(false, false, EPI_STORE_F32)      \
  X(false, true, EPI_DGRAD)           \
  X(false, true, EPI_DGRAD_UNPOOL)    \
  X(false, true, EPI_STORE_F32)       \
  X(true, true, EPI_STORE_F32)        \
  X(true, true, EPI_WGRAD_UPDATE)

// ---- halo-tile convolution (3x3, at most 64 channels on both sides) ------------------------------
#define LP_FOR_EACH_HALO_VARIANT(X) \
  X(false, EPI_FPROP)               \
  X(true, EPI_DGRAD)                \
  X(true, EPI_DGRAD_UNPOOL)

cudaError_t conv_halo_launch(int which, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmO,
                             const GemmArgs& args, cudaStream_t st) {
  const bool b_mn = (which != 0);
  const int tiles = args.g.kind == GEOM_PLAIN ? (args.M + GEMM_BM - 1) / GEMM_BM
                                               : args.g.tiles_w * args.g.tiles_h * (args.M / (args.g.H * args.g.W));
  const int grid = std::min(tiles, sm_count());
#define LP_TRYH(B, M)                                                                                          \
  if (b_mn == B && args.mode == M) {                                                                           \
    conv_halo_kernel<B, M><<<grid, HALO_THREADS, HALO_SMEM_BYTES, st>>>(tmA, tmB, tmO, args, tiles);                \
    return cudaGetLastError();                                                                                 \
  }
  LP_FOR_EACH_HALO_VARIANT(LP_TRYH)
#undef LP_TRYH
  return cudaErrorInvalidValue;
}

// G of a halo-tile layer: accumulate over 8 x 16 pixel tiles, then add the CTAs' partial sums and
// apply the update (upd.W null: store G only).
cudaError_t conv_halo_g_launch(const CUtensorMap& tmX, const CUtensorMap& tmD, const ConvGeom& g, int batch, float* partial,
                               HaloGUpdate upd, int* status, cudaStream_t st) {
  const int tiles = g.tiles_w * g.tiles_h * batch;
  const int grid = std::min(tiles, sm_count());
  upd.partial = partial;
  upd.n_ctas = grid;
  for (int co0 = 0; co0 < upd.n_out; co0 += 64) {      // one pass per 64 output channels; the stream orders the reuse of `partial`
    conv_halo_g_kernel<0><<<grid, GEMM_THREADS, HALOG_SMEM_BYTES, st>>>(tmX, tmD, g, tiles, co0, partial, status);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    upd.co0 = co0;
    conv_halo_g_update_kernel<0><<<(HALOG_PART_FLOATS + 255) / 256, 256, 0, st>>>(upd);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}
int conv_halo_g_max_ctas() { return sm_count(); }

cudaError_t gemm_configure() {
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(gemm2p_g_update_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM2P_SMEM_BYTES)) != cudaSuccess)
    return e;
  if ((e = cudaFuncSetAttribute(conv_halo_g_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, HALOG_SMEM_BYTES)) != cudaSuccess)
    return e;
#define LP_CFGH(B, M)                                                                                          \
  if ((e = cudaFuncSetAttribute(conv_halo_kernel<B, M>, cudaFuncAttributeMaxDynamicSharedMemorySize,           \
                                HALO_SMEM_BYTES)) != cudaSuccess)                                              \
    return e;
  LP_FOR_EACH_HALO_VARIANT(LP_CFGH)
#undef LP_CFGH
#define LP_CFGP(A, B, M) \
  if ((e = configure_pair<A, B, M>()) != cudaSuccess) return e;
  LP_FOR_EACH_PAIR_VARIANT(LP_CFGP)
#undef LP_CFGP
#define LP_CFG(BN, A, B, M) \
  if ((e = configure_one<BN, A, B, M>()) != cudaSuccess) return e;
  LP_FOR_EACH_VARIANT(LP_CFG, 64)
  LP_FOR_EACH_VARIANT(LP_CFG, 128)
  LP_FOR_EACH_VARIANT(LP_CFG, 256)
#undef LP_CFG
  return cudaSuccess;
}

cudaError_t gemm_launch(int which, int bn, const CUtensorMap& tmA, const CUtensorMap& tmB, const GemmArgs& args,
                        cudaStream_t st, const UpdMaps* um) {
  const bool a_mn = (which == 2), b_mn = (which != 0);
  if (bn == GEMM_BN_PAIR224) {
    if (a_mn || args.g.kind != GEOM_PLAIN) return cudaErrorInvalidValue;
#define LP_TRYP224(A, B, M) \
  if (!A && b_mn == B && args.mode == M) return launch_pair<A, B, M, 224>(tmA, tmB, args, st, nullptr);
    LP_FOR_EACH_PAIR_VARIANT(LP_TRYP224)
#undef LP_TRYP224
    return cudaErrorInvalidValue;
  }
  if (bn == GEMM_BN_PAIR) {
    if (args.g.kind == GEOM_PIX_K) return cudaErrorInvalidValue;
#define LP_TRYP(A, B, M) \
  if (a_mn == A && b_mn == B && args.mode == M) return launch_pair<A, B, M>(tmA, tmB, args, st, um);
    LP_FOR_EACH_PAIR_VARIANT(LP_TRYP)
#undef LP_TRYP
    return cudaErrorInvalidValue;
  }
#define LP_TRY(BN, A, B, M) \
  if (bn == BN && a_mn == A && b_mn == B && args.mode == M) return launch_one<BN, A, B, M>(tmA, tmB, args, st, um);
  LP_FOR_EACH_VARIANT(LP_TRY, 64)
  LP_FOR_EACH_VARIANT(LP_TRY, 128)
  LP_FOR_EACH_VARIANT(LP_TRY, 256)
#undef LP_TRY
  return cudaErrorInvalidValue;
}

}  // namespace lp

namespace lp {
cudaError_t gemm_set_tmem_table(int* table) {
  return cudaMemcpyToSymbol(g_tmem_table, &table, sizeof(table));
}
}  // namespace lp

// status word for the stand-alone entry point (handles keep theirs in the workspace)
__device__ int g_gemm_status = 0;

namespace {
// Per device: the address of g_gemm_status there, and whether the kernels' shared-memory attributes
// have been set on it.  Written once per device under the mutex.
constexpr int kMaxGemmDevices = 64;
std::atomic<int*> g_gemm_status_addr[kMaxGemmDevices];
std::mutex g_gemm_setup_mutex;

int gemm_device_setup(int** status_dev) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxGemmDevices) {
    lp::set_global_error("lp_gemm_bf16: no current CUDA device");
    return LP_ERR_CUDA;
  }
  int* p = g_gemm_status_addr[dev].load(std::memory_order_acquire);
  if (p == nullptr) {
    std::lock_guard<std::mutex> lock(g_gemm_setup_mutex);
    p = g_gemm_status_addr[dev].load(std::memory_order_relaxed);
    if (p == nullptr) {
      void* q = nullptr;
      cudaError_t e = cudaGetSymbolAddress(&q, g_gemm_status);
      if (e == cudaSuccess) e = lp::gemm_configure();
      if (e != cudaSuccess || q == nullptr) {
        lp::set_global_error(std::string("lp_gemm_bf16 set-up: ") + cudaGetErrorString(e));
        return LP_ERR_CUDA;
      }
      p = static_cast<int*>(q);
      g_gemm_status_addr[dev].store(p, std::memory_order_release);
    }
  }
  *status_dev = p;
  return LP_OK;
}

int gemm_standalone(int which, int M, int N, int K, const void* A, int lda, const void* B, int ldb, float* C, int ldc,
                    void* stream, long long wait_limit, int starve_kb) {
  using namespace lp;
  if (which < 0 || which > 2 || M < 1 || N < 1 || K < 1 || !A || !B || !C) return LP_ERR_INVALID_ARG;
  if ((lda & 7) || (ldb & 7) || (ldc & 3)) return LP_ERR_INVALID_ARG;
  int* status_dev = nullptr;
  int rc = gemm_device_setup(&status_dev);
  if (rc != LP_OK) return rc;
  const int bn = gemm_pick_bn(which, M, N, K);
  uint32_t boxA[2], boxB[2];
  gemm_box_dims(which, bn, boxA, boxB);
  CUtensorMap tmA, tmB;
  std::string err;
  // A: forward/delta K-major -> rows = M, inner = K; G: stored [K][M] -> inner = M, rows = K
  if (which == 2) rc = make_tmap_bf16_2d(&tmA, A, M, K, lda, boxA[0], boxA[1], &err);
  else            rc = make_tmap_bf16_2d(&tmA, A, K, M, lda, boxA[0], boxA[1], &err);
  if (rc != LP_OK) { set_global_error(err); return rc; }
  // B: forward stored [N][K]; delta and G stored [K][N]
  if (which == 0) rc = make_tmap_bf16_2d(&tmB, B, K, N, ldb, boxB[0], boxB[1], &err);
  else            rc = make_tmap_bf16_2d(&tmB, B, N, K, ldb, boxB[0], boxB[1], &err);
  if (rc != LP_OK) { set_global_error(err); return rc; }
  GemmArgs a{};
  a.M = M; a.N = N; a.K = K;
  a.mode = EPI_STORE_F32;
  a.out = C; a.ld_out = ldc;
  a.status = status_dev;
  a.wait_limit = wait_limit;
  a.starve_kb = starve_kb;
  cudaError_t e = gemm_launch(which, bn, tmA, tmB, a, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) { set_global_error(std::string("lp_gemm_bf16 launch: ") + cudaGetErrorString(e)); return LP_ERR_CUDA; }
  return LP_OK;
}
}  // namespace

// ---------------------------------------------------------------------------
extern "C" int lp_gemm_bf16(int which, int M, int N, int K, const void* A, int lda, const void* B, int ldb,
                            float* C, int ldc, void* stream) {
  return gemm_standalone(which, M, N, K, A, lda, B, ldb, C, ldc, stream, 0, 0);
}

extern "C" int lp_gemm_status(int* detail) {
  int* status_dev = nullptr;
  int rc = gemm_device_setup(&status_dev);
  if (rc != LP_OK) return rc;
  int st = 0;
  const int zero = 0;
  if (cudaDeviceSynchronize() != cudaSuccess || cudaMemcpy(&st, status_dev, 4, cudaMemcpyDeviceToHost) != cudaSuccess ||
      cudaMemcpy(status_dev, &zero, 4, cudaMemcpyHostToDevice) != cudaSuccess) {
    lp::set_global_error("lp_gemm_status: a CUDA call failed");
    return LP_ERR_CUDA;
  }
  if (detail) *detail = st;
  if (st != 0) {
    lp::set_global_error("lp_gemm_bf16: a bounded device-side wait expired (status " + std::to_string(st) + ")");
    return LP_ERR_TIMEOUT;
  }
  return LP_OK;
}

extern "C" int lp_debug_gemm_starved(int M, int N, int K, const void* A, int lda, const void* B, int ldb, float* C,
                                     int ldc, long long limit_cycles, void* stream) {
  if (limit_cycles < 1000 || limit_cycles > 2000000000ll || K <= lp::GEMM_BK) return LP_ERR_INVALID_ARG;
  return gemm_standalone(0, M, N, K, A, lda, B, ldb, C, ldc, stream, limit_cycles, 1);
}
