// Internal declarations shared by the host-side translation units.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <algorithm>
#include <string>
#include <vector>

#include "../../include/layerpipe.h"

namespace lp {

// ---- lp_api.cu --------------------------------------------------------------
// Error text of calls that have no handle: what lp_last_error(NULL) returns on this thread.
void set_global_error(const std::string& msg);

// ---- gemm.cu ---------------------------------------------------------------
// Encode a 2-D bf16 tensor map (128-byte swizzle, zero fill out of bounds).
// inner/outer are the logical extents in elements, pitch_elems the row pitch.
int make_tmap_bf16_2d(CUtensorMap* out, const void* base, uint64_t inner, uint64_t outer,
                      uint64_t pitch_elems, uint32_t box_inner, uint32_t box_outer, std::string* err);

int make_tmap_bf16_nhwc(CUtensorMap* out, const void* base, uint64_t C, uint64_t W, uint64_t H, uint64_t N,
                        uint64_t pitch_c, uint32_t bw, uint32_t bh, uint32_t bn, std::string* err, uint32_t step = 1);

// fp32 (elem_bytes 4) or bf16 (2) row-major tensor moved in boxes of 32 columns x box_outer rows
// (the streamed tiles of the fused update).
int make_tmap_rows32(CUtensorMap* out, const void* base, int elem_bytes, uint64_t inner, uint64_t outer,
                     uint64_t pitch_elems, uint32_t box_outer, std::string* err);

struct GemmArgs;
struct UpdMaps;
constexpr int GEMM_BN_PAIR = 512;   // tile code: 256 x 256 tile computed by a pair of CTAs (cta_group::2)
constexpr int GEMM_BN_PAIR224 = 448;   // tile code: 256 x 224 tile on a pair of CTAs (forward / delta only)
inline bool gemm_is_pair(int bn) { return bn == GEMM_BN_PAIR || bn == GEMM_BN_PAIR224; }
inline int gemm_tile_cols(int bn) { return gemm_is_pair(bn) ? bn / 2 : bn; }   // output columns of one tile
// which: 0 forward (A,B K-major), 1 delta (B MN-major), 2 G (A,B MN-major).
// Tile width BN is chosen from N and the box sizes of tmA/tmB must match it
// (see gemm_box_dims).
int gemm_pick_bn(int which, int M, int N, int K, bool allow_pair = true);
void gemm_box_dims(int which, int bn, uint32_t boxA[2], uint32_t boxB[2]);
// um (EPI_WGRAD_UPDATE only): tensor maps of the master, momentum and destination ring slot; when
// given, and the launch qualifies, the update's tiles are streamed by TMA.
cudaError_t gemm_launch(int which, int bn, const CUtensorMap& tmA, const CUtensorMap& tmB,
                        const GemmArgs& args, cudaStream_t stream, const UpdMaps* um = nullptr);
// 3x3 convolution forward (which = 0) / delta (which = 1) with at most 64 channels on both sides:
// tmA = NHWC tensor map with a 64 x 16 x 18 x 1 box, tmB = the layer's weight map (64 x 64 boxes);
// args.g describes 8 x 16 pixel tiles (lw = 3, lh = 4).  tmO (forward only; any valid map otherwise): the
// NHWC output with a 64 x 8 x 16 x 1 box, written by TMA stores.  With plain geometry (which = 0 only) the
// call is a forward GEMM with K <= 64 and N <= 64: tmA and tmO are 2-D maps with 64 x 128 boxes.
cudaError_t conv_halo_launch(int which, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmO,
                             const GemmArgs& args, cudaStream_t stream);
struct ConvGeom;
struct HaloGUpdate;
// G (+ fused update) of a halo-tile layer: tmX = the activations with the 64 x 10 x 18 x 1 halo box,
// tmD = delta with a 64 x 8 x 16 x 1 box; partial: conv_halo_g_max_ctas() x 5 x 128 x 64 floats.
int conv_halo_g_max_ctas();
cudaError_t gemm_configure();   // opt in to large dynamic shared memory; call once per process
void gemm_set_tuning(int bn, int stages, int splits);   // 0 = automatic
int gemm_pick_splits(int M, int N, int K, int bn);

// ---- planner.cpp ------------------------------------------------------------
struct PlanResult {
  std::vector<int> stage, delay;
  std::vector<int> piece_stage;          // [2*L]
  std::vector<long long> piece_amount;   // [2*L]
  int used = 0;
  long long Tp = 0;
  int rounds = 0;
};
int plan_layers(const lp_layer* layers, int L, int batch, int Np, PlanResult* out);
int layer_macs(const lp_layer& y, int batch, long long* macs);   // the planner's cost of one contraction of the layer

// ---- elementwise.cu ---------------------------------------------------------
cudaError_t launch_cast_stash(const void* batch, int input_is_bf16, const int* labels, __nv_bfloat16* x0,
                              int* labels_copy, int rows, int B, int n_in, int ld, cudaStream_t stream);
cudaError_t launch_cast_patch3x3(const void* batch, int input_is_bf16, const int* labels, __nv_bfloat16* x0,
                                 int* labels_copy, int B, int H, int W, int C, int ld, cudaStream_t stream);
// The same for any filter, stride and padding (R*S*C <= 128): one row per OUTPUT pixel, column (r*S + s)*C + ch.
cudaError_t launch_cast_patch_general(const void* batch, int input_is_bf16, const int* labels, __nv_bfloat16* x0,
                                      int* labels_copy, int B, int H, int W, int C, int R, int S, int stride, int pad,
                                      int Ho, int Wo, int ld, cudaStream_t stream);
// diagnosis: the per-SM tensor-memory table (160 x 16 ints of device memory, zeroed) that the kernels keep, or null
cudaError_t gemm_set_tmem_table(int* table);
// one thread writes `value` to *flag (mapped host memory): the progress mark after a task
cudaError_t launch_trace_mark(unsigned* flag, unsigned value, cudaStream_t stream);
cudaError_t launch_softmax_xent(const float* zL, int ldz, const int* labels, __nv_bfloat16* delta, int ldd,
                                float* row_loss, unsigned* ticket, float* loss_out, int B, int C,
                                int* status, cudaStream_t stream);
// Value of a device status word that does not come from a bounded wait (those are 1..23).
constexpr int LP_STATUS_BAD_LABEL = 64;   // a label outside [0, classes) reached the loss kernel
struct UpdateArgs {
  const float* dW;      // [out][ldw] fp32 (pad lanes zero)
  float* W;             // master [out][ldw]
  float* mW;            // momentum or null
  __nv_bfloat16* ring;  // bf16 slot that receives RN(W)
  long long n_elems;    // out * ldw (multiple of 8)
  const __nv_bfloat16* delta;  // [rows][ldd]: bias gradient = column sums (null: no bias)
  int rows, ldd, n_out;
  const float* col_partial;    // if set: [chunks][n_out] partial column sums to add instead of delta
  int n_chunks;
  float* b;             // master bias
  float* mb;            // bias momentum or null
  float* db;            // bias gradient out
  float* bring;         // fp32 bias slot that receives b
  float lr, mu;
};
cudaError_t launch_sgd_update(const UpdateArgs& a, cudaStream_t stream);
// 2x2 stride-2 max pool of an NHWC bf16 tensor (C a multiple of 8); idx = position of the first
// maximum in (dh, dw) row-major order.
cudaError_t launch_maxpool2(const __nv_bfloat16* a, __nv_bfloat16* pooled, unsigned char* idx, int B, int H, int W,
                            int C, cudaStream_t stream);
// Column sums of a [rows][ld] bf16 matrix in two deterministic passes: partial[chunk][col] over
// chunks of colsum_chunk_rows(rows) rows, then (inside launch_sgd_update) the chunk sums on four
// interleaved thread rows.  One pass (a serial loop over rows / 4 per thread) only up to 512 rows.
inline int colsum_chunk_rows(int rows) { return rows <= 131072 ? 256 : 2048; }
inline int colsum_chunks(int rows) { return rows > 512 ? (rows + colsum_chunk_rows(rows) - 1) / colsum_chunk_rows(rows) : 0; }
cudaError_t launch_colsum_partial(const __nv_bfloat16* x, int rows, int ld, int n_cols, float* partial,
                                  cudaStream_t stream);
cudaError_t launch_round_to_bf16(const float* src, __nv_bfloat16* dst, long long n_elems, cudaStream_t stream);

}  // namespace lp
