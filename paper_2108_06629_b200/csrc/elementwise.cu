// HBM-bound kernels of the training step: input cast + stash, softmax cross-entropy with
// delta^L, and the fused SGD update (Eq. 6) that also refreshes the bf16 weight-ring slot.
#include <atomic>
#include <cstdio>
#include <mutex>

#include "common.h"

namespace lp {

__global__ void trace_mark_kernel(unsigned* flag, unsigned value) {
  *reinterpret_cast<volatile unsigned*>(flag) = value;
  __threadfence_system();
}
cudaError_t launch_trace_mark(unsigned* flag, unsigned value, cudaStream_t stream) {
  trace_mark_kernel<<<1, 1, 0, stream>>>(flag, value);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// a^0 = RN_bf16(batch) into the first layer's activation-stash slot; labels are copied
// into the library's label ring so that the caller may reuse its buffers.
__global__ void cast_stash_kernel(const void* __restrict__ batch, int input_is_bf16,
                                  const int* __restrict__ labels, __nv_bfloat16* __restrict__ x0,
                                  int* __restrict__ labels_copy, int rows, int B, int n_in, int ld) {
  const long long groups_per_row = ld / 8;
  const long long total = (long long)rows * groups_per_row;
  for (long long g = blockIdx.x * (long long)blockDim.x + threadIdx.x; g < total;
       g += (long long)gridDim.x * blockDim.x) {
    const int row = int(g / groups_per_row);
    const int c0 = int(g % groups_per_row) * 8;
    float v[8];
    if (input_is_bf16) {
      const __nv_bfloat16* src = reinterpret_cast<const __nv_bfloat16*>(batch) + (long long)row * n_in;
#pragma unroll
      for (int j = 0; j < 8; ++j) v[j] = (c0 + j < n_in) ? __bfloat162float(src[c0 + j]) : 0.f;
    } else {
      const float* src = reinterpret_cast<const float*>(batch) + (long long)row * n_in;
      if ((n_in & 3) == 0 && c0 + 8 <= n_in) {
        const float4 a = *reinterpret_cast<const float4*>(src + c0);
        const float4 b = *reinterpret_cast<const float4*>(src + c0 + 4);
        v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
      } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = (c0 + j < n_in) ? src[c0 + j] : 0.f;
      }
    }
    __nv_bfloat162 p0 = __floats2bfloat162_rn(v[0], v[1]);
    __nv_bfloat162 p1 = __floats2bfloat162_rn(v[2], v[3]);
    __nv_bfloat162 p2 = __floats2bfloat162_rn(v[4], v[5]);
    __nv_bfloat162 p3 = __floats2bfloat162_rn(v[6], v[7]);
    uint4 o;
    o.x = *reinterpret_cast<uint32_t*>(&p0);
    o.y = *reinterpret_cast<uint32_t*>(&p1);
    o.z = *reinterpret_cast<uint32_t*>(&p2);
    o.w = *reinterpret_cast<uint32_t*>(&p3);
    *reinterpret_cast<uint4*>(x0 + (long long)row * ld + c0) = o;
  }
  if (blockIdx.x == 0) {
    for (int i = threadIdx.x; i < B; i += blockDim.x) labels_copy[i] = labels[i];
  }
}

cudaError_t launch_cast_stash(const void* batch, int input_is_bf16, const int* labels, __nv_bfloat16* x0,
                              int* labels_copy, int rows, int B, int n_in, int ld, cudaStream_t stream) {
  const long long total = (long long)rows * (ld / 8);
  int blocks = int(std::min<long long>((total + 255) / 256, 148 * 8));
  if (blocks < 1) blocks = 1;
  cast_stash_kernel<<<blocks, 256, 0, stream>>>(batch, input_is_bf16, labels, x0, labels_copy, rows, B, n_in, ld);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// First convolution layer with very few input channels (an RGB image): a^0 is stashed as the
// matrix of 3x3 patches, one row per output pixel, column (r*3 + s)*C + ch = the input at
// (h + r - 1, w + s - 1, ch) or zero outside the image, padded with zero columns to `ld`.  The
// layer's contractions (Eq. 1 and Eq. 5 written for a convolution) then run as plain GEMMs over
// 9*C columns instead of nine taps of a 64-wide k-block that would be 95 % padding.
// One thread per output pixel; C is a template parameter so that the 9*C gathered values stay in
// registers and the column arithmetic folds at compile time.
template <int C>
__global__ void cast_patch3x3_kernel(const void* __restrict__ batch, int input_is_bf16,
                                     const int* __restrict__ labels, __nv_bfloat16* __restrict__ x0,
                                     int* __restrict__ labels_copy, int B, int H, int W) {
  constexpr int LD = (9 * C + 7) / 8 * 8;
  const int total = B * H * W;
  for (int pix = blockIdx.x * blockDim.x + threadIdx.x; pix < total; pix += gridDim.x * blockDim.x) {
    const int w = pix % W;
    const int h = (pix / W) % H;
    float v[LD];
#pragma unroll
    for (int k = 0; k < LD; ++k) v[k] = 0.f;
#pragma unroll
    for (int r = 0; r < 3; ++r) {
      const int hh = h + r - 1;
      if (hh < 0 || hh >= H) continue;
#pragma unroll
      for (int s = 0; s < 3; ++s) {
        const int ww = w + s - 1;
        if (ww < 0 || ww >= W) continue;
        const long long idx = ((long long)pix + (r - 1) * W + (s - 1)) * C;
#pragma unroll
        for (int ch = 0; ch < C; ++ch)
          v[(r * 3 + s) * C + ch] = input_is_bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(batch)[idx + ch])
                                                  : reinterpret_cast<const float*>(batch)[idx + ch];
      }
    }
    uint4* dst = reinterpret_cast<uint4*>(x0 + (long long)pix * LD);
#pragma unroll
    for (int g = 0; g < LD / 8; ++g) {
      __nv_bfloat162 p0 = __floats2bfloat162_rn(v[8 * g + 0], v[8 * g + 1]);
      __nv_bfloat162 p1 = __floats2bfloat162_rn(v[8 * g + 2], v[8 * g + 3]);
      __nv_bfloat162 p2 = __floats2bfloat162_rn(v[8 * g + 4], v[8 * g + 5]);
      __nv_bfloat162 p3 = __floats2bfloat162_rn(v[8 * g + 6], v[8 * g + 7]);
      uint4 o;
      o.x = *reinterpret_cast<uint32_t*>(&p0);
      o.y = *reinterpret_cast<uint32_t*>(&p1);
      o.z = *reinterpret_cast<uint32_t*>(&p2);
      o.w = *reinterpret_cast<uint32_t*>(&p3);
      dst[g] = o;
    }
  }
  if (blockIdx.x == 0) {
    for (int i = threadIdx.x; i < B; i += blockDim.x) labels_copy[i] = labels[i];
  }
}

cudaError_t launch_cast_patch3x3(const void* batch, int input_is_bf16, const int* labels, __nv_bfloat16* x0,
                                 int* labels_copy, int B, int H, int W, int C, int ld, cudaStream_t stream) {
  const long long total = (long long)B * H * W;
  if (C < 1 || C > 7 || ld != (9 * C + 7) / 8 * 8 || total >= (1ll << 31)) return cudaErrorInvalidValue;
  int blocks = int(std::min<long long>((total + 255) / 256, 148 * 8));
  if (blocks < 1) blocks = 1;
#define LP_PATCH_CASE(c)                                                                                        \
  case c: cast_patch3x3_kernel<c><<<blocks, 256, 0, stream>>>(batch, input_is_bf16, labels, x0, labels_copy, B, H, W); break;
  switch (C) {
    LP_PATCH_CASE(1) LP_PATCH_CASE(2) LP_PATCH_CASE(3) LP_PATCH_CASE(4) LP_PATCH_CASE(5) LP_PATCH_CASE(6) LP_PATCH_CASE(7)
  }
#undef LP_PATCH_CASE
  return cudaGetLastError();
}

// General filters / strides: thread t handles 8 consecutive columns of one patch row (one 16-byte
// store); the column's (tap, channel) and the tap's input pixel are decoded per element.
__global__ void cast_patch_general_kernel(const void* __restrict__ batch, int input_is_bf16, const int* __restrict__ labels,
                                          __nv_bfloat16* __restrict__ x0, int* __restrict__ labels_copy, int B, int H, int W,
                                          int C, int R, int S, int stride, int pad, int Ho, int Wo, int ld) {
  const int groups = ld / 8;
  const long long total = (long long)B * Ho * Wo * groups;
  const int n_cols = R * S * C;
  for (long long t = blockIdx.x * (long long)blockDim.x + threadIdx.x; t < total; t += (long long)gridDim.x * blockDim.x) {
    const int g = int(t % groups);
    const long long pix = t / groups;
    const int wo = int(pix % Wo), ho = int((pix / Wo) % Ho), b = int(pix / ((long long)Wo * Ho));
    float v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int col = g * 8 + j;
      v[j] = 0.f;
      if (col < n_cols) {
        const int tap = col / C, ch = col % C;
        const int hh = ho * stride + tap / S - pad, ww = wo * stride + tap % S - pad;
        if (hh >= 0 && hh < H && ww >= 0 && ww < W) {
          const long long idx = (((long long)b * H + hh) * W + ww) * C + ch;
          v[j] = input_is_bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(batch)[idx])
                               : reinterpret_cast<const float*>(batch)[idx];
        }
      }
    }
    __nv_bfloat162 p0 = __floats2bfloat162_rn(v[0], v[1]), p1 = __floats2bfloat162_rn(v[2], v[3]);
    __nv_bfloat162 p2 = __floats2bfloat162_rn(v[4], v[5]), p3 = __floats2bfloat162_rn(v[6], v[7]);
    uint4 o;
    o.x = *reinterpret_cast<uint32_t*>(&p0); o.y = *reinterpret_cast<uint32_t*>(&p1);
    o.z = *reinterpret_cast<uint32_t*>(&p2); o.w = *reinterpret_cast<uint32_t*>(&p3);
    *reinterpret_cast<uint4*>(x0 + pix * ld + g * 8) = o;
  }
  if (blockIdx.x == 0) {
    for (int i = threadIdx.x; i < B; i += blockDim.x) labels_copy[i] = labels[i];
  }
}

cudaError_t launch_cast_patch_general(const void* batch, int input_is_bf16, const int* labels, __nv_bfloat16* x0,
                                      int* labels_copy, int B, int H, int W, int C, int R, int S, int stride, int pad,
                                      int Ho, int Wo, int ld, cudaStream_t stream) {
  const long long total = (long long)B * Ho * Wo * (ld / 8);
  if (C < 1 || R * S * C > ld || (ld & 7) || total >= (1ll << 40)) return cudaErrorInvalidValue;
  int blocks = int(std::min<long long>((total + 255) / 256, 148 * 16));
  if (blocks < 1) blocks = 1;
  cast_patch_general_kernel<<<blocks, 256, 0, stream>>>(batch, input_is_bf16, labels, x0, labels_copy, B, H, W, C, R, S, stride,
                                                        pad, Ho, Wo, ld);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// One block per row: p = softmax(z^L), delta^L = RN((p - onehot)/B), row loss; the last
// block to finish adds the row losses in row order (deterministic mean).
__device__ __forceinline__ float block_reduce(float v, float* sh, bool is_max) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float other = __shfl_xor_sync(0xffffffffu, v, o);
    v = is_max ? fmaxf(v, other) : v + other;
  }
  __syncthreads();
  if (lane == 0) sh[w] = v;
  __syncthreads();
  const int nw = blockDim.x >> 5;
  float r = sh[0];
  for (int i = 1; i < nw; ++i) r = is_max ? fmaxf(r, sh[i]) : r + sh[i];
  return r;
}

__global__ void softmax_xent_kernel(const float* __restrict__ zL, int ldz, const int* __restrict__ labels,
                                    __nv_bfloat16* __restrict__ delta, int ldd, float* __restrict__ row_loss,
                                    unsigned* __restrict__ ticket, float* __restrict__ loss_out, int B, int C,
                                    int* __restrict__ status) {
  __shared__ float sh[32];
  __shared__ bool last;
  const int row = blockIdx.x;
  const float* z = zL + (long long)row * ldz;
  float mx = -INFINITY;
  for (int c = threadIdx.x; c < C; c += blockDim.x) mx = fmaxf(mx, z[c]);
  mx = block_reduce(mx, sh, true);
  float s = 0.f;
  for (int c = threadIdx.x; c < C; c += blockDim.x) s += expf(z[c] - mx);
  s = block_reduce(s, sh, false);
  // A label outside [0, C) comes from caller memory: it must not become an address.  Such a row
  // gets no one-hot term, its loss is NaN (so the minibatch loss is NaN) and the status word, where
  // there is one, records it.
  const int y = labels[row];
  const bool y_ok = unsigned(y) < unsigned(C);
  const float invB = 1.0f / float(B);
  const float inv_s = 1.0f / s;
  __nv_bfloat16* d = delta + (long long)row * ldd;
  const int Cpad = (C + 7) & ~7;
  for (int c = threadIdx.x; c < Cpad; c += blockDim.x) {
    float v = 0.f;
    if (c < C) v = (expf(z[c] - mx) * inv_s - (c == y ? 1.f : 0.f)) * invB;
    d[c] = __float2bfloat16_rn(v);
  }
  if (threadIdx.x == 0) {
    row_loss[row] = y_ok ? -((z[y] - mx) - logf(s)) : __int_as_float(0x7fc00000);
    if (!y_ok && status != nullptr) atomicCAS(status, 0, LP_STATUS_BAD_LABEL);
    __threadfence();
    const unsigned t = atomicAdd(ticket, 1u);
    last = (t == unsigned(B) - 1u);
  }
  __syncthreads();
  if (last) {
    // deterministic mean: thread t adds rows t, t + 256, ... in that order, then the 256 partial
    // sums are added in thread order
    __threadfence();
    float acc = 0.f;
    for (int i = threadIdx.x; i < B; i += blockDim.x) acc += __ldcg(row_loss + i);
    __shared__ float part[256];
    part[threadIdx.x] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
      float tot = 0.f;
      for (int i = 0; i < int(blockDim.x); ++i) tot += part[i];
      *loss_out = tot * invB;
      *ticket = 0u;     // ready for the next launch on this scratch
    }
  }
}

cudaError_t launch_softmax_xent(const float* zL, int ldz, const int* labels, __nv_bfloat16* delta, int ldd,
                                float* row_loss, unsigned* ticket, float* loss_out, int B, int C,
                                int* status, cudaStream_t stream) {
  softmax_xent_kernel<<<B, 256, 0, stream>>>(zL, ldz, labels, delta, ldd, row_loss, ticket, loss_out, B, C, status);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Fused update (Eq. 6, optional momentum): m <- mu m + G; W <- W - eta m; ring <- RN(W).
// 8 elements per thread, 128-bit loads and stores throughout.  Blocks past the weight
// range own 64 bias columns each: bias gradient = column sums of delta (row order),
// then the same update for the bias.
constexpr int UPD_THREADS = 256;
constexpr int UPD_VEC_PER_THREAD = 2;     // x 8 elements
constexpr int BIAS_COLS = 64;

__global__ void __launch_bounds__(UPD_THREADS) sgd_update_kernel(const UpdateArgs a, int w_blocks) {
  if (int(blockIdx.x) < w_blocks) {
    const long long nvec = a.n_elems >> 3;
    const long long base = (long long)blockIdx.x * (UPD_THREADS * UPD_VEC_PER_THREAD) + threadIdx.x;
#pragma unroll
    for (int u = 0; u < UPD_VEC_PER_THREAD; ++u) {
      const long long v = base + (long long)u * UPD_THREADS;
      if (v >= nvec) break;
      const long long e = v << 3;
      const float4 g0 = __ldcs(reinterpret_cast<const float4*>(a.dW + e));
      const float4 g1 = __ldcs(reinterpret_cast<const float4*>(a.dW + e + 4));
      float4 w0 = *reinterpret_cast<const float4*>(a.W + e);
      float4 w1 = *reinterpret_cast<const float4*>(a.W + e + 4);
      float4 m0 = g0, m1 = g1;
      if (a.mW != nullptr) {
        const float4 p0 = *reinterpret_cast<const float4*>(a.mW + e);
        const float4 p1 = *reinterpret_cast<const float4*>(a.mW + e + 4);
        m0.x = a.mu * p0.x + g0.x; m0.y = a.mu * p0.y + g0.y; m0.z = a.mu * p0.z + g0.z; m0.w = a.mu * p0.w + g0.w;
        m1.x = a.mu * p1.x + g1.x; m1.y = a.mu * p1.y + g1.y; m1.z = a.mu * p1.z + g1.z; m1.w = a.mu * p1.w + g1.w;
        *reinterpret_cast<float4*>(a.mW + e) = m0;
        *reinterpret_cast<float4*>(a.mW + e + 4) = m1;
      }
      w0.x -= a.lr * m0.x; w0.y -= a.lr * m0.y; w0.z -= a.lr * m0.z; w0.w -= a.lr * m0.w;
      w1.x -= a.lr * m1.x; w1.y -= a.lr * m1.y; w1.z -= a.lr * m1.z; w1.w -= a.lr * m1.w;
      *reinterpret_cast<float4*>(a.W + e) = w0;
      *reinterpret_cast<float4*>(a.W + e + 4) = w1;
      __nv_bfloat162 q0 = __floats2bfloat162_rn(w0.x, w0.y);
      __nv_bfloat162 q1 = __floats2bfloat162_rn(w0.z, w0.w);
      __nv_bfloat162 q2 = __floats2bfloat162_rn(w1.x, w1.y);
      __nv_bfloat162 q3 = __floats2bfloat162_rn(w1.z, w1.w);
      uint4 o;
      o.x = *reinterpret_cast<uint32_t*>(&q0);
      o.y = *reinterpret_cast<uint32_t*>(&q1);
      o.z = *reinterpret_cast<uint32_t*>(&q2);
      o.w = *reinterpret_cast<uint32_t*>(&q3);
      *reinterpret_cast<uint4*>(a.ring + e) = o;
    }
    return;
  }
  // ---- bias part: this block owns BIAS_COLS columns --------------------------
  __shared__ float part[UPD_THREADS / BIAS_COLS][BIAS_COLS];
  const int cb = (int(blockIdx.x) - w_blocks) * BIAS_COLS;
  const int tx = threadIdx.x % BIAS_COLS, ty = threadIdx.x / BIAS_COLS;
  constexpr int NY = UPD_THREADS / BIAS_COLS;
  const int col = cb + tx;
  float acc = 0.f;
  if (col < a.n_out) {
    if (a.col_partial != nullptr) {
      // chunk sums of the first pass, interleaved over the four thread rows; the loads of eight
      // chunks are in flight together (one dependent load per chunk cost 124 us on 1568 chunks)
#pragma unroll 8
      for (int ch = ty; ch < a.n_chunks; ch += NY) acc += __ldg(a.col_partial + (long long)ch * a.n_out + col);
    } else {
      for (int r = ty; r < a.rows; r += NY) acc += __bfloat162float(a.delta[(long long)r * a.ldd + col]);
    }
  }
  part[ty][tx] = acc;
  __syncthreads();
  if (ty == 0 && col < a.n_out) {
    float g = 0.f;
#pragma unroll
    for (int i = 0; i < NY; ++i) g += part[i][tx];
    a.db[col] = g;
    float m = g;
    if (a.mb != nullptr) {
      m = a.mu * a.mb[col] + g;
      a.mb[col] = m;
    }
    const float b = a.b[col] - a.lr * m;
    a.b[col] = b;
    a.bring[col] = b;
  }
}

cudaError_t launch_sgd_update(const UpdateArgs& a, cudaStream_t stream) {
  const long long nvec = a.n_elems >> 3;
  const long long per_block = UPD_THREADS * UPD_VEC_PER_THREAD;
  const int w_blocks = int((nvec + per_block - 1) / per_block);
  const int b_blocks = a.delta ? (a.n_out + BIAS_COLS - 1) / BIAS_COLS : 0;
  sgd_update_kernel<<<w_blocks + b_blocks, UPD_THREADS, 0, stream>>>(a, w_blocks);
  return cudaGetLastError();
}

}  // namespace lp

namespace lp {
// dst = RN_bf16(src), n a multiple of 8 (used once per layer to seed ring slot 0).
__global__ void round_to_bf16_kernel(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst, long long nvec) {
  for (long long v = blockIdx.x * (long long)blockDim.x + threadIdx.x; v < nvec; v += (long long)gridDim.x * blockDim.x) {
    const float4 a = *reinterpret_cast<const float4*>(src + v * 8);
    const float4 b = *reinterpret_cast<const float4*>(src + v * 8 + 4);
    __nv_bfloat162 q0 = __floats2bfloat162_rn(a.x, a.y), q1 = __floats2bfloat162_rn(a.z, a.w);
    __nv_bfloat162 q2 = __floats2bfloat162_rn(b.x, b.y), q3 = __floats2bfloat162_rn(b.z, b.w);
    uint4 o;
    o.x = *reinterpret_cast<uint32_t*>(&q0); o.y = *reinterpret_cast<uint32_t*>(&q1);
    o.z = *reinterpret_cast<uint32_t*>(&q2); o.w = *reinterpret_cast<uint32_t*>(&q3);
    *reinterpret_cast<uint4*>(dst + v * 8) = o;
  }
}
cudaError_t launch_round_to_bf16(const float* src, __nv_bfloat16* dst, long long n_elems, cudaStream_t stream) {
  const long long nvec = n_elems >> 3;
  int blocks = int(std::min<long long>((nvec + 255) / 256, 148 * 16));
  if (blocks < 1) blocks = 1;
  round_to_bf16_kernel<<<blocks, 256, 0, stream>>>(src, dst, nvec);
  return cudaGetLastError();
}
}  // namespace lp

namespace lp {
// ---------------------------------------------------------------------------
// 2x2 stride-2 max pool, NHWC, 8 channels (16 bytes) per thread.
__global__ void maxpool2_kernel(const __nv_bfloat16* __restrict__ a, __nv_bfloat16* __restrict__ pooled,
                                unsigned char* __restrict__ idx, int B, int H, int W, int C) {
  const int Hp = H / 2, Wp = W / 2, cg = C / 8;
  const long long total = (long long)B * Hp * Wp * cg;
  for (long long t = blockIdx.x * (long long)blockDim.x + threadIdx.x; t < total; t += (long long)gridDim.x * blockDim.x) {
    const int c8 = int(t % cg);
    long long pp = t / cg;
    const int pw = int(pp % Wp);
    const int ph = int((pp / Wp) % Hp);
    const int n = int(pp / ((long long)Wp * Hp));
    float best[8];
    unsigned char bi[8];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const long long src = (((long long)n * H + 2 * ph + (k >> 1)) * W + 2 * pw + (k & 1)) * C + c8 * 8;
      const uint4 v = *reinterpret_cast<const uint4*>(a + src);
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float lo = __uint_as_float(w[j] << 16), hi = __uint_as_float(w[j] & 0xFFFF0000u);
        if (k == 0 || lo > best[2 * j]) { best[2 * j] = lo; bi[2 * j] = (unsigned char)k; }
        if (k == 0 || hi > best[2 * j + 1]) { best[2 * j + 1] = hi; bi[2 * j + 1] = (unsigned char)k; }
      }
    }
    uint4 o;
    uint32_t* ow = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
    for (int j = 0; j < 4; ++j)
      ow[j] = (__float_as_uint(best[2 * j]) >> 16) | (__float_as_uint(best[2 * j + 1]) & 0xFFFF0000u);
    const long long dst = pp * C + c8 * 8;
    *reinterpret_cast<uint4*>(pooled + dst) = o;
    uint2 ib;
    ib.x = bi[0] | (bi[1] << 8) | (bi[2] << 16) | (bi[3] << 24);
    ib.y = bi[4] | (bi[5] << 8) | (bi[6] << 16) | (bi[7] << 24);
    *reinterpret_cast<uint2*>(idx + dst) = ib;
  }
}
cudaError_t launch_maxpool2(const __nv_bfloat16* a, __nv_bfloat16* pooled, unsigned char* idx, int B, int H, int W,
                            int C, cudaStream_t stream) {
  const long long total = (long long)B * (H / 2) * (W / 2) * (C / 8);
  int blocks = int(std::min<long long>((total + 255) / 256, 148 * 16));
  if (blocks < 1) blocks = 1;
  maxpool2_kernel<<<blocks, 256, 0, stream>>>(a, pooled, idx, B, H, W, C);
  return cudaGetLastError();
}

// partial[chunk][col] = sum over the chunk's rows (in row order, 4-way interleaved like the
// single-pass bias reduction) of x[row][col]
__global__ void colsum_partial_kernel(const __nv_bfloat16* __restrict__ x, int rows, int ld, int n_cols, int chunk_rows,
                                      float* __restrict__ partial) {
  __shared__ float part[4][64];
  const int tx = threadIdx.x % 64, ty = threadIdx.x / 64;
  const int col = blockIdx.x * 64 + tx;
  const int r0 = blockIdx.y * chunk_rows, r1 = min(rows, r0 + chunk_rows);
  float acc = 0.f;
  if (col < n_cols)
    for (int r = r0 + ty; r < r1; r += 4) acc += __bfloat162float(x[(long long)r * ld + col]);
  part[ty][tx] = acc;
  __syncthreads();
  if (ty == 0 && col < n_cols) partial[(long long)blockIdx.y * n_cols + col] = part[0][tx] + part[1][tx] + part[2][tx] + part[3][tx];
}
cudaError_t launch_colsum_partial(const __nv_bfloat16* x, int rows, int ld, int n_cols, float* partial,
                                  cudaStream_t stream) {
  const int chunk = colsum_chunk_rows(rows);
  dim3 grid((n_cols + 63) / 64, (rows + chunk - 1) / chunk);
  colsum_partial_kernel<<<grid, 256, 0, stream>>>(x, rows, ld, n_cols, chunk, partial);
  return cudaGetLastError();
}
}  // namespace lp

// ---------------------------------------------------------------------------
// lp_softmax_xent_static: the loss kernel for callers that cannot supply scratch memory.
// The per-row losses and the completion counter live in this fixed device array instead
// of a workspace.  Host code must not pass `g_xent_scratch` itself to a kernel: in host
// code that name is only a handle for the runtime.  The device address is looked up once
// per device with cudaGetSymbolAddress and that pointer is what the kernel receives.
struct XentScratch {
  float row_loss[LP_XENT_STATIC_MAX_BATCH];
  unsigned ticket;
};
static __device__ __align__(256) unsigned char g_xent_scratch[sizeof(XentScratch)];

namespace {
constexpr int kMaxDevices = 64;
// device address of the array, per device; written once per device under the mutex, read with acquire
std::atomic<XentScratch*> g_xent_scratch_addr[kMaxDevices];
std::mutex g_xent_setup_mutex;
int xent_fail(int code, const std::string& why) {
  lp::set_global_error("lp_softmax_xent_static: " + why);     // readable through lp_last_error(NULL)
  return code;
}
}  // namespace

extern "C" int lp_softmax_xent_static(const float* logits_dev, int ld_logits, const int* labels_dev,
                                      void* delta_dev, int ld_delta, float* loss_dev, int batch, int classes,
                                      void* stream) {
  if (!logits_dev || !labels_dev || !delta_dev || !loss_dev) return xent_fail(LP_ERR_INVALID_ARG, "null pointer");
  if (batch < 1 || classes < 1) return xent_fail(LP_ERR_INVALID_ARG, "batch and classes must be positive");
  if (batch > LP_XENT_STATIC_MAX_BATCH)     // the fixed scratch holds no more rows
    return xent_fail(LP_ERR_INVALID_ARG, "batch exceeds LP_XENT_STATIC_MAX_BATCH (" + std::to_string(LP_XENT_STATIC_MAX_BATCH) + " rows of built-in scratch)");
  if (ld_logits < classes || ld_delta < ((classes + 7) & ~7))
    return xent_fail(LP_ERR_INVALID_ARG, "row pitch smaller than the (padded) number of classes");
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return xent_fail(LP_ERR_CUDA, "no current CUDA device");
  XentScratch* s = g_xent_scratch_addr[dev].load(std::memory_order_acquire);
  if (s == nullptr) {
    // set-up, once per device, with that device current: ask the runtime where the array lives
    std::lock_guard<std::mutex> lock(g_xent_setup_mutex);
    s = g_xent_scratch_addr[dev].load(std::memory_order_relaxed);
    if (s == nullptr) {
      void* p = nullptr;
      cudaError_t e = cudaGetSymbolAddress(&p, g_xent_scratch);
      if (e != cudaSuccess || p == nullptr) return xent_fail(LP_ERR_CUDA, std::string("cudaGetSymbolAddress: ") + cudaGetErrorString(e));
      s = static_cast<XentScratch*>(p);
      g_xent_scratch_addr[dev].store(s, std::memory_order_release);
    }
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the counter must start at zero whatever an earlier (possibly failed) call left behind
  cudaError_t e = cudaMemsetAsync(&s->ticket, 0, sizeof(unsigned), st);
  if (e != cudaSuccess) return xent_fail(LP_ERR_CUDA, std::string("cudaMemsetAsync: ") + cudaGetErrorString(e));
  e = lp::launch_softmax_xent(logits_dev, ld_logits, labels_dev, static_cast<__nv_bfloat16*>(delta_dev), ld_delta,
                              s->row_loss, &s->ticket, loss_dev, batch, classes, nullptr, st);
  if (e != cudaSuccess) return xent_fail(LP_ERR_CUDA, std::string("kernel launch: ") + cudaGetErrorString(e));
  return LP_OK;
}
