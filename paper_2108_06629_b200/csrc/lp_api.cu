// The trainer behind the C ABI: workspace layout, weight-version rings, activation
// stashes, and the stage scheduler that maps the paper's processors onto CUDA streams.
//
// Scheduling model.  Every lp_step enqueues all tasks of one minibatch n:
//   cast -> F_1..F_L -> loss -> for l = L..1 { delta_l , G_l -> U_l }
// Each task declares the buffers (ring slots, stash slots, delta buffers) it reads and
// writes; a small tracker turns read-after-write, write-after-read and write-after-write
// hazards on those buffers into event waits between streams.  Because F_l(n) only needs
// weight version max(0, n - d_l), tasks of consecutive minibatches overlap on the device
// exactly as far as the delays allow -- the pipelining of Section III-A -- while the
// results stay those of the minibatch-by-minibatch recursion.
//   LayerPipe schedule: per stage group three streams -- G+update (highest priority: it
//   hands buffers back to later minibatches), delta, forward -- so delta_l and G_l of one
//   layer run concurrently and delta^{l-1} is released as soon as delta_l is done.
//   Fused-B schedule: delta_l, G_l, U_l run back to back as ONE task on the stage's
//   backward stream and delta^{l-1} is released only when the whole task has finished.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <memory>

#include "common.h"
#include "gemm.cuh"
#include "conv_halo.cuh"

namespace lp {

cudaError_t conv_halo_g_launch(const CUtensorMap& tmX, const CUtensorMap& tmD, const ConvGeom& g, int batch, float* partial,
                               HaloGUpdate upd, int* status, cudaStream_t st);

constexpr int kDeltaSlots = 4;
constexpr int kLossRing = 256;
constexpr int kLogRing = 4096;
constexpr int kEventPool = 2048;
constexpr int kExtraStashSlots = 1;   // activation stash = d_l + 1 (retiming) + 1 so F may run one ahead

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
static inline int pad8(int x) { return (x + 7) & ~7; }

struct Ev {
  cudaEvent_t e = nullptr;
  cudaStream_t s = nullptr;
  int si = -1;             // index of the stream it was recorded on (see lp_ctx::stream_index)
  long long seq = 0;       // position in the handle's sequence of recorded events
};

struct Res {                 // one buffer (or ring slot) the tracker protects
  Ev last_write;
  std::vector<Ev> readers;
};

struct PixBox {          // box of pixels used as one tile dimension (see ConvGeom)
  int lw = 0, lh = 0, bw = 1, bh = 1, bn = 1, tiles_w = 1, tiles_h = 1;
};

struct Layer {
  lp_layer d;
  int stage = 0, delay = 0, slots = 1;
  int n_in = 0, n_out = 0, ld_in = 0, ld_out = 0;   // FC: features; conv: channels (ld = padded to 8)
  int x_slots = 1;
  // geometry.  FC: H = W = 1, in_rows = out_rows = B.  Conv (3x3, stride 1, pad 1): in_rows =
  // out_rows = B*H*W; weights are the matrix [Cout][9 * ld_in] (tap-major, padded channels).
  bool conv = false;
  int imH = 1, imW = 1, taps = 1;   // conv: INPUT image size; taps = R * S
  int oH = 1, oW = 1;               // conv: OUTPUT image size (before pooling)
  int cR = 1, cS = 1, cstride = 1, cpad = 0;
  bool gen = false;                 // a filter other than 3x3 / stride 1 / pad 1: general implicit-GEMM path only
  PixBox boxD;                      // delta of a strided layer: boxes of 128 pixels over one residue class of the input grid
  // First convolution layer with few input channels (9 * Cin <= 64): the stash holds 3x3 patches
  // [B*H*W][9 * Cin] and the layer runs as a plain GEMM over pixel rows; n_in = 9 * Cin, taps = 1,
  // c_in = the image's channel count.
  bool patch = false;
  int c_in = 0;
  int in_rows = 0, out_rows = 0;
  int w_rows = 0, w_ld = 0;          // weight matrix [w_rows][w_ld]
  int pool = 0, Hp = 1, Wp = 1;      // 2x2 max pool after the activation: pooled image size
  int next_rows = 0;                 // rows of the next layer's input matrix (pooled pixels or B)
  PixBox box128, box64;              // pixel boxes of 128 (forward / delta) and 64 (G) pixels
  __nv_bfloat16* a_full = nullptr;   // pool layers: activation before pooling [out_rows][ld_out]
  unsigned char* pidx = nullptr;     // pool layers: argmax per pooled element, one slot per stash slot of the next layer
  size_t pidx_elems = 0;
  float* col_partial = nullptr;      // bias gradient of large layers: partial column sums
  int col_chunks = 0;
  int split_g = 1;
  float* part_g = nullptr;
  unsigned* cnt_g = nullptr;
  Res rAfull;
  // device memory (all inside the workspace)
  float *W = nullptr, *mW = nullptr, *b = nullptr, *mb = nullptr, *dW = nullptr, *db = nullptr, *bring = nullptr;
  __nv_bfloat16 *ring = nullptr, *X = nullptr, *Z = nullptr, *delta = nullptr;
  size_t w_elems = 0, x_elems = 0, z_elems = 0, delta_elems = 0;
  int z_slots = 0;
  int bn_f = 128, bn_d = 128, bn_g = 128;
  int split_f = 1, split_d = 1;                 // split-K factors of the forward / delta contractions
  float *part_f = nullptr, *part_d = nullptr;   // fp32 partial tiles [tiles][splits][128][BN]
  unsigned *cnt_f = nullptr, *cnt_d = nullptr;  // per-tile arrival counters
  std::vector<CUtensorMap> tm_f_A, tm_f_B, tm_d_A, tm_d_B, tm_g_A, tm_g_B;
  // 3x3 layers with at most 64 channels on both sides and images tiled by 8 x 16 pixels: the
  // activation / delta box is fetched once per tile with its halo (see conv_halo.cuh)
  bool halo_f = false, halo_d = false, halo_g = false;
  std::vector<CUtensorMap> tm_hg_D;             // delta as 8 x 16 pixel boxes (the halo-tile G kernel)
  bool lean_f = false;                          // patch-matrix layer with at most 64 output channels: forward through the same kernel
  std::vector<CUtensorMap> tm_hf_A, tm_hd_A;    // halo boxes over the stash slots / the delta slots
  std::vector<CUtensorMap> tm_hf_O;             // forward output (next layer's stash slots, or the pre-pool buffer) as 8 x 16 pixel boxes
  bool upd_maps = false;                        // fused update streamed by TMA (fully connected layers, 128-wide tiles)
  CUtensorMap tm_u_W, tm_u_M;                   // fp32 master / momentum as 32-column boxes
  std::vector<CUtensorMap> tm_u_R;              // each ring slot as 32-column bf16 boxes
  std::vector<Res> rX, rZ, rDelta, rRing, rPidx;
  Res rDW;
  Ev last_update;
  // Section III-B: the delta contraction of this layer split by output columns into delta'' =
  // columns [0, split_col), run on the streams of piece_stage[0] (the stage holding layer l+1),
  // and delta' = columns [split_col, n_in), run on piece_stage[1].  split_col = 0: one piece.
  int split_col = 0;
  int piece_stage[2] = {0, 0};
  // Activation recomputation (LP_RECOMPUTE): this layer's INPUT a^{l-1} (with the stored z^{l-1} and the
  // pooling positions that go with it) is not stashed for d_l + 2 minibatches.  The forward pass
  // keeps it in two short-lived slots (0, 1); when the backward pass of minibatch n reaches the
  // layer's stage, the forward task of layer l-1 is run again, with the same stashed weight
  // version, into slots 2 + n % 2, which is what G_l(n) and the f' multiply read.
  bool recomp = false;
};
// slot of layer y's input stash (and of what is stored with it) used by the forward pass / by the
// backward pass of minibatch n
static inline int xf_slot(const Layer& y, long long n) { return y.recomp ? int(n & 1) : int(n % y.x_slots); }
static inline int xb_slot(const Layer& y, long long n) { return y.recomp ? 2 + int(n & 1) : int(n % y.x_slots); }

}  // namespace lp

struct lp_ctx {
  std::vector<lp::Layer> L;
  lp_config cfg{};
  int n_stages = 0;
  int stages_used = 0;
  int n_groups = 1;             // stream triples; stage s runs on triple s % n_groups
  int tmem_policy = 0;          // TMEM_*: how pair and single-CTA kernels keep out of each other's tensor memory
  int classes = 0, ld_cls = 0;
  // shared buffers
  float* zL = nullptr;          // [kDeltaSlots][B][ld_cls] fp32
  int* labels = nullptr;        // [kDeltaSlots][B]
  float* row_loss = nullptr;    // [kDeltaSlots][B]
  unsigned* ticket = nullptr;   // [kDeltaSlots]
  float* loss = nullptr;        // [kLossRing]
  int* status = nullptr;        // device status word
  std::vector<lp::Res> rZL, rLabels;
  // streams / events
  std::vector<cudaStream_t> sF, sD, sG;
  // Events of the hazard tracker.  A handle stored in a Res must stay valid until that buffer's next
  // write, at most max(x_slots) minibatches later, so the pool holds more events than that many
  // minibatches can record; joins that nothing stores (lp_flush, the two pieces of a split delta)
  // take theirs from a small pool of their own.
  std::vector<cudaEvent_t> pool;
  size_t pool_next = 0;
  std::vector<cudaEvent_t> jpool;
  size_t jpool_next = 0;
  long long ev_seq = 0;
  // waited[a][b]: the latest event (by sequence number) of stream b that stream a already waits for.
  // Events of one stream complete in order, so waiting for an earlier one again is redundant.
  std::vector<cudaStream_t> streams;          // index 0 = the caller's stream of the current lp_step
  std::vector<std::vector<long long>> waited;
  int stream_index(cudaStream_t s) const {
    for (size_t i = 1; i < streams.size(); ++i) if (streams[i] == s) return int(i);
    return 0;
  }
  std::vector<lp::Ev> loss_ev;
  // bookkeeping
  long long n_steps = 0;
  long long launches = 0;
  std::vector<int> log_v, log_slot;   // [kLogRing][L]
  std::vector<cudaEvent_t> tpool;              // timing events (LP_TIME_TASKS)
  size_t tpool_next = 0;
  std::vector<std::pair<cudaEvent_t, cudaEvent_t>> timed[6];
  std::vector<int> timed_layer[6];             // layer of each timed launch (-1: none)
  // task progress marks (LP_TRACE_TASKS): per scheduler stream, how many tasks were enqueued and, in
  // pinned host memory that a one-thread kernel writes after each task, how many have completed
  struct TraceRec { int kind, layer; long long n; };
  static constexpr int kTraceRing = 1024;
  unsigned* trace_done = nullptr;              // [2][streams.size()] pinned, mapped: tasks finished, tasks started
  std::vector<unsigned> trace_enq;
  std::vector<std::vector<TraceRec>> trace_ring;
  int* tmem_table = nullptr;                   // [160][16] per-SM tensor-memory accounting (device)
  cudaStream_t peek_stream = nullptr;          // reads the status word while the scheduler streams are busy
  int* peek_host = nullptr;
  std::string err;
  int latched = 0;
  char* ws = nullptr;
  size_t ws_bytes = 0;
};

namespace lp {

static thread_local std::string g_err;   // for calls without a handle
void set_global_error(const std::string& msg) { g_err = msg; }

static int fail(lp_ctx* h, int code, const std::string& msg) {
  if (h) {
    h->err = msg;
    if (code == LP_ERR_CUDA) h->latched = code;
  } else {
    g_err = msg;
  }
  return code;
}
#define LP_CUDA(h, call)                                                                        \
  do {                                                                                          \
    cudaError_t e__ = (call);                                                                   \
    if (e__ != cudaSuccess)                                                                     \
      return fail(h, LP_ERR_CUDA, std::string(#call) + ": " + cudaGetErrorString(e__));         \
  } while (0)

// Factor `pixels` (128 or 64) into a box bw x bh x bn of powers of two with bw | W, bh | H, bn | B,
// widest in w first (longest contiguous runs).
static int pick_box(int W, int H, int B, int pixels, PixBox* out) {
  int bw = 1, lw = 0;
  while (bw * 2 <= pixels && W % (bw * 2) == 0) { bw *= 2; ++lw; }
  int bh = 1, lh = 0;
  while (bw * bh * 2 <= pixels && H % (bh * 2) == 0) { bh *= 2; ++lh; }
  const int bn = pixels / (bw * bh);
  if (bn < 1 || B % bn != 0) return LP_ERR_UNSUPPORTED;
  if (out) { out->lw = lw; out->lh = lh; out->bw = bw; out->bh = bh; out->bn = bn; out->tiles_w = W / bw; out->tiles_h = H / bh; }
  return LP_OK;
}

// ---------------------------------------------------------------------------
static int validate(const lp_layer* layers, int n, const lp_config* cfg, std::string* why) {
  if (!layers || n < 1 || !cfg) { *why = "null layer list or config"; return LP_ERR_INVALID_ARG; }
  if (cfg->batch < 1) { *why = "batch must be >= 1"; return LP_ERR_INVALID_ARG; }
  if (cfg->schedule != LP_SCHED_LAYERPIPE && cfg->schedule != LP_SCHED_FUSED_B) { *why = "unknown schedule"; return LP_ERR_INVALID_ARG; }
  if (cfg->input_dtype != LP_F32 && cfg->input_dtype != LP_BF16) { *why = "unknown input dtype"; return LP_ERR_INVALID_ARG; }
  for (int l = 0; l < n; ++l) {
    const lp_layer& y = layers[l];
    if (y.kind != LP_FC && y.kind != LP_CONV) { *why = "unknown layer kind"; return LP_ERR_INVALID_ARG; }
    if (y.in < 1 || y.out < 1) { *why = "layer sizes must be positive"; return LP_ERR_INVALID_ARG; }
    if (y.act < LP_ACT_NONE || y.act > LP_ACT_GELU) { *why = "unknown activation"; return LP_ERR_INVALID_ARG; }
    if (l == n - 1 && y.act != LP_ACT_NONE) { *why = "last layer must have no activation"; return LP_ERR_INVALID_ARG; }
    if (y.kind == LP_CONV) {
      if (y.R < 1 || y.R > 7 || y.S < 1 || y.S > 7 || y.stride < 1 || y.stride > 2 || y.pad < 0 || y.pad >= y.R || y.pad >= y.S) {
        *why = "convolutions are built for filters up to 7x7, stride 1 or 2, padding smaller than the filter"; return LP_ERR_UNSUPPORTED;
      }
      if (y.H < 1 || y.W < 1) { *why = "bad image size"; return LP_ERR_INVALID_ARG; }
      if (y.H + 2 * y.pad < y.R || y.W + 2 * y.pad < y.S) { *why = "filter larger than the padded image"; return LP_ERR_INVALID_ARG; }
      if (y.H % y.stride || y.W % y.stride) { *why = "a strided convolution needs an image size divisible by the stride"; return LP_ERR_UNSUPPORTED; }
      if ((long long)cfg->batch * y.H * y.W >= (1ll << 31) / 64) { *why = "batch x image size too large (pixel rows are indexed with 32 bits)"; return LP_ERR_UNSUPPORTED; }
      if (y.act == LP_ACT_GELU) { *why = "GELU after a convolution is not built"; return LP_ERR_UNSUPPORTED; }
      if (y.out % 8 != 0) { *why = "convolution output channels must be a multiple of 8"; return LP_ERR_UNSUPPORTED; }
      const int oh = (y.H + 2 * y.pad - y.R) / y.stride + 1, ow = (y.W + 2 * y.pad - y.S) / y.stride + 1;
      if (y.pool != 0 && (y.pool != 2 || oh % 2 || ow % 2 || y.act != LP_ACT_RELU)) { *why = "pooling must be 2x2 on even images after ReLU"; return LP_ERR_UNSUPPORTED; }
      if (l == n - 1) { *why = "the last layer must be fully connected"; return LP_ERR_UNSUPPORTED; }
      if (pick_box(ow, oh, cfg->batch, 128, nullptr) != LP_OK || pick_box(ow, oh, cfg->batch, 64, nullptr) != LP_OK ||
          pick_box(y.W / y.stride, y.H / y.stride, cfg->batch, 128, nullptr) != LP_OK) {
        *why = "image size / batch cannot be tiled into boxes of 128 and 64 pixels"; return LP_ERR_UNSUPPORTED;
      }
    } else if (y.pool != 0) { *why = "pooling needs a convolution layer"; return LP_ERR_INVALID_ARG; }
    if (l > 0) {
      const lp_layer& pv = layers[l - 1];
      const int ph = pv.kind == LP_CONV ? ((pv.H + 2 * pv.pad - pv.R) / pv.stride + 1) / (pv.pool ? 2 : 1) : 1;
      const int pw = pv.kind == LP_CONV ? ((pv.W + 2 * pv.pad - pv.S) / pv.stride + 1) / (pv.pool ? 2 : 1) : 1;
      if (y.kind == LP_CONV) {
        if (pv.kind != LP_CONV || pv.out != y.in || ph != y.H || pw != y.W) { *why = "layer sizes do not chain"; return LP_ERR_INVALID_ARG; }
      } else {
        if ((long long)pv.out * ph * pw != y.in) { *why = "layer sizes do not chain"; return LP_ERR_INVALID_ARG; }
        if (pv.kind == LP_CONV && pv.act == LP_ACT_GELU) { *why = "GELU after a convolution is not built"; return LP_ERR_UNSUPPORTED; }
      }
    }
  }
  return LP_OK;
}

static int resolve_plan(const lp_layer* layers, int n, int n_stages, const int* stage, const int* delays,
                        const lp_config* cfg, std::vector<int>* st, std::vector<int>* dl, int* used, std::string* why) {
  if (n_stages < 1) { *why = "n_stages must be >= 1"; return LP_ERR_INVALID_ARG; }
  st->assign(n, 0);
  dl->assign(n, 0);
  if (stage) {
    int mx = 0;
    for (int l = 0; l < n; ++l) {
      if (stage[l] < 0 || stage[l] >= n_stages || (l > 0 && stage[l] < stage[l - 1])) {
        *why = "stage map must be non-decreasing and within [0, n_stages)";
        return LP_ERR_INVALID_ARG;
      }
      (*st)[l] = stage[l];
      mx = std::max(mx, stage[l]);
    }
    *used = mx + 1;
  } else {
    PlanResult r;
    int rc = plan_layers(layers, n, cfg->batch, n_stages, &r);
    if (rc != LP_OK) { *why = "planner rejected the layer list"; return rc; }
    *st = r.stage;
    *used = r.used;
    if (delays) {
      // explicit delays with a planned stage map: keep the planner's stages for stream placement
    }
  }
  for (int l = 0; l < n; ++l) {
    (*dl)[l] = delays ? delays[l] : (*used - 1 - (*st)[l]);
    if ((*dl)[l] < 0 || (*dl)[l] > 1024) { *why = "delays must be in [0, 1024]"; return LP_ERR_INVALID_ARG; }
  }
  return LP_OK;
}

// Lays the network out in the workspace.  With base == nullptr only sizes are computed.
static size_t carve(lp_ctx* c, char* base) {
  size_t off = 0;
  auto take = [&](size_t bytes) -> char* {
    off = align_up(off, 256);
    char* p = base ? base + off : nullptr;
    off += bytes;
    return p;
  };
  const int B = c->cfg.batch;
  const bool mom = c->cfg.momentum != 0.f;
  const int nL = int(c->L.size());
  for (int l = 0; l < nL; ++l) {
    Layer& y = c->L[l];
    y.w_elems = size_t(y.w_rows) * y.w_ld;
    y.W = reinterpret_cast<float*>(take(y.w_elems * 4));
    y.mW = mom ? reinterpret_cast<float*>(take(y.w_elems * 4)) : nullptr;
    const bool keep_G = (c->cfg.flags & (LP_CAPTURE_GRADS | LP_UNFUSED_UPDATE)) != 0;
    y.dW = keep_G ? reinterpret_cast<float*>(take(y.w_elems * 4)) : nullptr;
    y.ring = reinterpret_cast<__nv_bfloat16*>(take(y.w_elems * 2 * y.slots));
    y.b = reinterpret_cast<float*>(take(size_t(y.ld_out) * 4));
    y.mb = mom ? reinterpret_cast<float*>(take(size_t(y.ld_out) * 4)) : nullptr;
    y.db = reinterpret_cast<float*>(take(size_t(y.ld_out) * 4));
    y.bring = reinterpret_cast<float*>(take(size_t(y.ld_out) * 4 * y.slots));
    y.x_elems = size_t(y.in_rows) * y.ld_in;
    y.X = reinterpret_cast<__nv_bfloat16*>(take(y.x_elems * 2 * y.x_slots));
    y.delta_elems = size_t(y.out_rows) * y.ld_out;
    y.delta = reinterpret_cast<__nv_bfloat16*>(take(y.delta_elems * 2 * kDeltaSlots));
    y.z_slots = 0;
    y.Z = nullptr;
    if (y.d.act == LP_ACT_GELU && l + 1 < nL) {
      y.z_slots = c->L[l + 1].x_slots;
      y.z_elems = size_t(B) * y.ld_out;
      y.Z = reinterpret_cast<__nv_bfloat16*>(take(y.z_elems * 2 * y.z_slots));
    }
    if (y.pool && l + 1 < nL) {
      y.a_full = reinterpret_cast<__nv_bfloat16*>(take(y.delta_elems * 2));
      y.pidx_elems = size_t(B) * y.Hp * y.Wp * y.ld_out;
      y.pidx = reinterpret_cast<unsigned char*>(take(y.pidx_elems * c->L[l + 1].x_slots));
    }
    if (y.col_chunks > 0) y.col_partial = reinterpret_cast<float*>(take(size_t(y.col_chunks) * y.ld_out * 4));
    auto tiles_of = [&](int M, int N, int bn) { return size_t((M + GEMM_BM - 1) / GEMM_BM) * ((N + bn - 1) / bn); };
    if (y.split_f > 1) {
      const size_t t = tiles_of(B, y.n_out, y.bn_f);
      y.part_f = reinterpret_cast<float*>(take(t * y.split_f * GEMM_BM * y.bn_f * 4));
      y.cnt_f = reinterpret_cast<unsigned*>(take(t * 4));
    }
    if (y.split_d > 1 && l > 0) {
      const size_t t = tiles_of(B, y.n_in, y.bn_d);
      y.part_d = reinterpret_cast<float*>(take(t * y.split_d * GEMM_BM * y.bn_d * 4));
      y.cnt_d = reinterpret_cast<unsigned*>(take(t * 4));
    }
    if (y.halo_g) {
      y.part_g = reinterpret_cast<float*>(take(size_t(conv_halo_g_max_ctas()) * HALOG_PART_FLOATS * 4));
    } else if (y.split_g > 1) {
      const size_t t = size_t((y.n_out + GEMM_BM - 1) / GEMM_BM) * y.taps * ((y.ld_in + y.bn_g - 1) / y.bn_g);
      y.part_g = reinterpret_cast<float*>(take(t * y.split_g * GEMM_BM * y.bn_g * 4));
      y.cnt_g = reinterpret_cast<unsigned*>(take(t * 4));
    }
  }
  c->zL = reinterpret_cast<float*>(take(size_t(kDeltaSlots) * B * c->ld_cls * 4));
  c->labels = reinterpret_cast<int*>(take(size_t(kDeltaSlots) * B * 4));
  c->row_loss = reinterpret_cast<float*>(take(size_t(kDeltaSlots) * B * 4));
  c->ticket = reinterpret_cast<unsigned*>(take(size_t(kDeltaSlots) * 4));
  c->loss = reinterpret_cast<float*>(take(size_t(kLossRing) * 4));
  c->status = reinterpret_cast<int*>(take(256));
  c->tmem_table = reinterpret_cast<int*>(take(160 * 16 * 4));
  return align_up(off, 256);
}

static void shape_layers(lp_ctx* c, const lp_layer* layers, int n, const std::vector<int>& st,
                         const std::vector<int>& dl) {
  c->L.resize(n);
  for (int l = 0; l < n; ++l) {
    Layer& y = c->L[l];
    y.d = layers[l];
    y.stage = st[l];
    y.delay = dl[l];
    y.slots = dl[l] + 1;
    y.n_in = layers[l].in;
    y.n_out = layers[l].out;
    y.ld_in = pad8(y.n_in);
    y.ld_out = pad8(y.n_out);
    y.x_slots = y.delay + 1 + kExtraStashSlots;
    // recomputation pays where the stash would hold more than the four slots it needs instead, and is
    // possible where the producing layer sits in the same stage (a stage keeps its own input stashed)
    y.recomp = (c->cfg.flags & LP_RECOMPUTE) != 0 && l > 0 && st[l] == st[l - 1] && y.x_slots > 4;
    if (y.recomp) y.x_slots = 4;
    const int B = c->cfg.batch;
    y.conv = layers[l].kind == LP_CONV;
    if (y.conv) {
      y.imH = layers[l].H; y.imW = layers[l].W;
      y.cR = layers[l].R; y.cS = layers[l].S; y.cstride = layers[l].stride; y.cpad = layers[l].pad;
      y.taps = y.cR * y.cS;
      y.oH = (y.imH + 2 * y.cpad - y.cR) / y.cstride + 1;
      y.oW = (y.imW + 2 * y.cpad - y.cS) / y.cstride + 1;
      y.gen = !(y.cR == 3 && y.cS == 3 && y.cstride == 1 && y.cpad == 1);
      // A first layer with few input channels keeps its input as the matrix of filter patches, one
      // row per OUTPUT pixel: 3x3 / stride 1 with at most 7 channels (9 Cin <= 64), and general filters
      // and strides with R S Cin <= 128 (the 5x5, stride-2, 3-channel layer of the paper's sample
      // network: 75 products per pixel instead of 25 taps x 64 padded channels).
      y.patch = l == 0 && (y.gen ? (y.taps * y.n_in <= 128 && y.n_in <= 8) : 9 * y.n_in <= 64);
      y.out_rows = B * y.oH * y.oW;
      y.in_rows = y.patch ? y.out_rows : B * y.imH * y.imW;
      if (y.patch) { y.c_in = y.n_in; y.n_in = y.taps * y.c_in; y.ld_in = pad8(y.n_in); y.taps = 1; }
      y.w_rows = y.n_out; y.w_ld = y.taps * y.ld_in;
      y.pool = layers[l].pool;
      y.Hp = y.pool ? y.oH / 2 : y.oH; y.Wp = y.pool ? y.oW / 2 : y.oW;
      y.next_rows = (l + 1 < n && layers[l + 1].kind == LP_CONV) ? B * y.Hp * y.Wp : B;
      pick_box(y.oW, y.oH, B, 128, &y.box128);      // forward: tile rows = output pixels
      pick_box(y.oW, y.oH, B, 64, &y.box64);        // G: the contraction runs over output pixels
      pick_box(y.imW / y.cstride, y.imH / y.cstride, B, 128, &y.boxD);   // delta: tile rows = input pixels of one residue class
      y.bn_f = y.n_out <= 64 ? 64 : 128;
      y.bn_d = y.ld_in <= 64 ? 64 : 128;
      y.bn_g = y.ld_in <= 64 ? 64 : 128;
      // Wide layers (at least 256 channels on both sides) on an even number of pixel boxes:
      // 256-pixel x 256-column tiles on SM pairs.  Measured on the VGG-16 layers at batch 64,
      // pair against single CTA: 512 -> 512 at 28^2 forward 180 / 245 us, delta 189 / 253 us;
      // 256 -> 256 at 56^2 216 / 240 and 230 / 249 us; 512 -> 512 at 14^2 66 / 79 and 67 / 84 us;
      // 128 -> 256 forward (18 k-blocks) is slower as a pair (149 / 131 us) and stays single.
      // Off by default: a convolutional network always has single-CTA kernels too, and the two kinds of
      // tensor-memory allocation do not mix (see the end of this function).  LP_CONV_PAIR=1 in the
      // environment turns the pair tiles on, as persistent CTA pairs that have their SMs to themselves
      // (gemm2q.cuh; VGG-16 step 7.75 ms against 8.38 ms) -- for measurements and the kernels' parity
      // tests, not for long runs.
      const bool even_boxes = ((y.in_rows / GEMM_BM) % 2) == 0;
      // 128 x 256 single-CTA tiles where gemm_pick_bn's rule for them holds (a long contraction, enough tiles for
      // one persistent CTA on every SM): a third less operand traffic per multiply-accumulate than 128 x 128
      const long long row_tiles = y.in_rows / GEMM_BM;
      if (!y.gen) {      // (VGG-16 step 8.40 -> 8.17 ms)
        if (y.n_out >= 256 && y.taps * y.ld_in >= 1024 && row_tiles * ((y.n_out + 255) / 256) >= 2 * 148) y.bn_f = 256;
        if (l > 0 && y.ld_in >= 256 && y.taps * y.n_out >= 1024 && row_tiles * ((y.ld_in + 255) / 256) >= 2 * 148) y.bn_d = 256;
      }
      const bool conv_pair = getenv("LP_CONV_PAIR") != nullptr;
      if (conv_pair && !y.gen && even_boxes && y.n_out >= 256 && y.ld_in >= 256) y.bn_f = GEMM_BN_PAIR;
      if (conv_pair && !y.gen && even_boxes && l > 0 && y.ld_in >= 256 && y.n_out >= 256) y.bn_d = GEMM_BN_PAIR;
      y.split_f = y.split_d = 1;
      const bool tiles_8x16 = !y.gen && (y.imW % 8 == 0) && (y.imH % 16 == 0);
      y.halo_f = !y.patch && tiles_8x16 && y.ld_in <= 64 && y.n_out <= 64;
      y.halo_d = l > 0 && tiles_8x16 && y.ld_out <= 64 && y.n_in <= 64;
      y.halo_g = y.halo_f;   // (128 output channels in two passes of the G kernel measured slower than the split-K kernel: 182 / 160 us)
      y.lean_f = y.patch && y.n_out <= 64 && y.ld_in <= 64 && l + 1 < n;
      // G contracts over all B*H*W pixels but has only (Cout/128) x 9 x (Cin/BN) tiles: the pixel
      // range is split.  A split costs the last CTA of the tile one more partial tile to add
      // (measured about 1.1 us for a 128-wide tile, half that for 64), a k-block about 0.33 us, so
      // the time kb/s * 0.33 + s * 1.1 is least near s = sqrt(0.3 kb) (0.6 kb for 64-wide tiles);
      // never more splits than fill two CTAs per SM.  Swept on the small VGG (2 .. 148 splits):
      // the measured optimum of every layer is the power of two next to this value.
      const int tiles = ((y.n_out + GEMM_BM - 1) / GEMM_BM) * y.taps * ((y.ld_in + y.bn_g - 1) / y.bn_g);
      const int num_kb = y.out_rows / GEMM_BK;
      const int s_opt = int(std::lround(std::sqrt(double(num_kb) * (y.bn_g <= 64 ? 0.6 : 0.3))));
      y.split_g = std::max(1, std::min(std::min(296 / std::max(tiles, 1), s_opt), y.patch ? 148 : 64));
      const int per = (num_kb + y.split_g - 1) / y.split_g;
      y.split_g = (num_kb + per - 1) / per;
    } else {
      y.in_rows = y.out_rows = y.next_rows = B;
      y.w_rows = y.n_out; y.w_ld = y.ld_in;
      y.bn_f = gemm_pick_bn(0, B, y.n_out, y.n_in);
      y.bn_d = gemm_pick_bn(1, B, y.n_in, y.n_out);
      y.bn_g = gemm_pick_bn(2, y.n_out, y.n_in, B);
      y.split_f = gemm_is_pair(y.bn_f) ? 1 : gemm_pick_splits(B, y.n_out, y.n_in, y.bn_f);
      y.split_d = gemm_is_pair(y.bn_d) ? 1 : gemm_pick_splits(B, y.n_in, y.n_out, y.bn_d);
      y.split_g = 1;
    }
    y.col_chunks = colsum_chunks(y.out_rows);
  }
  // One kind of tensor-memory allocation per handle.  SM-pair kernels (tcgen05 cta_group::2) and
  // single-CTA kernels (cta_group::1) that alternate on the same SMs ended, about once in 10^6 pair
  // CTAs, with a pair CTA waiting in tcgen05.alloc for ever on an otherwise idle GPU; handles of one
  // kind only never did.  So a fully connected network whose layers are mostly wide runs EVERY
  // contraction on SM pairs (the narrow classifier too: a 256-column tile that is mostly padding
  // costs microseconds), and every other network runs none there.
  const int B = c->cfg.batch;
  bool any_conv = false;
  int fc_pair = 0;
  for (int l = 0; l < n; ++l) {
    const Layer& y = c->L[l];
    any_conv = any_conv || y.conv;
    if (!y.conv && (gemm_is_pair(y.bn_f) || (l > 0 && gemm_is_pair(y.bn_d)) || gemm_is_pair(y.bn_g))) ++fc_pair;
  }
  const bool conv_pair = getenv("LP_CONV_PAIR") != nullptr;     // measurement aid, see the convolution branch above
  if (!conv_pair) {
    const bool pure_pair = !any_conv && fc_pair * 2 >= n;
    for (int l = 0; l < n; ++l) {
      Layer& y = c->L[l];
      if (y.conv) continue;
      if (pure_pair) {
        if (!gemm_is_pair(y.bn_f)) y.bn_f = GEMM_BN_PAIR;
        if (!gemm_is_pair(y.bn_d)) y.bn_d = GEMM_BN_PAIR;
        if (!gemm_is_pair(y.bn_g)) y.bn_g = GEMM_BN_PAIR;
        y.split_f = y.split_d = 1;
      } else if (fc_pair > 0) {
        y.bn_f = gemm_pick_bn(0, B, y.n_out, y.n_in, false);
        y.bn_d = gemm_pick_bn(1, B, y.n_in, y.n_out, false);
        y.bn_g = gemm_pick_bn(2, y.n_out, y.n_in, B, false);
        y.split_f = gemm_is_pair(y.bn_f) ? 1 : gemm_pick_splits(B, y.n_out, y.n_in, y.bn_f);
        y.split_d = gemm_is_pair(y.bn_d) ? 1 : gemm_pick_splits(B, y.n_in, y.n_out, y.bn_d);
      }
    }
  }
  c->tmem_policy = conv_pair ? TMEM_PAIR_ALONE : TMEM_DEFAULT;
  c->classes = layers[n - 1].out;
  c->ld_cls = pad8(c->classes);
}

// ---------------------------------------------------------------------------
// hazard tracker
static inline void wait_on(lp_ctx* c, cudaStream_t s, int si, const Ev& e, cudaError_t* err) {
  if (!e.e || e.s == s) return;
  if (e.si > 0) {                         // (index 0 is whatever stream the caller passes: never pruned)
    long long& w = c->waited[si][e.si];
    if (w >= e.seq) return;               // this stream already waits for that event or a later one of its stream
    w = e.seq;
  }
  cudaError_t r = cudaStreamWaitEvent(s, e.e, 0);
  if (r != cudaSuccess && *err == cudaSuccess) *err = r;
}

static cudaError_t task_begin(lp_ctx* c, cudaStream_t s, std::initializer_list<Res*> reads,
                              std::initializer_list<Res*> writes) {
  cudaError_t err = cudaSuccess;
  const int si = c->stream_index(s);
  for (Res* r : reads) if (r) wait_on(c, s, si, r->last_write, &err);
  for (Res* w : writes) {
    if (!w) continue;
    wait_on(c, s, si, w->last_write, &err);
    for (const Ev& e : w->readers) wait_on(c, s, si, e, &err);
  }
  return err;
}

static cudaError_t task_end(lp_ctx* c, cudaStream_t s, std::initializer_list<Res*> reads,
                            std::initializer_list<Res*> writes, Ev* out_ev) {
  cudaEvent_t e = c->pool[c->pool_next++ % c->pool.size()];
  cudaError_t r = cudaEventRecord(e, s);
  Ev ev{e, s, c->stream_index(s), ++c->ev_seq};
  for (Res* x : reads) if (x) x->readers.push_back(ev);
  for (Res* w : writes) {
    if (!w) continue;
    w->last_write = ev;
    w->readers.clear();
  }
  if (out_ev) *out_ev = ev;
  return r;
}

// ---------------------------------------------------------------------------
static int build_tensor_maps(lp_ctx* c) {
  const int B = c->cfg.batch;
  const int nL = int(c->L.size());
  std::string err;
  for (int l = 0; l < nL; ++l) {
    Layer& y = c->L[l];
    uint32_t bA[2], bB[2];
    int rc;
    y.tm_f_A.resize(y.x_slots);
    y.tm_f_B.resize(y.slots);
    y.tm_d_A.resize(kDeltaSlots);
    y.tm_d_B.resize(y.slots);
    y.tm_g_A.resize(kDeltaSlots);
    y.tm_g_B.resize(y.x_slots);
    if (y.conv && !y.patch) {
      // forward: A = a^{l-1} as NHWC boxes of 128 pixels; B = W [Cout][9 * ld_in] K-major
      // delta:   A = delta^l as NHWC boxes of 128 pixels; B = the same W matrix read MN-major
      // G:       A = delta^l, B = a^{l-1}, both as NHWC boxes of 64 pixels (the contraction index)
      for (int s = 0; s < y.x_slots; ++s) {
        // (the stash is the layer's INPUT image; a box of output pixels reads every stride-th input pixel)
        if ((rc = make_tmap_bf16_nhwc(&y.tm_f_A[s], y.X + s * y.x_elems, y.ld_in, y.imW, y.imH, B, y.ld_in, y.box128.bw,
                                      y.box128.bh, y.box128.bn, &err, y.cstride)) != LP_OK) return fail(c, rc, err);
        if ((rc = make_tmap_bf16_nhwc(&y.tm_g_B[s], y.X + s * y.x_elems, y.ld_in, y.imW, y.imH, B, y.ld_in, y.box64.bw,
                                      y.box64.bh, y.box64.bn, &err, y.cstride)) != LP_OK) return fail(c, rc, err);
      }
      for (int s = 0; s < kDeltaSlots; ++s) {
        // (delta^l lives on the layer's OUTPUT grid; the delta contraction walks it in boxes that match one residue class
        // of the input grid, the G contraction in boxes of 64 output pixels)
        if ((rc = make_tmap_bf16_nhwc(&y.tm_d_A[s], y.delta + s * y.delta_elems, y.ld_out, y.oW, y.oH, B, y.ld_out,
                                      y.boxD.bw, y.boxD.bh, y.boxD.bn, &err)) != LP_OK) return fail(c, rc, err);
        if ((rc = make_tmap_bf16_nhwc(&y.tm_g_A[s], y.delta + s * y.delta_elems, y.ld_out, y.oW, y.oH, B, y.ld_out,
                                      y.box64.bw, y.box64.bh, y.box64.bn, &err)) != LP_OK) return fail(c, rc, err);
      }
      if (y.halo_f || y.halo_g) {      // the halo box over the stashed input (forward and G)
        y.tm_hf_A.resize(y.x_slots);
        for (int s = 0; s < y.x_slots; ++s)
          if ((rc = make_tmap_bf16_nhwc(&y.tm_hf_A[s], y.X + s * y.x_elems, y.ld_in, y.imW, y.imH, B, y.ld_in, HALO_W, HALO_H, 1,
                                        &err)) != LP_OK) return fail(c, rc, err);
      }
      if (y.halo_f) {
        // the layer's output: NHWC [B][H][W][ld_out], one map per destination
        Layer& nx = c->L[l + 1];
        const int n_dst = y.pool ? 1 : nx.x_slots;
        y.tm_hf_O.resize(n_dst);
        for (int s = 0; s < n_dst; ++s) {
          const __nv_bfloat16* dst = y.pool ? y.a_full : nx.X + size_t(s) * nx.x_elems;
          if ((rc = make_tmap_bf16_nhwc(&y.tm_hf_O[s], dst, y.ld_out, y.imW, y.imH, B, y.ld_out, 8, 16, 1, &err)) != LP_OK)
            return fail(c, rc, err);
        }
      }
      if (y.halo_g) {
        y.tm_hg_D.resize(kDeltaSlots);
        for (int s = 0; s < kDeltaSlots; ++s)
          if ((rc = make_tmap_bf16_nhwc(&y.tm_hg_D[s], y.delta + s * y.delta_elems, y.ld_out, y.imW, y.imH, B, y.ld_out, 8, 16, 1,
                                        &err)) != LP_OK) return fail(c, rc, err);
      }
      if (y.halo_d) {
        y.tm_hd_A.resize(kDeltaSlots);
        for (int s = 0; s < kDeltaSlots; ++s)
          if ((rc = make_tmap_bf16_nhwc(&y.tm_hd_A[s], y.delta + s * y.delta_elems, y.ld_out, y.imW, y.imH, B, y.ld_out, HALO_W,
                                        HALO_H, 1, &err)) != LP_OK) return fail(c, rc, err);
      }
      for (int s = 0; s < y.slots; ++s) {
        if ((rc = make_tmap_bf16_2d(&y.tm_f_B[s], y.ring + s * y.w_elems, y.w_ld, y.n_out, y.w_ld, 64,
                                    y.bn_f == GEMM_BN_PAIR ? 128 : y.bn_f, &err)) != LP_OK)   // a pair CTA stages half of the 256 columns
          return fail(c, rc, err);
        if ((rc = make_tmap_bf16_2d(&y.tm_d_B[s], y.ring + s * y.w_elems, y.w_ld, y.n_out, y.w_ld, 64, 64, &err)) != LP_OK)
          return fail(c, rc, err);
      }
      continue;
    }
    if (y.lean_f) {
      Layer& nx = c->L[l + 1];
      const int n_dst = y.pool ? 1 : nx.x_slots;
      y.tm_hf_O.resize(n_dst);
      for (int s = 0; s < n_dst; ++s) {
        const __nv_bfloat16* dst = y.pool ? y.a_full : nx.X + size_t(s) * nx.x_elems;
        if ((rc = make_tmap_bf16_2d(&y.tm_hf_O[s], dst, y.ld_out, y.out_rows, y.ld_out, 64, GEMM_BM, &err)) != LP_OK)
          return fail(c, rc, err);
      }
    }
    // (fully connected layers, and the patch layer whose rows are pixels)
    // forward: A = a^{l-1} [B][in] K-major; B = W [out][in] K-major
    gemm_box_dims(0, y.bn_f, bA, bB);
    for (int s = 0; s < y.x_slots; ++s)
      if ((rc = make_tmap_bf16_2d(&y.tm_f_A[s], y.X + s * y.x_elems, y.n_in, y.in_rows, y.ld_in, bA[0], bA[1], &err)) != LP_OK)
        return fail(c, rc, err);
    for (int s = 0; s < y.slots; ++s)
      if ((rc = make_tmap_bf16_2d(&y.tm_f_B[s], y.ring + s * y.w_elems, y.n_in, y.n_out, y.ld_in, bB[0], bB[1], &err)) != LP_OK)
        return fail(c, rc, err);
    // delta: A = delta^l [B][out] K-major (K = out); B = W [out][in] MN-major (N = in contiguous)
    gemm_box_dims(1, y.bn_d, bA, bB);
    for (int s = 0; s < kDeltaSlots; ++s)
      if ((rc = make_tmap_bf16_2d(&y.tm_d_A[s], y.delta + s * y.delta_elems, y.n_out, y.out_rows, y.ld_out, bA[0], bA[1], &err)) != LP_OK)
        return fail(c, rc, err);
    for (int s = 0; s < y.slots; ++s)
      if ((rc = make_tmap_bf16_2d(&y.tm_d_B[s], y.ring + s * y.w_elems, y.n_in, y.n_out, y.ld_in, bB[0], bB[1], &err)) != LP_OK)
        return fail(c, rc, err);
    // G: A = delta^l stored [B][out] -> MN-major (M = out contiguous); B = a^{l-1} stored [B][in] -> MN-major
    y.upd_maps = (y.bn_g == 128 || y.bn_g == 256 || y.bn_g == GEMM_BN_PAIR) && y.split_g == 1;
    if (y.upd_maps) {
      if ((rc = make_tmap_rows32(&y.tm_u_W, y.W, 4, y.n_in, y.n_out, y.w_ld, GEMM_BM, &err)) != LP_OK) return fail(c, rc, err);
      if (y.mW && (rc = make_tmap_rows32(&y.tm_u_M, y.mW, 4, y.n_in, y.n_out, y.w_ld, GEMM_BM, &err)) != LP_OK) return fail(c, rc, err);
      y.tm_u_R.resize(y.slots);
      for (int s = 0; s < y.slots; ++s)
        if ((rc = make_tmap_rows32(&y.tm_u_R[s], y.ring + s * y.w_elems, 2, y.n_in, y.n_out, y.w_ld, GEMM_BM, &err)) != LP_OK)
          return fail(c, rc, err);
    }
    gemm_box_dims(2, y.bn_g, bA, bB);
    for (int s = 0; s < kDeltaSlots; ++s)
      if ((rc = make_tmap_bf16_2d(&y.tm_g_A[s], y.delta + s * y.delta_elems, y.n_out, y.out_rows, y.ld_out, bA[0], bA[1], &err)) != LP_OK)
        return fail(c, rc, err);
    for (int s = 0; s < y.x_slots; ++s)
      if ((rc = make_tmap_bf16_2d(&y.tm_g_B[s], y.X + s * y.x_elems, y.n_in, y.in_rows, y.ld_in, bB[0], bB[1], &err)) != LP_OK)
        return fail(c, rc, err);
  }
  return LP_OK;
}

static void destroy_ctx(lp_ctx* c) {
  if (!c) return;
  auto kill = [](std::vector<cudaStream_t>& v) {
    for (cudaStream_t s : v) if (s) cudaStreamDestroy(s);
    v.clear();
  };
  cudaDeviceSynchronize();
  kill(c->sF);
  kill(c->sD);
  kill(c->sG);
  for (cudaEvent_t e : c->pool) if (e) cudaEventDestroy(e);
  for (cudaEvent_t e : c->jpool) if (e) cudaEventDestroy(e);
  for (cudaEvent_t e : c->tpool) if (e) cudaEventDestroy(e);
  if (c->trace_done) { gemm_set_tmem_table(nullptr); cudaFreeHost(c->trace_done); }
  if (c->peek_host) cudaFreeHost(c->peek_host);
  if (c->peek_stream) cudaStreamDestroy(c->peek_stream);
  delete c;
}

// Optional per-kernel timing: a start/stop event pair on the kernel's own stream.
struct TimedScope {
  lp_ctx* c;
  cudaStream_t st;
  int kind;
  cudaEvent_t e1 = nullptr;
  TimedScope(lp_ctx* c_, int kind_, cudaStream_t st_, int layer_ = -1) : c(c_), st(st_), kind(kind_), layer(layer_) {
    if ((c->cfg.flags & LP_TIME_TASKS) && c->tpool_next + 2 <= c->tpool.size()) {
      cudaEvent_t e0 = c->tpool[c->tpool_next++];
      e1 = c->tpool[c->tpool_next++];
      cudaEventRecord(e0, st);
      c->timed[kind].push_back({e0, e1});
      c->timed_layer[kind].push_back(layer);
    }
    if (c->trace_done) {     // runs once everything the task waits for has completed
      const int si = c->stream_index(st);
      launch_trace_mark(c->trace_done + c->streams.size() + si, c->trace_enq[si] + 1, st);
    }
  }
  ~TimedScope() {
    if (e1) cudaEventRecord(e1, st);
    if (c->trace_done) {
      const int si = c->stream_index(st);
      const unsigned seq = ++c->trace_enq[si];
      c->trace_ring[si][seq % lp_ctx::kTraceRing] = {kind, layer, c->n_steps};
      launch_trace_mark(c->trace_done + si, seq, st);
    }
  }
  int layer = -1;
};

// ---------------------------------------------------------------------------
// the kernels of one minibatch
static ConvGeom conv_geom(const Layer& y, int kind, const PixBox& bx, int flip, int chunks_per_tap, int n_per_tap) {
  ConvGeom g{};
  g.kind = kind;
  // PIX_M forward: rows index the output image; PIX_M delta: the input image (delta^{l-1}); PIX_K: the output grid
  g.H = (kind == GEOM_PIX_M && flip) ? y.imH : y.oH;
  g.W = (kind == GEOM_PIX_M && flip) ? y.imW : y.oW;
  g.lw = bx.lw; g.lh = bx.lh;
  g.tiles_w = bx.tiles_w; g.tiles_h = bx.tiles_h;
  g.S = y.cS; g.pad = y.cpad;
  g.flip = flip;
  g.chunks_per_tap = chunks_per_tap;
  g.tap_pitch = y.ld_in;
  g.n_per_tap = n_per_tap;
  g.stride = y.cstride;
  g.rs = 1; g.roff_h = g.roff_w = 0;
  g.tap_r0 = g.tap_s0 = 0; g.tap_step = 1; g.tap_ns = y.cS;      // all R x S taps
  return g;
}

// geometry of the halo-tile kernel: 8 x 16 pixel tiles of one image
static ConvGeom halo_geom(const Layer& y, int flip) {
  ConvGeom g{};
  g.kind = GEOM_PIX_M;
  g.H = y.imH; g.W = y.imW;
  g.lw = 3; g.lh = 4;
  g.tiles_w = y.imW / 8; g.tiles_h = y.imH / 16;
  g.S = 3; g.pad = 1;
  g.flip = flip;
  g.chunks_per_tap = 1;
  g.tap_pitch = y.ld_in;
  g.stride = 1;
  g.rs = 1;
  g.tap_step = 1; g.tap_ns = 3;
  return g;
}

// again = false: the forward pass of minibatch n.  again = true: the same task re-run by the backward
// pass (activation recomputation): reads the backward-side slot of its input, writes the backward-side
// slots of the next layer's input, stored z and pooling positions.
static cudaError_t launch_forward(lp_ctx* c, int l, long long n, int ring_slot, cudaStream_t st, bool again = false) {
  Layer& y = c->L[l];
  const int nL = int(c->L.size());
  const bool last = (l == nL - 1);
  const int xin = again ? xb_slot(y, n) : xf_slot(y, n);
  const int xout = last ? 0 : (again ? xb_slot(c->L[l + 1], n) : xf_slot(c->L[l + 1], n));
  GemmArgs a{};
  a.M = y.out_rows; a.N = y.n_out; a.K = y.n_in;
  if (y.conv && !y.patch) {
    const int cpt = (y.ld_in + 63) / 64;
    a.K = y.taps * cpt * GEMM_BK;
    a.g = conv_geom(y, GEOM_PIX_M, y.box128, 0, cpt, 0);
  }
  a.mode = EPI_FPROP;
  a.act = y.d.act;
  a.bias = y.d.has_bias ? y.bring + size_t(ring_slot) * y.ld_out : nullptr;
  a.status = c->status;
  a.tmem_policy = c->tmem_policy;
  a.phase = c->trace_done ? c->status + 8 : nullptr;
  if (last) {
    a.out = nullptr;
    a.out2 = c->zL + size_t(n % kDeltaSlots) * c->cfg.batch * c->ld_cls;
    a.ld_out2 = c->ld_cls;
    a.out2_is_f32 = 1;
  } else if (y.pool) {
    a.out = y.a_full;                 // pooled into the next layer's stash by launch_pool
    a.ld_out = y.ld_out;
  } else {
    Layer& nx = c->L[l + 1];
    a.out = nx.X + size_t(xout) * nx.x_elems;
    a.ld_out = y.ld_out;              // = nx.ld_in for conv -> conv and FC -> FC; a flattened conv output keeps its channel pitch
    if (y.Z && (again || !nx.recomp)) {       // (a layer whose output is recomputed stores z only on the second pass)
      a.out2 = y.Z + size_t(xout) * y.z_elems;
      a.ld_out2 = y.ld_out;
    }
  }
  a.splits = y.split_f; a.partial = y.part_f; a.tile_counter = y.cnt_f;
  ++c->launches;
  TimedScope ts(c, LP_TASK_FORWARD, st, l);
  if (y.lean_f) {
    const CUtensorMap& tmo = y.pool ? y.tm_hf_O[0] : y.tm_hf_O[xout];
    return conv_halo_launch(0, y.tm_f_A[xin], y.tm_f_B[ring_slot], tmo, a, st);
  }
  if (y.halo_f) {
    a.g = halo_geom(y, 0);
    const CUtensorMap& tmo = y.pool ? y.tm_hf_O[0] : y.tm_hf_O[xout];
    return conv_halo_launch(0, y.tm_hf_A[xin], y.tm_f_B[ring_slot], tmo, a, st);
  }
  return gemm_launch(0, y.bn_f, y.tm_f_A[xin], y.tm_f_B[ring_slot], a, st);
}

// 2x2 max pool of layer l's activation into the next layer's stash slot (+ argmax)
static cudaError_t launch_pool(lp_ctx* c, int l, long long n, cudaStream_t st, bool again = false) {
  Layer& y = c->L[l];
  Layer& nx = c->L[l + 1];
  const int xout = again ? xb_slot(nx, n) : xf_slot(nx, n);
  ++c->launches;
  TimedScope ts(c, LP_TASK_FORWARD, st, l);
  return launch_maxpool2(y.a_full, nx.X + size_t(xout) * nx.x_elems, y.pidx + size_t(xout) * y.pidx_elems,
                         c->cfg.batch, y.oH, y.oW, y.ld_out, st);
}

// piece: -1 = the whole contraction; 0 = delta'' (columns [0, split_col)); 1 = delta' (the rest)
static cudaError_t launch_delta(lp_ctx* c, int l, long long n, int ring_slot, cudaStream_t st, int piece = -1) {
  Layer& y = c->L[l];
  Layer& pv = c->L[l - 1];
  GemmArgs a{};
  a.M = y.in_rows; a.N = y.n_in; a.K = y.n_out;
  if (piece == 0) a.N = y.split_col;
  if (piece == 1) a.n_begin = y.split_col;
  if (y.conv) {
    const int cpt = (y.ld_out + 63) / 64;
    a.K = y.taps * cpt * GEMM_BK;
    a.g = conv_geom(y, GEOM_PIX_M, y.boxD, 1, cpt, 0);
  }
  a.act = pv.d.act;
  a.out = pv.delta + size_t(n % kDeltaSlots) * pv.delta_elems;
  a.ld_out = pv.ld_out;
  if (pv.pool) {
    // the layer below ended in ReLU + max pool: the product lives on the pooled grid and is
    // routed back through the recorded argmax, gated by the pooled activation
    a.mode = EPI_DGRAD_UNPOOL;
    a.pool_idx = pv.pidx + size_t(xb_slot(y, n)) * pv.pidx_elems;
    a.pool_C = pv.ld_out;
    a.pool_ppr = y.conv ? 1 : pv.Hp * pv.Wp;
    a.pool_Hp = pv.Hp; a.pool_Wp = pv.Wp;
    a.aux = y.X + size_t(xb_slot(y, n)) * y.x_elems;
    a.ld_aux = pv.ld_out;
  } else {
    a.mode = EPI_DGRAD;
    if (pv.d.act == LP_ACT_GELU) {
      a.aux = pv.Z + size_t(xb_slot(y, n)) * pv.z_elems;    // stored z^{l-1}
      a.ld_aux = pv.ld_out;
    } else {
      a.aux = y.X + size_t(xb_slot(y, n)) * y.x_elems;      // a^{l-1} > 0  <=>  z^{l-1} > 0
      a.ld_aux = y.ld_in;
    }
    if (!y.conv && pv.conv) {
      // FC on a flattened (unpooled) conv output: [B][H*W*C] and [B*H*W][C] are the same memory
      a.ld_out = y.ld_in;
      a.ld_aux = y.ld_in;
    }
  }
  a.status = c->status;
  a.tmem_policy = c->tmem_policy;
  a.phase = c->trace_done ? c->status + 8 : nullptr;
  a.splits = y.split_d; a.partial = y.part_d; a.tile_counter = y.cnt_d;
  ++c->launches;
  TimedScope ts(c, LP_TASK_DELTA, st, l);
  if (y.halo_d) {
    a.g = halo_geom(y, 1);
    return conv_halo_launch(1, y.tm_hd_A[n % kDeltaSlots], y.tm_d_B[ring_slot], y.tm_hd_A[0], a, st);
  }
  if (y.conv && y.cstride > 1) {
    // Strided layer: input pixel (h, w) is reached through tap (r, s) only when h + pad - r and
    // w + pad - s are multiples of the stride.  One launch per residue class of (h, w) modulo the
    // stride: its rows are the pixels of that class, its contraction runs over the taps of that
    // class only -- together the launches do exactly the R * S * Cout multiply-accumulates per
    // input pixel that exist, and each element of delta^{l-1} is written once.
    const int sd = y.cstride, cpt = (y.ld_out + 63) / 64;
    a.M = y.in_rows / (sd * sd);
    for (int ph = 0; ph < sd; ++ph)
      for (int pw = 0; pw < sd; ++pw) {
        const int r0 = (ph + y.cpad) % sd, s0 = (pw + y.cpad) % sd;
        const int nr = r0 < y.cR ? (y.cR - r0 + sd - 1) / sd : 0, ns = s0 < y.cS ? (y.cS - s0 + sd - 1) / sd : 0;
        a.g.rs = sd; a.g.roff_h = ph; a.g.roff_w = pw;
        a.g.tap_r0 = r0; a.g.tap_s0 = s0; a.g.tap_step = sd; a.g.tap_ns = std::max(ns, 1);
        a.K = nr * ns * cpt * GEMM_BK;        // (a class without taps stores f'(.) x 0: K = 0 runs the epilogue on zeros)
        if (ph + pw > 0) ++c->launches;
        cudaError_t e = gemm_launch(1, y.bn_d, y.tm_d_A[n % kDeltaSlots], y.tm_d_B[ring_slot], a, st);
        if (e != cudaSuccess) return e;
      }
    return cudaSuccess;
  }
  return gemm_launch(1, y.bn_d, y.tm_d_A[n % kDeltaSlots], y.tm_d_B[ring_slot], a, st);
}

static inline bool fused_update(const lp_ctx* c) { return (c->cfg.flags & LP_UNFUSED_UPDATE) == 0; }
// The G kernel with the TMA update also does the bias gradient and bias update of a fully connected
// layer (one launch less per layer); convolution layers and the other G forms keep the bias kernel.
static inline bool fused_bias(const lp_ctx* c, const Layer& y) {
  return fused_update(c) && y.upd_maps && y.bn_g != GEMM_BN_PAIR && y.d.has_bias && y.col_chunks == 0 && !y.conv;
}

static cudaError_t launch_G(lp_ctx* c, int l, long long n, cudaStream_t st) {
  Layer& y = c->L[l];
  if (y.halo_g) {
    // 3x3 layer with at most 64 channels: G over 8 x 16 pixel tiles, then the CTAs' partial sums
    // are added in order and Eq. 6 applied (two launches)
    HaloGUpdate u{};
    u.n_out = y.n_out; u.n_in = y.n_in; u.ld_w = y.w_ld; u.tap_pitch = y.ld_in;
    u.G = y.dW;                                   // kept only with LP_CAPTURE_GRADS / LP_UNFUSED_UPDATE
    if (fused_update(c)) {
      u.W = y.W; u.mW = y.mW;
      u.ring = y.ring + size_t((n + 1) % y.slots) * y.w_elems;
      u.lr = c->cfg.lr; u.mu = c->cfg.momentum;
    }
    c->launches += 2 * ((y.n_out + 63) / 64);
    TimedScope ts(c, LP_TASK_G, st, l);
    return conv_halo_g_launch(y.tm_hf_A[xb_slot(y, n)], y.tm_hg_D[n % kDeltaSlots], halo_geom(y, 0), c->cfg.batch, y.part_g,
                              u, c->status, st);
  }
  GemmArgs a{};
  a.M = y.n_out; a.N = y.w_ld; a.K = y.out_rows;      // the contraction runs over the samples / output pixels (delta^l's rows)
  if (!y.conv || y.patch) a.N = y.n_in;
  a.ld_out = y.w_ld;
  a.status = c->status;
  a.tmem_policy = c->tmem_policy;
  a.phase = c->trace_done ? c->status + 8 : nullptr;
  if (y.conv && !y.patch) a.g = conv_geom(y, GEOM_PIX_K, y.box64, 0, 0, (y.ld_in + y.bn_g - 1) / y.bn_g);
  if (y.split_g > 1) { a.splits = y.split_g; a.partial = y.part_g; a.tile_counter = y.cnt_g; }
  if (fused_update(c)) {
    // Eq. 5 and Eq. 6 in one kernel: the accumulator tile is G; the epilogue reads the fp32
    // master (and momentum) tile, applies the update and writes master, momentum and the
    // bf16 version for minibatch n+1 -- G itself only goes to memory when it is captured
    a.mode = EPI_WGRAD_UPDATE;
    a.out = (c->cfg.flags & LP_CAPTURE_GRADS) ? y.dW : nullptr;
    a.W = y.W; a.mW = y.mW;
    a.ring = y.ring + size_t((n + 1) % y.slots) * y.w_elems;
    a.lr = c->cfg.lr; a.mu = c->cfg.momentum;
  } else {
    a.mode = EPI_STORE_F32;
    a.out = y.dW;
  }
  ++c->launches;
  TimedScope ts(c, LP_TASK_G, st, l);
  if (fused_bias(c, y)) {
    a.bdelta = y.delta + size_t(n % kDeltaSlots) * y.delta_elems;
    a.bld = y.ld_out; a.brows = y.out_rows;
    a.bb = y.b; a.bmb = y.mb; a.bdb = y.db;
    a.bbring = y.bring + size_t((n + 1) % y.slots) * y.ld_out;
  }
  if (y.upd_maps && a.mode == EPI_WGRAD_UPDATE) {
    UpdMaps um;
    um.W = y.tm_u_W;
    um.M = y.mW ? y.tm_u_M : y.tm_u_W;
    um.R = y.tm_u_R[(n + 1) % y.slots];
    return gemm_launch(2, y.bn_g, y.tm_g_A[n % kDeltaSlots], y.tm_g_B[xb_slot(y, n)], a, st, &um);
  }
  return gemm_launch(2, y.bn_g, y.tm_g_A[n % kDeltaSlots], y.tm_g_B[xb_slot(y, n)], a, st);
}

static cudaError_t launch_update(lp_ctx* c, int l, long long n, cudaStream_t st) {
  Layer& y = c->L[l];
  const int dst_slot = int((n + 1) % y.slots);
  UpdateArgs u{};
  u.dW = y.dW; u.W = y.W; u.mW = y.mW;
  u.ring = y.ring + size_t(dst_slot) * y.w_elems;
  u.n_elems = fused_update(c) ? 0 : (long long)y.w_elems;   // fused: W was updated by the G kernel
  if (u.n_elems == 0 && !y.d.has_bias) return cudaSuccess;  // nothing left to do
  if (fused_bias(c, y)) return cudaSuccess;                 // the G kernel did the bias as well
  if (y.d.has_bias) {
    u.delta = y.delta + size_t(n % kDeltaSlots) * y.delta_elems;
    u.rows = y.out_rows; u.ldd = y.ld_out; u.n_out = y.n_out;
    u.b = y.b; u.mb = y.mb; u.db = y.db;
    u.bring = y.bring + size_t(dst_slot) * y.ld_out;
    if (y.col_chunks > 0) {
      // many rows (convolution): column sums in two deterministic passes
      ++c->launches;
      cudaError_t e = launch_colsum_partial(u.delta, u.rows, u.ldd, u.n_out, y.col_partial, st);
      if (e != cudaSuccess) return e;
      u.col_partial = y.col_partial;
      u.n_chunks = y.col_chunks;
    }
  }
  u.lr = c->cfg.lr; u.mu = c->cfg.momentum;
  ++c->launches;
  TimedScope ts(c, LP_TASK_UPDATE, st, l);
  return launch_sgd_update(u, st);
}

}  // namespace lp

using namespace lp;

// ===========================================================================
extern "C" int lp_workspace_size(const lp_layer* layers, int n_layers, int n_stages, const int* stage,
                                 const int* delays, const lp_config* cfg, size_t* bytes_out) {
  std::string why;
  if (!bytes_out) return fail(nullptr, LP_ERR_INVALID_ARG, "bytes_out is null");
  int rc = validate(layers, n_layers, cfg, &why);
  if (rc != LP_OK) return fail(nullptr, rc, why);
  std::vector<int> st, dl;
  int used = 0;
  rc = resolve_plan(layers, n_layers, n_stages, stage, delays, cfg, &st, &dl, &used, &why);
  if (rc != LP_OK) return fail(nullptr, rc, why);
  lp_ctx tmp;
  tmp.cfg = *cfg;
  shape_layers(&tmp, layers, n_layers, st, dl);
  *bytes_out = carve(&tmp, nullptr);
  return LP_OK;
}

extern "C" int lp_create(lp_handle* out, const lp_layer* layers, int n_layers, int n_stages, const int* stage,
                         const int* delays, const lp_config* cfg, const float* const* W0_host,
                         const float* const* b0_host, void* workspace_dev, size_t workspace_bytes) {
  std::string why;
  if (!out) return fail(nullptr, LP_ERR_INVALID_ARG, "out is null");
  *out = nullptr;
  if (!W0_host || !workspace_dev) return fail(nullptr, LP_ERR_INVALID_ARG, "W0_host or workspace is null");
  int rc = validate(layers, n_layers, cfg, &why);
  if (rc != LP_OK) return fail(nullptr, rc, why);
  for (int l = 0; l < n_layers; ++l)
    if (!W0_host[l]) return fail(nullptr, LP_ERR_INVALID_ARG, "W0_host[l] is null");
  std::vector<int> st, dl;
  int used = 0;
  rc = resolve_plan(layers, n_layers, n_stages, stage, delays, cfg, &st, &dl, &used, &why);
  if (rc != LP_OK) return fail(nullptr, rc, why);

  int dev = 0;
  cudaDeviceProp prop;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess)
    return fail(nullptr, LP_ERR_CUDA, "no CUDA device");
  if (prop.major != 10) return fail(nullptr, LP_ERR_UNSUPPORTED, "this library needs an sm_100 device");

  std::unique_ptr<lp_ctx, void (*)(lp_ctx*)> c(new lp_ctx, destroy_ctx);
  c->cfg = *cfg;
  c->n_stages = n_stages;
  c->stages_used = used;
  shape_layers(c.get(), layers, n_layers, st, dl);
  const size_t need = carve(c.get(), nullptr);
  if ((reinterpret_cast<uintptr_t>(workspace_dev) & 255) != 0 || workspace_bytes < need)
    return fail(nullptr, LP_ERR_WORKSPACE, "workspace misaligned or smaller than lp_workspace_size");
  c->ws = static_cast<char*>(workspace_dev);
  c->ws_bytes = need;
  carve(c.get(), c->ws);

  lp_ctx* h = c.get();
  LP_CUDA(nullptr, cudaMemset(c->ws, 0, need));
  LP_CUDA(nullptr, gemm_configure());
  int least = 0, greatest = 0;
  LP_CUDA(nullptr, cudaDeviceGetStreamPriorityRange(&least, &greatest));
  // Priorities: G + update highest, delta next, forward lowest.  The paper puts delta first because
  // it carries the critical loop between processors; on one GPU the step time is set by how full
  // the SMs are kept, and the G + update task is the one that hands buffers back (the delta slot,
  // the ring slot of the next version), so starving it stalls later minibatches.  Measured per step
  // with every stream on its own hardware queue and four delta slots, (delta > forward > G) against
  // this order: 8 x 4096 MLP 589 / 588 us, small VGG 478 / 384 us, VGG-16 9.43 / 9.20 ms, 16 x 8192
  // MLP 11.11 / 10.89 ms; all priorities equal lies in between.
  // A network whose kernels are too small to fill the GPU (the 784-256-256-256-10 MLP at batch
  // 32: 0.110 ms per step with delta first, 0.130 ms with G first) is bound by the latency of the
  // delta chain instead, and keeps the paper's order.
  long long step_macs = 0;
  for (int l = 0; l < n_layers; ++l) {
    long long m = 0;
    if (layer_macs(layers[l], cfg->batch, &m) == LP_OK) step_macs += 3 * m;
  }
  const bool g_first = step_macs >= 1000000000ll;
  const int pMid = std::min(least, greatest + 1);
  const int pG = g_first ? greatest : least, pD = g_first ? pMid : greatest, pF = g_first ? least : pMid;
  // Streams only run concurrently while each has a hardware work queue of its own; the process
  // has CUDA_DEVICE_MAX_CONNECTIONS of them (8 unless the variable was set, up to 32, before the
  // CUDA context was created).  Streams that share a queue serialise in enqueue order, which
  // stalls tasks behind unrelated event waits (measured on the 8 x 4096 workload: 24 streams on 8
  // queues 838 us per step, on 32 queues 591 us).  So the stages share as many stream triples as
  // the queues allow, two queues being left to the caller's stream and the default stream.
  int conn = 8;
  if (const char* e = getenv("CUDA_DEVICE_MAX_CONNECTIONS")) conn = std::max(1, std::min(32, atoi(e)));
  c->n_groups = std::max(1, std::min(used, (conn - 2) / 3));
  // A network whose step is bound by the host's enqueue time gains nothing from many stream
  // triples: every cross-stream edge costs an event wait on the host, same-stream order is free.
  // Measured on the 784-256-256-256-10 MLP at batch 32 (samples/s, 1 / 2 / 4 triples): 593 k / 645 k / 582 k.
  if (!g_first) c->n_groups = std::min(c->n_groups, 2);
  if (const char* e = getenv("LP_STREAM_TRIPLES")) c->n_groups = std::max(1, std::min(c->n_groups, atoi(e)));   // experiments: fewer triples
  c->sF.assign(c->n_groups, nullptr);
  c->sD.assign(c->n_groups, nullptr);
  c->sG.assign(c->n_groups, nullptr);
  for (int s = 0; s < c->n_groups; ++s) {
    LP_CUDA(nullptr, cudaStreamCreateWithPriority(&c->sF[s], cudaStreamNonBlocking, pF));
    LP_CUDA(nullptr, cudaStreamCreateWithPriority(&c->sD[s], cudaStreamNonBlocking, pD));
    LP_CUDA(nullptr, cudaStreamCreateWithPriority(&c->sG[s], cudaStreamNonBlocking, pG));
  }
  {
    int max_delay = 0;
    for (int d : dl) max_delay = std::max(max_delay, d);
    const size_t per_step = size_t(5) * n_layers + 8;                  // tasks of one minibatch, with room to spare
    const size_t want = std::max<size_t>(kEventPool, (size_t(max_delay) + 4) * per_step);
    if (want > (size_t(1) << 20)) return fail(nullptr, LP_ERR_UNSUPPORTED, "delays x layers need more than 2^20 scheduler events");
    c->pool.assign(want, nullptr);
  }
  for (auto& e : c->pool) LP_CUDA(nullptr, cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
  c->jpool.assign(64, nullptr);
  for (auto& e : c->jpool) LP_CUDA(nullptr, cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
  c->streams.assign(1, nullptr);
  for (int s = 0; s < c->n_groups; ++s) { c->streams.push_back(c->sF[s]); c->streams.push_back(c->sD[s]); c->streams.push_back(c->sG[s]); }
  c->waited.assign(c->streams.size(), std::vector<long long>(c->streams.size(), 0));
  if (c->cfg.flags & LP_TRACE_TASKS) {
    const size_t ns = c->streams.size();
    LP_CUDA(nullptr, cudaHostAlloc(reinterpret_cast<void**>(&c->trace_done), 2 * ns * sizeof(unsigned), cudaHostAllocMapped));
    LP_CUDA(nullptr, cudaHostAlloc(reinterpret_cast<void**>(&c->peek_host), 128 + 160 * 16 * 4, cudaHostAllocDefault));
    LP_CUDA(nullptr, gemm_set_tmem_table(c->tmem_table));
    LP_CUDA(nullptr, cudaStreamCreateWithFlags(&c->peek_stream, cudaStreamNonBlocking));
    for (size_t i = 0; i < 2 * ns; ++i) c->trace_done[i] = 0;
    c->trace_enq.assign(ns, 0u);
    c->trace_ring.assign(ns, std::vector<lp_ctx::TraceRec>(lp_ctx::kTraceRing));
  }
  if (cfg->flags & LP_TIME_TASKS) {
    c->tpool.assign(2 * 32768, nullptr);
    for (auto& e : c->tpool) LP_CUDA(nullptr, cudaEventCreate(&e));
  }
  c->loss_ev.assign(kLossRing, Ev{});
  c->rZL.assign(kDeltaSlots, Res{});
  c->rLabels.assign(kDeltaSlots, Res{});
  c->log_v.assign(size_t(kLogRing) * n_layers, 0);
  c->log_slot.assign(size_t(kLogRing) * n_layers, 0);

  // initial weights: fp32 master (padded pitch) and version 0 in ring slot 0
  for (int l = 0; l < n_layers; ++l) {
    Layer& y = c->L[l];
    y.rX.assign(y.x_slots, Res{});
    y.rZ.assign(std::max(y.z_slots, 1), Res{});
    y.rDelta.assign(kDeltaSlots, Res{});
    y.rRing.assign(y.slots, Res{});
    y.rPidx.assign(l + 1 < n_layers ? c->L[l + 1].x_slots : 1, Res{});
    // host [out][in] (conv: [Cout][R][S][Cin]) -> device rows of padded pitch ld_in
    LP_CUDA(nullptr, cudaMemcpy2D(y.W, size_t(y.ld_in) * 4, W0_host[l], size_t(y.n_in) * 4, size_t(y.n_in) * 4,
                                  size_t(y.n_out) * y.taps, cudaMemcpyHostToDevice));
    LP_CUDA(nullptr, launch_round_to_bf16(y.W, y.ring, (long long)y.w_elems, 0));
    if (y.d.has_bias && b0_host && b0_host[l]) {
      LP_CUDA(nullptr, cudaMemcpy(y.b, b0_host[l], size_t(y.n_out) * 4, cudaMemcpyHostToDevice));
      LP_CUDA(nullptr, cudaMemcpy(y.bring, b0_host[l], size_t(y.n_out) * 4, cudaMemcpyHostToDevice));
    }
  }
  LP_CUDA(nullptr, cudaDeviceSynchronize());
  rc = build_tensor_maps(h);
  if (rc != LP_OK) { g_err = h->err; return rc; }
  *out = c.release();
  return LP_OK;
}

extern "C" int lp_destroy(lp_handle h) {
  if (!h) return LP_ERR_INVALID_ARG;
  destroy_ctx(h);
  return LP_OK;
}

extern "C" const char* lp_last_error(lp_handle h) { return h ? h->err.c_str() : g_err.c_str(); }

extern "C" int lp_set_tuning(int tile_n, int stages, int split_k) {
  if ((tile_n != 0 && tile_n != 64 && tile_n != 128 && tile_n != 256 && tile_n != GEMM_BN_PAIR && tile_n != GEMM_BN_PAIR224) || stages < 0 || stages > GEMM_MAX_STAGES ||
      split_k < 0 || (split_k & 0xFF) > 64 || (split_k >> 10) != 0)
    return LP_ERR_INVALID_ARG;
  gemm_set_tuning(tile_n, stages, split_k);
  return LP_OK;
}

extern "C" int lp_get_task_time(lp_handle h, int task, long long* launches, double* total_ms) {
  if (!h || task < 0 || task > LP_TASK_CAST) return LP_ERR_INVALID_ARG;
  if (!(h->cfg.flags & LP_TIME_TASKS)) return fail(h, LP_ERR_NOT_READY, "handle was created without LP_TIME_TASKS");
  LP_CUDA(h, cudaDeviceSynchronize());
  double tot = 0.0;
  for (auto& pr : h->timed[task]) {
    float ms = 0.f;
    LP_CUDA(h, cudaEventElapsedTime(&ms, pr.first, pr.second));
    tot += ms;
  }
  if (launches) *launches = (long long)h->timed[task].size();
  if (total_ms) *total_ms = tot;
  return LP_OK;
}

extern "C" int lp_get_task_timeline(lp_handle h, int task, int capacity, float* start_ms, float* end_ms, int* count_out) {
  if (!h || task < 0 || task > LP_TASK_CAST || capacity < 0 || !count_out || (capacity > 0 && (!start_ms || !end_ms)))
    return LP_ERR_INVALID_ARG;
  if (!(h->cfg.flags & LP_TIME_TASKS)) return fail(h, LP_ERR_NOT_READY, "handle was created without LP_TIME_TASKS");
  LP_CUDA(h, cudaDeviceSynchronize());
  *count_out = 0;
  if (h->tpool_next == 0) return LP_OK;
  cudaEvent_t base = h->tpool[0];      // events are handed out in order: the first one since the reset
  int n = 0;
  for (auto& pr : h->timed[task]) {
    if (n >= capacity) break;
    LP_CUDA(h, cudaEventElapsedTime(&start_ms[n], base, pr.first));
    LP_CUDA(h, cudaEventElapsedTime(&end_ms[n], base, pr.second));
    ++n;
  }
  *count_out = n;
  return LP_OK;
}

extern "C" int lp_get_layer_task_time(lp_handle h, int task, int layer, long long* launches, double* total_ms) {
  if (!h || task < 0 || task > LP_TASK_CAST) return LP_ERR_INVALID_ARG;
  if (layer < 0 || layer >= int(h->L.size())) return fail(h, LP_ERR_INVALID_ARG, "layer index out of range");
  if (!(h->cfg.flags & LP_TIME_TASKS)) return fail(h, LP_ERR_NOT_READY, "handle was created without LP_TIME_TASKS");
  LP_CUDA(h, cudaDeviceSynchronize());
  double tot = 0.0;
  long long cnt = 0;
  for (size_t i = 0; i < h->timed[task].size(); ++i) {
    if (h->timed_layer[task][i] != layer) continue;
    float ms = 0.f;
    LP_CUDA(h, cudaEventElapsedTime(&ms, h->timed[task][i].first, h->timed[task][i].second));
    tot += ms;
    ++cnt;
  }
  if (launches) *launches = cnt;
  if (total_ms) *total_ms = tot;
  return LP_OK;
}

extern "C" int lp_set_delta_split(lp_handle h, const int* piece_stage, const long long* piece_amount, int* split_col_out) {
  if (!h || !piece_stage || !piece_amount) return LP_ERR_INVALID_ARG;
  if (h->n_steps != 0) return fail(h, LP_ERR_NOT_READY, "the split must be set before the first lp_step");
  const int nL = int(h->L.size());
  for (int l = 0; l < nL; ++l) {
    const long long a0 = piece_amount[2 * l], a1 = piece_amount[2 * l + 1];
    if (a0 < 0 || a1 < 0) return fail(h, LP_ERR_INVALID_ARG, "negative piece amount");
    for (int k = 0; k < 2; ++k)
      if ((k == 0 ? a0 : a1) > 0 && (piece_stage[2 * l + k] < 0 || piece_stage[2 * l + k] >= h->n_stages))
        return fail(h, LP_ERR_INVALID_ARG, "piece stage outside [0, n_stages)");
  }
  for (int l = 0; l < nL; ++l) {
    Layer& y = h->L[l];
    y.split_col = 0;
    const long long a0 = piece_amount[2 * l], a1 = piece_amount[2 * l + 1];
    if (split_col_out) split_col_out[l] = 0;
    if (l == 0 || a0 == 0 || a1 == 0) continue;        // no delta task, or placed whole
    // The pieces are column ranges of whole tiles: kernels with a single column tile (the halo-tile
    // kernel, narrow layers) and split-K launches (their partial-tile scratch is indexed by the
    // tile number of the whole contraction) keep the contraction in one piece.
    const int wd = gemm_tile_cols(y.bn_d);
    if (y.halo_d || y.split_d > 1 || y.n_in <= wd) continue;
    const int tiles = (y.n_in + wd - 1) / wd;
    long long t0 = (tiles * a0 + (a0 + a1) / 2) / (a0 + a1);        // nearest whole number of tiles for delta''
    t0 = std::max<long long>(1, std::min<long long>(tiles - 1, t0));
    y.split_col = int(t0) * wd;
    y.piece_stage[0] = piece_stage[2 * l];
    y.piece_stage[1] = piece_stage[2 * l + 1];
    if (split_col_out) split_col_out[l] = y.split_col;
  }
  return LP_OK;
}

extern "C" int lp_reset_task_times(lp_handle h) {
  if (!h) return LP_ERR_INVALID_ARG;
  LP_CUDA(h, cudaDeviceSynchronize());
  for (auto& v : h->timed) v.clear();
  for (auto& v : h->timed_layer) v.clear();
  h->tpool_next = 0;
  return LP_OK;
}

extern "C" long long lp_kernel_launches(lp_handle h) { return h ? h->launches : 0; }

extern "C" int lp_step(lp_handle h, const void* batch_dev, const int* labels_dev, void* stream) {
  if (!h) return LP_ERR_INVALID_ARG;
  if (h->latched) return h->latched;
  if (!batch_dev || !labels_dev) return fail(h, LP_ERR_INVALID_ARG, "batch or labels is null");
  lp_ctx* c = h;
  cudaStream_t user = static_cast<cudaStream_t>(stream);
  const long long n = c->n_steps;
  const int nL = int(c->L.size());
  const int B = c->cfg.batch;
  const bool fusedB = (c->cfg.schedule == LP_SCHED_FUSED_B);
  const bool serial = (c->cfg.flags & LP_SERIAL_TASKS) != 0;   // every task on the caller's stream
  const int ds = int(n % kDeltaSlots);
  if (c->streams[0] != user) {            // what the previous caller's stream waited for says nothing about this one
    c->streams[0] = user;
    std::fill(c->waited[0].begin(), c->waited[0].end(), 0ll);
  }

  // version bookkeeping (the integers the parity tests compare bit-exactly)
  std::vector<int> slot(nL);
  for (int l = 0; l < nL; ++l) {
    const long long v = std::max<long long>(0, n - c->L[l].delay);
    slot[l] = int(v % c->L[l].slots);
    c->log_v[size_t(n % kLogRing) * nL + l] = int(v);
    c->log_slot[size_t(n % kLogRing) * nL + l] = slot[l];
  }

  // ---- cast + stash on the caller's stream ----------------------------------
  {
    Layer& y0 = c->L[0];
    Res* rx = &y0.rX[n % y0.x_slots];
    Res* rl = &c->rLabels[ds];
    LP_CUDA(c, task_begin(c, user, {}, {rx, rl}));
    ++c->launches;
    TimedScope ts(c, LP_TASK_CAST, user);
    if (y0.patch && y0.gen)
      LP_CUDA(c, launch_cast_patch_general(batch_dev, c->cfg.input_dtype == LP_BF16, labels_dev,
                                           y0.X + size_t(n % y0.x_slots) * y0.x_elems, c->labels + size_t(ds) * B, B, y0.imH,
                                           y0.imW, y0.c_in, y0.cR, y0.cS, y0.cstride, y0.cpad, y0.oH, y0.oW, y0.ld_in, user));
    else if (y0.patch)
      LP_CUDA(c, launch_cast_patch3x3(batch_dev, c->cfg.input_dtype == LP_BF16, labels_dev,
                                      y0.X + size_t(n % y0.x_slots) * y0.x_elems, c->labels + size_t(ds) * B, B, y0.imH,
                                      y0.imW, y0.c_in, y0.ld_in, user));
    else
      LP_CUDA(c, launch_cast_stash(batch_dev, c->cfg.input_dtype == LP_BF16, labels_dev,
                                   y0.X + size_t(n % y0.x_slots) * y0.x_elems, c->labels + size_t(ds) * B, y0.in_rows, B,
                                   y0.n_in, y0.ld_in, user));
    LP_CUDA(c, task_end(c, user, {}, {rx, rl}, nullptr));
  }
  // ---- forward ---------------------------------------------------------------
  for (int l = 0; l < nL; ++l) {
    Layer& y = c->L[l];
    cudaStream_t st = (serial ? user : c->sF[y.stage % c->n_groups]);
    Res* rin = &y.rX[xf_slot(y, n)];
    Res* rw = &y.rRing[slot[l]];
    const int xo = (l == nL - 1) ? 0 : xf_slot(c->L[l + 1], n);
    Res* rout = (l == nL - 1) ? &c->rZL[ds] : &c->L[l + 1].rX[xo];
    Res* rz = y.Z ? &y.rZ[xo] : nullptr;
    Res* rpool = y.pool ? &y.rPidx[xo] : nullptr;
    Res* rfull = y.pool ? &y.rAfull : nullptr;
    LP_CUDA(c, task_begin(c, st, {rin, rw}, {rout, rz, rpool, rfull}));
    LP_CUDA(c, launch_forward(c, l, n, slot[l], st));
    if (y.pool) LP_CUDA(c, launch_pool(c, l, n, st));
    LP_CUDA(c, task_end(c, st, {rin, rw}, {rout, rz, rpool, rfull}, nullptr));
  }
  // ---- loss and delta^L --------------------------------------------------------
  {
    Layer& yl = c->L[nL - 1];
    cudaStream_t st = (serial ? user : c->sD[yl.stage % c->n_groups]);
    Res* rd = &yl.rDelta[ds];
    LP_CUDA(c, task_begin(c, st, {&c->rZL[ds], &c->rLabels[ds]}, {rd}));
    ++c->launches;
    TimedScope ts(c, LP_TASK_LOSS, st);
    LP_CUDA(c, launch_softmax_xent(c->zL + size_t(ds) * B * c->ld_cls, c->ld_cls, c->labels + size_t(ds) * B,
                                   yl.delta + size_t(ds) * yl.delta_elems, yl.ld_out, c->row_loss + size_t(ds) * B,
                                   c->ticket + ds, c->loss + (n % kLossRing), B, c->classes, c->status, st));
    LP_CUDA(c, task_end(c, st, {&c->rZL[ds], &c->rLabels[ds]}, {rd}, &c->loss_ev[n % kLossRing]));
  }
  // ---- backward: delta and G are independent tasks; update follows G -----------
  for (int l = nL - 1; l >= 0; --l) {
    Layer& y = c->L[l];
    // Activation recomputation: when the backward pass reaches a stage (at its last layer), the
    // forward tasks that produce the recomputed inputs of its layers run again, first layer first,
    // each from the stashed (or just recomputed) input of its own layer and the weight version the
    // forward pass of this minibatch used -- the same kernels on the same operands, hence the same bits.
    if (l == nL - 1 || c->L[l + 1].stage != y.stage) {
      int lo = l;
      while (lo > 0 && c->L[lo - 1].stage == y.stage) --lo;
      for (int k = lo + 1; k <= l; ++k) {
        if (!c->L[k].recomp) continue;
        Layer& src = c->L[k - 1];
        cudaStream_t st = (serial ? user : c->sD[y.stage % c->n_groups]);
        const int xo = xb_slot(c->L[k], n);
        Res* rin = &src.rX[xb_slot(src, n)];
        Res* rwv = &src.rRing[slot[k - 1]];
        Res* rout = &c->L[k].rX[xo];
        Res* rz = src.Z ? &src.rZ[xo] : nullptr;
        Res* rpool = src.pool ? &src.rPidx[xo] : nullptr;
        Res* rfull = src.pool ? &src.rAfull : nullptr;
        LP_CUDA(c, task_begin(c, st, {rin, rwv}, {rout, rz, rpool, rfull}));
        LP_CUDA(c, launch_forward(c, k - 1, n, slot[k - 1], st, true));
        if (src.pool) LP_CUDA(c, launch_pool(c, k - 1, n, st, true));
        LP_CUDA(c, task_end(c, st, {rin, rwv}, {rout, rz, rpool, rfull}, nullptr));
      }
    }
    Res* rdl = &y.rDelta[ds];
    Res* rw = &y.rRing[slot[l]];
    Res* rx = &y.rX[xb_slot(y, n)];
    Res* rnew = &y.rRing[(n + 1) % y.slots];
    Res* rdprev = nullptr;
    Res* raux = nullptr;
    Res* ridx = nullptr;
    if (l > 0) {
      Layer& pv = c->L[l - 1];
      rdprev = &pv.rDelta[ds];
      raux = (pv.d.act == LP_ACT_GELU) ? &pv.rZ[xb_slot(y, n)] : rx;
      if (pv.pool) ridx = &pv.rPidx[xb_slot(y, n)];
    }
    if (fusedB) {
      cudaStream_t st = (serial ? user : c->sD[y.stage % c->n_groups]);
      LP_CUDA(c, task_begin(c, st, {rdl, rw, rx, raux, ridx}, {rdprev, &y.rDW, rnew}));
      if (l > 0 && y.split_col > 0) {      // (one serial task: the pieces follow one another)
        LP_CUDA(c, launch_delta(c, l, n, slot[l], st, 0));
        LP_CUDA(c, launch_delta(c, l, n, slot[l], st, 1));
      } else if (l > 0) {
        LP_CUDA(c, launch_delta(c, l, n, slot[l], st));
      }
      LP_CUDA(c, launch_G(c, l, n, st));
      LP_CUDA(c, launch_update(c, l, n, st));
      LP_CUDA(c, task_end(c, st, {rdl, rw, rx, raux, ridx}, {rdprev, &y.rDW, rnew}, &y.last_update));
    } else {
      if (l > 0 && y.split_col > 0 && !serial) {
        // delta'' on the streams of the stage that holds layer l+1, delta' on this layer's own:
        // two kernels over disjoint column ranges of delta^{l-1}, concurrent; the buffer counts as
        // written when both are done (the second stream joins the first before the event that
        // later tasks wait on)
        cudaStream_t s0 = c->sD[y.piece_stage[0] % c->n_groups], s1 = c->sD[y.piece_stage[1] % c->n_groups];
        LP_CUDA(c, task_begin(c, s0, {rdl, rw, raux, ridx}, {rdprev}));
        LP_CUDA(c, task_begin(c, s1, {rdl, rw, raux, ridx}, {rdprev}));
        LP_CUDA(c, launch_delta(c, l, n, slot[l], s0, 0));
        LP_CUDA(c, launch_delta(c, l, n, slot[l], s1, 1));
        if (s0 != s1) {
          cudaEvent_t e = c->jpool[c->jpool_next++ % c->jpool.size()];
          LP_CUDA(c, cudaEventRecord(e, s0));
          LP_CUDA(c, cudaStreamWaitEvent(s1, e, 0));
        }
        LP_CUDA(c, task_end(c, s1, {rdl, rw, raux, ridx}, {rdprev}, nullptr));
      } else if (l > 0) {
        cudaStream_t st = (serial ? user : c->sD[y.stage % c->n_groups]);
        LP_CUDA(c, task_begin(c, st, {rdl, rw, raux, ridx}, {rdprev}));
        if (y.split_col > 0) {
          LP_CUDA(c, launch_delta(c, l, n, slot[l], st, 0));
          LP_CUDA(c, launch_delta(c, l, n, slot[l], st, 1));
        } else {
          LP_CUDA(c, launch_delta(c, l, n, slot[l], st));
        }
        LP_CUDA(c, task_end(c, st, {rdl, rw, raux, ridx}, {rdprev}, nullptr));
      }
      cudaStream_t sg = (serial ? user : c->sG[y.stage % c->n_groups]);
      if (fused_update(c)) {
        // G + update of W in one kernel, then the bias update: one task that writes the ring
        // slot of version n+1 (the slot delta_l(n) reads, so the tracker orders it after it)
        LP_CUDA(c, task_begin(c, sg, {rdl, rx}, {&y.rDW, rnew}));
        LP_CUDA(c, launch_G(c, l, n, sg));
        LP_CUDA(c, launch_update(c, l, n, sg));
        LP_CUDA(c, task_end(c, sg, {rdl, rx}, {&y.rDW, rnew}, &y.last_update));
      } else {
        LP_CUDA(c, task_begin(c, sg, {rdl, rx}, {&y.rDW}));
        LP_CUDA(c, launch_G(c, l, n, sg));
        LP_CUDA(c, task_end(c, sg, {rdl, rx}, {&y.rDW}, nullptr));
        LP_CUDA(c, task_begin(c, sg, {&y.rDW, rdl}, {rnew}));
        LP_CUDA(c, launch_update(c, l, n, sg));
        LP_CUDA(c, task_end(c, sg, {&y.rDW, rdl}, {rnew}, &y.last_update));
      }
    }
  }
  c->n_steps = n + 1;
  return LP_OK;
}

extern "C" int lp_flush(lp_handle h, void* stream) {
  if (!h) return LP_ERR_INVALID_ARG;
  if (h->latched) return h->latched;
  cudaStream_t user = static_cast<cudaStream_t>(stream);
  auto join = [&](std::vector<cudaStream_t>& v) -> cudaError_t {
    for (cudaStream_t s : v) {
      cudaEvent_t e = h->jpool[h->jpool_next++ % h->jpool.size()];
      cudaError_t r = cudaEventRecord(e, s);
      if (r != cudaSuccess) return r;
      r = cudaStreamWaitEvent(user, e, 0);
      if (r != cudaSuccess) return r;
    }
    return cudaSuccess;
  };
  LP_CUDA(h, join(h->sF));
  LP_CUDA(h, join(h->sD));
  LP_CUDA(h, join(h->sG));
  return LP_OK;
}

extern "C" int lp_get_weights(lp_handle h, int layer, float* W_out, float* b_out, long long* version) {
  if (!h) return LP_ERR_INVALID_ARG;
  if (layer < 0 || layer >= int(h->L.size())) return fail(h, LP_ERR_INVALID_ARG, "layer index out of range");
  Layer& y = h->L[layer];
  if (y.last_update.e) LP_CUDA(h, cudaEventSynchronize(y.last_update.e));
  if (W_out)
    LP_CUDA(h, cudaMemcpy2D(W_out, size_t(y.n_in) * 4, y.W, size_t(y.ld_in) * 4, size_t(y.n_in) * 4,
                            size_t(y.n_out) * y.taps, cudaMemcpyDeviceToHost));
  if (b_out) LP_CUDA(h, cudaMemcpy(b_out, y.b, size_t(y.n_out) * 4, cudaMemcpyDeviceToHost));
  if (version) *version = h->n_steps;
  return LP_OK;
}

extern "C" int lp_get_grads(lp_handle h, int layer, long long step, float* dW_out, float* db_out) {
  if (!h) return LP_ERR_INVALID_ARG;
  if (layer < 0 || layer >= int(h->L.size())) return fail(h, LP_ERR_INVALID_ARG, "layer index out of range");
  if (step != h->n_steps - 1 || step < 0) return fail(h, LP_ERR_NOT_READY, "only the latest step's gradients are held");
  Layer& y = h->L[layer];
  if (dW_out && !y.dW) return fail(h, LP_ERR_NOT_READY, "G is not kept: create the handle with LP_CAPTURE_GRADS");
  if (y.last_update.e) LP_CUDA(h, cudaEventSynchronize(y.last_update.e));
  if (dW_out)
    LP_CUDA(h, cudaMemcpy2D(dW_out, size_t(y.n_in) * 4, y.dW, size_t(y.ld_in) * 4, size_t(y.n_in) * 4,
                            size_t(y.n_out) * y.taps, cudaMemcpyDeviceToHost));
  if (db_out) LP_CUDA(h, cudaMemcpy(db_out, y.db, size_t(y.n_out) * 4, cudaMemcpyDeviceToHost));
  return LP_OK;
}

namespace lp {
struct BufView {
  void* ptr = nullptr;
  int rows = 0, cols = 0, ld = 0;
  int dtype = 0;   // 0 bf16, 1 f32, 2 i32, 3 u8
};
static int locate(lp_ctx* h, int buffer, int layer, long long index, BufView* v) {
  const int nL = int(h->L.size());
  const int B = h->cfg.batch;
  if (index < 0) return fail(h, LP_ERR_INVALID_ARG, "negative index");
  if (buffer == LP_BUF_LOGITS) {
    *v = {h->zL + size_t(index % kDeltaSlots) * B * h->ld_cls, B, h->classes, h->ld_cls, 1};
    return LP_OK;
  }
  if (buffer == LP_BUF_LABELS) { *v = {h->labels + size_t(index % kDeltaSlots) * B, 1, B, B, 2}; return LP_OK; }
  if (buffer == LP_BUF_LOSS) { *v = {h->loss + (index % kLossRing), 1, 1, 1, 1}; return LP_OK; }
  if (layer < 0 || layer >= nL) return fail(h, LP_ERR_INVALID_ARG, "layer index out of range");
  Layer& y = h->L[layer];
  const int wr = y.n_out * y.taps;     // weight-shaped buffers as [Cout * taps][Cin] with pitch ld_in
  switch (buffer) {
    case LP_BUF_INPUT: *v = {y.X + size_t(xb_slot(y, index)) * y.x_elems, y.in_rows, y.n_in, y.ld_in, 0}; return LP_OK;
    case LP_BUF_Z:
      if (!y.Z) return fail(h, LP_ERR_NOT_READY, "this layer stores no pre-activation");
      *v = {y.Z + size_t(xb_slot(h->L[layer + 1], index)) * y.z_elems, B, y.n_out, y.ld_out, 0};
      return LP_OK;
    case LP_BUF_DELTA: *v = {y.delta + size_t(index % kDeltaSlots) * y.delta_elems, y.out_rows, y.n_out, y.ld_out, 0}; return LP_OK;
    case LP_BUF_POOL_IDX:
      if (!y.pidx) return fail(h, LP_ERR_NOT_READY, "this layer does not pool");
      *v = {y.pidx + size_t(xb_slot(h->L[layer + 1], index)) * y.pidx_elems, B * y.Hp * y.Wp, y.n_out, y.ld_out, 3};
      return LP_OK;
    case LP_BUF_RING_W:
      if (index >= y.slots) return fail(h, LP_ERR_INVALID_ARG, "ring slot out of range");
      *v = {y.ring + size_t(index) * y.w_elems, wr, y.n_in, y.ld_in, 0};
      return LP_OK;
    case LP_BUF_RING_B:
      if (index >= y.slots) return fail(h, LP_ERR_INVALID_ARG, "ring slot out of range");
      *v = {y.bring + size_t(index) * y.ld_out, 1, y.n_out, y.ld_out, 1};
      return LP_OK;
    case LP_BUF_MASTER_W: *v = {y.W, wr, y.n_in, y.ld_in, 1}; return LP_OK;
    case LP_BUF_MASTER_B: *v = {y.b, 1, y.n_out, y.ld_out, 1}; return LP_OK;
    case LP_BUF_MOM_W:
      if (!y.mW) return fail(h, LP_ERR_NOT_READY, "momentum is off");
      *v = {y.mW, wr, y.n_in, y.ld_in, 1};
      return LP_OK;
    case LP_BUF_MOM_B:
      if (!y.mb) return fail(h, LP_ERR_NOT_READY, "momentum is off");
      *v = {y.mb, 1, y.n_out, y.ld_out, 1};
      return LP_OK;
    case LP_BUF_GRAD_W:
      if (!y.dW) return fail(h, LP_ERR_NOT_READY, "G is not kept: create the handle with LP_CAPTURE_GRADS");
      *v = {y.dW, wr, y.n_in, y.ld_in, 1};
      return LP_OK;
    case LP_BUF_GRAD_B: *v = {y.db, 1, y.n_out, y.ld_out, 1}; return LP_OK;
  }
  return fail(h, LP_ERR_INVALID_ARG, "unknown buffer");
}
static inline uint16_t f32_to_bf16_rn(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  if ((u & 0x7FFFFFFFu) > 0x7F800000u) return uint16_t((u >> 16) | 0x40);
  u += 0x7FFFu + ((u >> 16) & 1u);
  return uint16_t(u >> 16);
}
// The patch layer's stash seen from the host as the image it was built from, NHWC [B][H][W][Cin]:
// a write builds every output pixel's patch row; a read returns the image from the taps that hold
// each pixel (stride 1 with the centre tap inside the filter only).
static int patch_io(lp_ctx* h, long long index, const float* in_host, float* out_host) {
  Layer& y = h->L[0];
  const int B = h->cfg.batch, H = y.imH, W = y.imW, C = y.c_in, ld = y.ld_in;
  const int R = y.cR, S = y.cS, sd = y.cstride, pad = y.cpad, Ho = y.oH, Wo = y.oW;
  __nv_bfloat16* dev = y.X + size_t(index % y.x_slots) * y.x_elems;
  std::vector<uint16_t> tmp(y.x_elems, 0);
  LP_CUDA(h, cudaDeviceSynchronize());
  if (out_host) {
    if (sd != 1 || pad >= R || pad >= S || Ho != H || Wo != W)
      return fail(h, LP_ERR_UNSUPPORTED, "the patch matrix of this layer does not hold every input pixel at a fixed tap");
    LP_CUDA(h, cudaMemcpy(tmp.data(), dev, tmp.size() * 2, cudaMemcpyDeviceToHost));
    const int centre = pad * S + pad;            // tap (pad, pad) of output pixel (h, w) is input pixel (h, w)
    for (size_t pix = 0; pix < size_t(B) * H * W; ++pix)
      for (int ch = 0; ch < C; ++ch) {
        const uint32_t bits = uint32_t(tmp[pix * ld + centre * C + ch]) << 16;
        memcpy(&out_host[pix * C + ch], &bits, 4);
      }
    return LP_OK;
  }
  for (int b = 0; b < B; ++b)
    for (int ho = 0; ho < Ho; ++ho)
      for (int wo = 0; wo < Wo; ++wo) {
        uint16_t* row = &tmp[((size_t(b) * Ho + ho) * Wo + wo) * ld];
        for (int tap = 0; tap < R * S; ++tap) {
          const int sh = ho * sd + tap / S - pad, sw = wo * sd + tap % S - pad;
          if (sh < 0 || sh >= H || sw < 0 || sw >= W) continue;
          const float* src = in_host + ((size_t(b) * H + sh) * W + sw) * C;
          for (int ch = 0; ch < C; ++ch) row[tap * C + ch] = f32_to_bf16_rn(src[ch]);
        }
      }
  LP_CUDA(h, cudaMemcpy(dev, tmp.data(), tmp.size() * 2, cudaMemcpyHostToDevice));
  return LP_OK;
}
}  // namespace lp

extern "C" int lp_debug_read(lp_handle h, int buffer, int layer, long long index, float* out_host) {
  if (!h || !out_host) return LP_ERR_INVALID_ARG;
  if (buffer == LP_BUF_INPUT && layer == 0 && index >= 0 && h->L[0].patch) return patch_io(h, index, nullptr, out_host);
  BufView v;
  int rc = locate(h, buffer, layer, index, &v);
  if (rc != LP_OK) return rc;
  LP_CUDA(h, cudaDeviceSynchronize());
  if (v.dtype == 1) {
    LP_CUDA(h, cudaMemcpy2D(out_host, size_t(v.cols) * 4, v.ptr, size_t(v.ld) * 4, size_t(v.cols) * 4, v.rows,
                            cudaMemcpyDeviceToHost));
    return LP_OK;
  }
  if (v.dtype == 2) {
    std::vector<int> tmp(v.cols);
    LP_CUDA(h, cudaMemcpy(tmp.data(), v.ptr, size_t(v.cols) * 4, cudaMemcpyDeviceToHost));
    for (int c = 0; c < v.cols; ++c) out_host[c] = float(tmp[c]);
    return LP_OK;
  }
  if (v.dtype == 3) {
    std::vector<unsigned char> tmp(size_t(v.rows) * v.ld);
    LP_CUDA(h, cudaMemcpy(tmp.data(), v.ptr, tmp.size(), cudaMemcpyDeviceToHost));
    for (int r = 0; r < v.rows; ++r)
      for (int c = 0; c < v.cols; ++c) out_host[size_t(r) * v.cols + c] = float(tmp[size_t(r) * v.ld + c]);
    return LP_OK;
  }
  std::vector<uint16_t> tmp(size_t(v.rows) * v.ld);
  LP_CUDA(h, cudaMemcpy(tmp.data(), v.ptr, tmp.size() * 2, cudaMemcpyDeviceToHost));
  for (int r = 0; r < v.rows; ++r)
    for (int c = 0; c < v.cols; ++c) {
      const uint32_t bits = uint32_t(tmp[size_t(r) * v.ld + c]) << 16;
      memcpy(&out_host[size_t(r) * v.cols + c], &bits, 4);
    }
  return LP_OK;
}

extern "C" int lp_debug_write(lp_handle h, int buffer, int layer, long long index, const float* in_host) {
  if (!h || !in_host) return LP_ERR_INVALID_ARG;
  if (buffer == LP_BUF_INPUT && layer == 0 && index >= 0 && h->L[0].patch) return patch_io(h, index, in_host, nullptr);
  BufView v;
  int rc = locate(h, buffer, layer, index, &v);
  if (rc != LP_OK) return rc;
  LP_CUDA(h, cudaDeviceSynchronize());
  if (v.dtype == 1) {
    LP_CUDA(h, cudaMemcpy2D(v.ptr, size_t(v.ld) * 4, in_host, size_t(v.cols) * 4, size_t(v.cols) * 4, v.rows,
                            cudaMemcpyHostToDevice));
    return LP_OK;
  }
  if (v.dtype == 2) {
    std::vector<int> tmp(v.cols);
    for (int c = 0; c < v.cols; ++c) tmp[c] = int(in_host[c]);
    LP_CUDA(h, cudaMemcpy(v.ptr, tmp.data(), size_t(v.cols) * 4, cudaMemcpyHostToDevice));
    return LP_OK;
  }
  if (v.dtype == 3) {
    std::vector<unsigned char> tmp(size_t(v.rows) * v.ld, 0);
    for (int r = 0; r < v.rows; ++r)
      for (int c = 0; c < v.cols; ++c) tmp[size_t(r) * v.ld + c] = (unsigned char)(in_host[size_t(r) * v.cols + c]);
    LP_CUDA(h, cudaMemcpy(v.ptr, tmp.data(), tmp.size(), cudaMemcpyHostToDevice));
    return LP_OK;
  }
  std::vector<uint16_t> tmp(size_t(v.rows) * v.ld, 0);
  for (int r = 0; r < v.rows; ++r)
    for (int c = 0; c < v.cols; ++c) tmp[size_t(r) * v.ld + c] = f32_to_bf16_rn(in_host[size_t(r) * v.cols + c]);
  LP_CUDA(h, cudaMemcpy(v.ptr, tmp.data(), tmp.size() * 2, cudaMemcpyHostToDevice));
  return LP_OK;
}

extern "C" int lp_debug_run_task(lp_handle h, int task, int layer, long long step) {
  if (!h) return LP_ERR_INVALID_ARG;
  if (h->latched) return h->latched;
  const int nL = int(h->L.size());
  if (step < 0) return fail(h, LP_ERR_INVALID_ARG, "negative step");
  if (task != LP_TASK_LOSS && (layer < 0 || layer >= nL)) return fail(h, LP_ERR_INVALID_ARG, "layer index out of range");
  LP_CUDA(h, cudaDeviceSynchronize());
  cudaStream_t st = h->sF[0];
  const int B = h->cfg.batch;
  const int ds = int(step % kDeltaSlots);
  int slot = 0;
  if (task != LP_TASK_LOSS) {
    Layer& y = h->L[layer];
    slot = int(std::max<long long>(0, step - y.delay) % y.slots);
  }
  switch (task) {
    case LP_TASK_FORWARD:
      LP_CUDA(h, launch_forward(h, layer, step, slot, st));
      if (h->L[layer].pool) LP_CUDA(h, launch_pool(h, layer, step, st));
      break;
    case LP_TASK_LOSS: {
      Layer& yl = h->L[nL - 1];
      ++h->launches;
      LP_CUDA(h, launch_softmax_xent(h->zL + size_t(ds) * B * h->ld_cls, h->ld_cls, h->labels + size_t(ds) * B,
                                     yl.delta + size_t(ds) * yl.delta_elems, yl.ld_out, h->row_loss + size_t(ds) * B,
                                     h->ticket + ds, h->loss + (step % kLossRing), B, h->classes, h->status, st));
      break;
    }
    case LP_TASK_DELTA:
      if (layer < 1) return fail(h, LP_ERR_INVALID_ARG, "the first layer has no delta task");
      if (h->L[layer].split_col > 0) {
        LP_CUDA(h, launch_delta(h, layer, step, slot, st, 0));
        LP_CUDA(h, launch_delta(h, layer, step, slot, st, 1));
      } else {
        LP_CUDA(h, launch_delta(h, layer, step, slot, st));
      }
      break;
    case LP_TASK_G: LP_CUDA(h, launch_G(h, layer, step, st)); break;
    case LP_TASK_UPDATE: LP_CUDA(h, launch_update(h, layer, step, st)); break;
    default: return fail(h, LP_ERR_INVALID_ARG, "unknown task");
  }
  LP_CUDA(h, cudaStreamSynchronize(st));
  return LP_OK;
}

extern "C" int lp_get_schedule(lp_handle h, int* stage, int* delay, int* ring_slots) {
  if (!h) return LP_ERR_INVALID_ARG;
  for (size_t l = 0; l < h->L.size(); ++l) {
    if (stage) stage[l] = h->L[l].stage;
    if (delay) delay[l] = h->L[l].delay;
    if (ring_slots) ring_slots[l] = h->L[l].slots;
  }
  return LP_OK;
}

extern "C" int lp_get_version_log(lp_handle h, long long step, int* v_fwd, int* v_bwd, int* slot) {
  if (!h) return LP_ERR_INVALID_ARG;
  if (step < 0 || step >= h->n_steps || step < h->n_steps - kLogRing)
    return fail(h, LP_ERR_NOT_READY, "step outside the version log");
  const size_t nL = h->L.size();
  for (size_t l = 0; l < nL; ++l) {
    const int v = h->log_v[size_t(step % kLogRing) * nL + l];
    if (v_fwd) v_fwd[l] = v;
    if (v_bwd) v_bwd[l] = v;      // weight stashing: delta reads the version the forward pass read
    if (slot) slot[l] = h->log_slot[size_t(step % kLogRing) * nL + l];
  }
  return LP_OK;
}

extern "C" int lp_get_loss(lp_handle h, long long step, float* loss) {
  if (!h || !loss) return LP_ERR_INVALID_ARG;
  if (step < 0 || step >= h->n_steps || step < h->n_steps - kLossRing)
    return fail(h, LP_ERR_NOT_READY, "step outside the loss ring");
  const Ev& e = h->loss_ev[step % kLossRing];
  if (e.e) LP_CUDA(h, cudaEventSynchronize(e.e));
  LP_CUDA(h, cudaMemcpy(loss, h->loss + (step % kLossRing), 4, cudaMemcpyDeviceToHost));
  return LP_OK;
}

extern "C" int lp_task_progress(lp_handle h, char* text, int capacity) {
  if (!h || !text || capacity < 1) return LP_ERR_INVALID_ARG;
  if (!h->trace_done) return fail(h, LP_ERR_NOT_READY, "the handle was created without LP_TRACE_TASKS");
  static const char* kinds[6] = {"forward", "loss", "delta", "G", "update", "cast"};
  std::string out;
  char line[400];
  for (size_t si = 0; si < h->streams.size(); ++si) {
    const unsigned done = *reinterpret_cast<volatile unsigned*>(h->trace_done + si), enq = h->trace_enq[si];
    if (done == enq) continue;
    const char* role = si == 0 ? "caller" : ((si - 1) % 3 == 0 ? "F" : (si - 1) % 3 == 1 ? "delta" : "G");
    const unsigned started = *reinterpret_cast<volatile unsigned*>(h->trace_done + h->streams.size() + si);
    snprintf(line, sizeof line, "stream %d (%s, triple %d): %u of %u tasks done, %s; unfinished:", int(si), role,
             si == 0 ? -1 : int((si - 1) / 3), done, enq, started > done ? "the next one has STARTED" : "the next one has not started");
    out += line;
    for (unsigned q = done + 1; q <= enq && q <= done + 3; ++q) {
      if (enq - q >= unsigned(lp_ctx::kTraceRing)) continue;
      const lp_ctx::TraceRec& r = h->trace_ring[si][q % lp_ctx::kTraceRing];
      snprintf(line, sizeof line, " %s(layer %d, minibatch %lld)", r.kind >= 0 && r.kind < 6 ? kinds[r.kind] : "?", r.layer, r.n);
      out += line;
    }
    out += "\n";
  }
  // the status word, read on a stream of its own: works while the scheduler's streams are stuck
  if (cudaMemcpyAsync(h->peek_host, h->status, 128, cudaMemcpyDeviceToHost, h->peek_stream) == cudaSuccess &&
      cudaStreamSynchronize(h->peek_stream) == cudaSuccess) {
    snprintf(line, sizeof line, "status word %d\n", h->peek_host[0]);
    out += line;
    const int* ph = h->peek_host + 8;
    snprintf(line, sizeof line, "pair-kernel CTAs past: entry %d, allocation %d, first cluster barrier %d, loads %d, MMAs (leaders) %d, "
             "epilogue %d, last cluster barrier %d, release %d\n", ph[0], ph[1], ph[2], ph[3], ph[4], ph[5], ph[6], ph[7]);
    out += line;
    snprintf(line, sizeof line, "tensor-memory allocations that waited more than 20000 cycles: %d of %d single-CTA, %d of %d pair CTAs\n",
             ph[8], ph[9], ph[10], ph[1]);
    out += line;
  }
  if (cudaMemcpyAsync(h->peek_host + 32, h->tmem_table, 160 * 16 * 4, cudaMemcpyDeviceToHost, h->peek_stream) == cudaSuccess &&
      cudaStreamSynchronize(h->peek_stream) == cudaSuccess) {
    static const char* tk[8] = {"-", "gemm", "gemm persistent", "pair", "pair G", "pair forward/delta", "halo", "halo G"};
    for (int sm = 0; sm < 160; ++sm) {
      const int* r = h->peek_host + 32 + 16 * sm;
      for (int k = 1; k < 8; ++k)
        if (r[k] != 0) {
          snprintf(line, sizeof line, "SM %d: %d CTA(s) of kernel '%s' inside tcgen05.alloc; this library's CTAs hold %d columns there; "
                   "latest deallocation by '%s', latest allocation by '%s', %d allocations so far\n",
                   sm, r[k], tk[k], r[8], tk[r[9] & 7], tk[r[10] & 7], r[11]);
          out += line;
        }
    }
  }
  if (out.empty()) out = "idle\n";
  snprintf(text, size_t(capacity), "%s", out.c_str());
  return LP_OK;
}

extern "C" int lp_device_status(lp_handle h, int* detail) {
  if (!h) return LP_ERR_INVALID_ARG;
  LP_CUDA(h, cudaDeviceSynchronize());
  int st = 0;
  LP_CUDA(h, cudaMemcpy(&st, h->status, 4, cudaMemcpyDeviceToHost));
  if (detail) *detail = st;
  if (st == LP_STATUS_BAD_LABEL)
    return fail(h, LP_ERR_INVALID_ARG, "a label outside [0, classes) reached the loss kernel (that minibatch's loss is NaN)");
  if (st != 0) return fail(h, LP_ERR_TIMEOUT, "a bounded device-side wait expired (status " + std::to_string(st) + ")");
  return LP_OK;
}
